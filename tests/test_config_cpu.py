"""Host-side configuration front end, pinned to the two examples the paper prints."""
import os

import pytest
import torch

from paper_2603_06588_b200 import config

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_layer_heads_string_matches_the_papers_example():
    line = [l for l in open(os.path.join(GOLDEN, "layer_heads_example.txt")) if l.strip() and not l.startswith("#")][0]
    text, want_s = (x.strip() for x in line.split("=>"))
    want = {int(p.split(":")[0]): [int(h) for h in p.split(":")[1].split(",")] for p in want_s.split("|")}
    assert want == {0: [0, 3, 6], 15: [2]}
    got = config.parse_layer_heads(text)
    assert got == want
    assert config.format_layer_heads(got) == text
    assert config.parse_layer_heads(config.format_layer_heads(got)) == got


def test_layer_heads_edge_cases():
    assert config.parse_layer_heads("") == {}
    assert config.parse_layer_heads(" 3 : 1 , 1, 2 ;; 3:7 ") == {3: [1, 2, 7]}
    for bad in ("3", "a:1", "1:x", "-1:2", "1:-2"):
        with pytest.raises(ValueError):
            config.parse_layer_heads(bad)


def test_json_config_matches_the_papers_example():
    cfg = config.load_hook_config(os.path.join(GOLDEN, "config_example.json"))
    assert cfg.name == "granite3-8b-attn" and cfg.model_id == "ibm-granite/granite-3.1-8b-instruct"
    assert cfg.hookq_mode == "last_token" and cfg.probe_rows == config.PROBE_ROWS_LAST
    assert sum(len(v) for v in cfg.layer_to_heads.values()) == 41
    assert cfg.important_layers == [6, 7, 8] + list(range(10, 20)) and 9 not in cfg.layer_to_heads
    assert cfg.layer_to_heads[8] == [1, 13, 14, 15] and cfg.layer_to_heads[19] == [1]
    # head indices reach 31: they index the query heads of a 32-head model
    assert max(max(v) for v in cfg.layer_to_heads.values()) == 31
    m = cfg.head_mask(11, 32)
    assert m.dtype == torch.uint8 and m.nonzero().flatten().tolist() == [4, 30, 31]
    assert cfg.head_mask(0, 32) is None and cfg.probed_heads(17) == [7, 11, 15, 19, 21, 25, 26]
    with pytest.raises(ValueError):
        cfg.head_mask(11, 16)
    assert config.parse_layer_heads(cfg.to_env_string()) == cfg.layer_to_heads


def test_defaults_and_errors():
    cfg = config.load_hook_config({"params": {"important_heads": [[0, 1], [0, 1], [2, 0]]}})
    assert cfg.hookq_mode == "all_tokens" and cfg.probe_rows == config.PROBE_ROWS_ALL
    assert cfg.layer_to_heads == {0: [1], 2: [0]}
    with pytest.raises(ValueError):
        config.load_hook_config({"hookq": {"hookq_mode": "first_token"}})
    with pytest.raises(ValueError):
        config.load_hook_config({"params": {"important_heads": [[1, 2, 3]]}})
    assert config.load_hook_config('{"hookq": {"hookq_mode": "last_token"}}').probe_rows == 1
