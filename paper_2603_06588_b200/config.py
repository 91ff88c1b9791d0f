"""Host-side front end of the hook configuration.

The paper configures its hooks with a JSON file (Section 2: ``model_info``,
``params/important_heads`` as ``[layer, head]`` pairs, ``hookq/hookq_mode``) and carries the
per-layer head sets into the worker process as a string such as ``'0:0,3,6;15:2'``
(Section 2.1).  This module parses both and turns them into what the kernels take per layer
call: a ``uint8`` query-head mask and the probe-row mode.  Pure host code, no arithmetic of the
attention path.
"""
from __future__ import annotations

import json
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple, Union

import torch

PROBE_ROWS_ALL = 0
PROBE_ROWS_LAST = 1
_MODES = {"all_tokens": PROBE_ROWS_ALL, "last_token": PROBE_ROWS_LAST}


def parse_layer_heads(text: str) -> Dict[int, List[int]]:
    """``'0:0,3,6;15:2'`` -> ``{0: [0, 3, 6], 15: [2]}``.  Layers are separated by ``;``, a layer
    and its heads by ``:``, heads by ``,``.  Empty input gives an empty mapping; repeated layers
    are merged; heads keep first-seen order without duplicates."""
    out: Dict[int, List[int]] = {}
    for part in text.split(";"):
        part = part.strip()
        if not part:
            continue
        if ":" not in part:
            raise ValueError(f"expected '<layer>:<head>,<head>...' but got {part!r}")
        layer_s, heads_s = part.split(":", 1)
        layer = int(layer_s)
        if layer < 0:
            raise ValueError(f"negative layer index in {part!r}")
        heads = out.setdefault(layer, [])
        for hs in heads_s.split(","):
            hs = hs.strip()
            if not hs:
                continue
            h = int(hs)
            if h < 0:
                raise ValueError(f"negative head index in {part!r}")
            if h not in heads:
                heads.append(h)
    return out


def format_layer_heads(layer_to_heads: Dict[int, Sequence[int]]) -> str:
    """Inverse of :func:`parse_layer_heads` (layers in ascending order)."""
    return ";".join(f"{layer}:{','.join(str(h) for h in layer_to_heads[layer])}"
                    for layer in sorted(layer_to_heads) if len(layer_to_heads[layer]))


def pairs_to_layer_heads(pairs: Sequence[Sequence[int]]) -> Dict[int, List[int]]:
    """``[[layer, head], ...]`` (the config's ``important_heads``) -> ``{layer: [heads]}``."""
    out: Dict[int, List[int]] = {}
    for pair in pairs:
        if len(pair) != 2:
            raise ValueError(f"important_heads entries are [layer, head] pairs, got {pair!r}")
        layer, head = int(pair[0]), int(pair[1])
        if layer < 0 or head < 0:
            raise ValueError(f"negative index in {pair!r}")
        heads = out.setdefault(layer, [])
        if head not in heads:
            heads.append(head)
    return out


@dataclass
class HookConfig:
    name: str = ""
    model_id: str = ""
    layer_to_heads: Dict[int, List[int]] = field(default_factory=dict)
    hookq_mode: str = "all_tokens"        # the worker's default when the variable is unset

    @property
    def probe_rows(self) -> int:
        return _MODES[self.hookq_mode]

    @property
    def important_layers(self) -> List[int]:
        return sorted(self.layer_to_heads)

    def head_mask(self, layer: int, num_q_heads: int) -> Optional[torch.Tensor]:
        """uint8 ``[num_q_heads]`` mask of the probed query heads of ``layer`` (``None`` when the
        layer is not hooked, which makes "hooks disabled" a launch-time fact)."""
        heads = self.layer_to_heads.get(int(layer))
        if not heads:
            return None
        mask = torch.zeros(num_q_heads, dtype=torch.uint8)
        for h in heads:
            if h >= num_q_heads:
                raise ValueError(f"head {h} of layer {layer} is outside a model with {num_q_heads} query heads")
            mask[h] = 1
        return mask

    def probed_heads(self, layer: int) -> List[int]:
        """Probed heads of ``layer`` in ascending order: slot ``i`` of ``span_mass`` is ``probed_heads[i]``."""
        return sorted(self.layer_to_heads.get(int(layer), []))

    def to_env_string(self) -> str:
        return format_layer_heads(self.layer_to_heads)


def load_hook_config(source: Union[str, dict]) -> HookConfig:
    """Parse a configuration given as a dict, a JSON string, or a path to a JSON file."""
    if isinstance(source, dict):
        cfg = source
    else:
        text = source
        if not source.lstrip().startswith("{"):
            with open(source) as f:
                text = f.read()
        cfg = json.loads(text)
    info = cfg.get("model_info", {})
    pairs = cfg.get("params", {}).get("important_heads", [])
    mode = cfg.get("hookq", {}).get("hookq_mode", "all_tokens")
    if mode not in _MODES:
        raise ValueError(f"hookq_mode must be one of {sorted(_MODES)}, got {mode!r}")
    return HookConfig(name=str(info.get("name", "")), model_id=str(info.get("model_id", "")),
                      layer_to_heads=pairs_to_layer_heads(pairs), hookq_mode=mode)
