/*
 * hook_attn.h -- C ABI of the hooked paged-attention library for NVIDIA B200 (sm_100a).
 *
 * One call computes, for a batch of sequences whose keys/values live in a paged KV cache,
 *
 *   (1) causal grouped-query attention   out[i,h,:] = softmax_t(scale * q[i,h,:].K[t,kv(h),:]) . V[t,kv(h),:]
 *   (2) the passive probe: for every *probed* query head and every configured key span
 *       [a_j, b_j) the exact post-softmax attention mass the query row places on the span,
 *           span_mass[i,h,j] = sum_{t in [a_j,b_j), t <= pos(i)} p[i,h,t]
 *       -- the quantity the paper's analyzer re-assembles from saved queries and keys and
 *       aggregates over token ranges (Section 2.2, the AttntrackerAnalyzer listing:
 *       "compute_attention_from_qk" followed by "attn2score" over "input_range"); the
 *       probed heads are the config's "important_heads" of one layer (Section 2, config
 *       listing), the probed rows its "hookq_mode" (last_token / all_tokens);
 *   (3) the active intervention: out[i,h,:] += alpha[h] * steer_vec[h,:] on the steered
 *       heads -- activation steering (Section 1, "Model Steering"; Section 3), applied per
 *       attention head after the softmax normalisation and before the single rounding of
 *       the output to bf16.
 *
 * Probing never changes `out` (Section 1 requires that passive programming leaves the model's
 * generation as it is): with and without probes the output bits are identical.  No attention matrix is materialised and no
 * query/key tensor leaves the GPU; span masses are carried as extra online-softmax
 * accumulators.
 *
 * Geometry.  Sequence s has L_s = seq_lens[s] keys in the cache (INCLUDING the keys of the
 * rows in this call: their K/V must already be written) and n_s query rows in this call.
 * Row i of sequence s sits at absolute position pos = L_s - n_s + i and sees keys 0..pos.
 * Logical key t of sequence s lives in physical page block_table[s][t / page_size], slot
 * t % page_size.  Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *
 * Pointers.  Unless a field says "host", every pointer is a DEVICE pointer owned by the
 * caller and borrowed until the work enqueued by the call has completed on the stream.  The
 * library writes only `out`, `span_mass`, `workspace` and `status`.  Calls enqueue work on the
 * caller's stream, never synchronise, and never allocate device memory.  Return codes are
 * synchronous and cover argument validation and launch errors; faults the device detects
 * (a block-table entry outside [0, num_blocks), a sequence longer than its table, more rows
 * than keys, a sequence longer than `max_seq_len`) are reported through the optional `status`
 * word, the affected rows of `out` and `span_mass` are written as zeros, and no out-of-range
 * address is dereferenced.  Every entry point that launches work returns
 * HOOK_ATTN_ERR_INVALID_ARG unless the handle's device is the current device.
 *
 * Supported: head_dim in {64, 128}; page_size = 16; num_q_heads % num_kv_heads == 0 with a
 * group size <= 8; num_q_heads <= 64; num_spans <= 8; strides multiples of 8 elements and
 * 16-byte aligned base pointers.  Anything else returns HOOK_ATTN_ERR_UNSUPPORTED.
 */
#ifndef HOOK_ATTN_H_
#define HOOK_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hook_attn_handle hook_attn_handle; /* per-device state: SM count, cache of the prefill
                                                     kernel's TMA descriptors (keyed by pointer, shape, strides) */

enum {
    HOOK_ATTN_OK = 0,
    HOOK_ATTN_ERR_INVALID_ARG = -1, /* null required pointer, negative size, inconsistent shapes */
    HOOK_ATTN_ERR_UNSUPPORTED = -2, /* shape outside the supported set listed above */
    HOOK_ATTN_ERR_WORKSPACE = -3,   /* workspace missing or smaller than hook_attn_workspace_bytes */
    HOOK_ATTN_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (launch, attribute) */
    HOOK_ATTN_ERR_TIMEOUT = -5,     /* device status: a bounded wait inside a kernel ran out */
    HOOK_ATTN_ERR_BOUNDS = -6       /* device status: block id / length outside its range */
};

/* Which query rows of a prefill call are probed: the config's "hookq_mode" (Section 2). */
enum {
    HOOK_PROBE_ROWS_ALL = 0,  /* "all_tokens": span_mass has one row per query row */
    HOOK_PROBE_ROWS_LAST = 1  /* "last_token": one row per sequence (its last query row) */
};

typedef struct {
    /* ---- shapes ---- */
    int32_t num_seqs;            /* sequences in the batch (>= 0) */
    int32_t total_q;             /* total query rows T = sum n_s (decode: == num_seqs) */
    int32_t num_q_heads;         /* Hq */
    int32_t num_kv_heads;        /* Hkv */
    int32_t head_dim;            /* D */
    int32_t page_size;           /* tokens per KV page */
    int32_t num_blocks;          /* physical pages in the cache (bounds for block_table) */
    int32_t max_blocks_per_seq;  /* row length of block_table */
    int32_t num_spans;           /* S spans per sequence (0 = no probe) */
    int32_t probe_rows;          /* HOOK_PROBE_ROWS_*; ignored by decode (always LAST) */
    float   scale;               /* softmax scale; <= 0 selects 1/sqrt(head_dim) */
    int32_t max_seq_len;         /* optional host-side bound on seq_lens (0 = unknown, then
                                    max_blocks_per_seq * page_size).  Block tables are often padded to
                                    the model's maximum length; with the bound, decode cuts its work and
                                    sizes its workspace for the lengths the batch really has.  A sequence
                                    longer than the bound is a device-detected fault (status, zeros). */

    /* ---- device tensors ---- */
    const void*    q;            /* bf16 [total_q][Hq][D], contiguous */
    const void*    k_cache;      /* bf16, element (block, slot, kv_head, d) at
                                    block*kv_block_stride + slot*kv_token_stride + kv_head*kv_head_stride + d */
    const void*    v_cache;      /* same layout and strides as k_cache */
    int64_t        kv_block_stride, kv_token_stride, kv_head_stride; /* in elements */
    const int32_t* block_table;  /* [num_seqs][max_blocks_per_seq]; entries past ceil(L_s/page_size)
                                    are never read */
    const int32_t* seq_lens;     /* [num_seqs] L_s */
    const int32_t* cu_q_lens;    /* [num_seqs+1] prefix sums of n_s; prefill only (decode: NULL) */
    const int32_t* spans;        /* [num_seqs][S][2] half-open absolute key ranges [a,b); clipped to the
                                    visible keys; a >= b is an empty span.  NULL = no probe */
    const float*   steer_vec;    /* fp32 [Hq][D]; NULL = no steering */
    void*          out;          /* bf16 [total_q][Hq][D] */
    float*         span_mass;    /* fp32 [rows][P][S]; rows = total_q (ALL) or num_seqs (LAST, decode);
                                    P = number of nonzero head_mask entries; the slot of a probed head is
                                    its rank among the probed heads in ascending head order.  In LAST mode
                                    a sequence without rows in the call gets zeros */
    void*          workspace;    /* scratch of at least hook_attn_workspace_bytes(); 256-byte aligned
                                    (checked: HOOK_ATTN_ERR_WORKSPACE otherwise) */
    size_t         workspace_bytes;
    int32_t*       status;       /* optional: one int32, set to a negative HOOK_ATTN_ERR_* code by the
                                    device on a detected fault; the caller zeroes it beforehand */

    /* ---- HOST arrays, read during the call and copied into the kernel parameters ---- */
    const uint8_t* head_mask;    /* host [Hq]; nonzero = probed head.  NULL = no probe */
    const float*   alpha;        /* host [Hq]; 0 = head not steered.  NULL = no steering */
} hook_attn_params;

/* Create / destroy the per-device handle.  `device` is a CUDA device ordinal.  Creation queries
 * device properties and configures the kernels; it fails with HOOK_ATTN_ERR_UNSUPPORTED on a
 * device that is not compute capability 10.x, HOOK_ATTN_ERR_CUDA if no device is usable. */
int hook_attn_create(hook_attn_handle** handle, int device);
int hook_attn_destroy(hook_attn_handle* handle);

/* Bytes of scratch the call described by `p` needs (only the shape fields and max_seq_len are read;
 * pass the same max_seq_len to the call).
 * is_decode = 1 sizes hook_attn_decode, 2 the decode half of hook_attn_mixed, 0 hook_attn_prefill.
 * Returns 0 when the call needs no scratch or when the shapes are invalid. */
size_t hook_attn_workspace_bytes(const hook_attn_params* p, int is_decode);

/* Prefill / chunked prefill: n_s >= 0 rows per sequence given by cu_q_lens, n_s <= L_s.
 * (Section 2.2 recompute + Section 2 steering, fused into the attention forward.) */
int hook_attn_prefill(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream);

/* Decode: exactly one query row per sequence (total_q == num_seqs, cu_q_lens ignored).  The keys of a
 * (sequence, KV head) unit are cut into pieces that are reduced independently and then merged.  The
 * cut is chosen from the host-known shape of the batch: with many units (num_seqs * num_kv_heads >=
 * 296) every sequence is cut into chunks of a fixed length (a power of two in 256..2048 keys, from
 * num_seqs, num_kv_heads and the length bound); with fewer, the pages of all units form one list
 * that is dealt out in equal shares to a fixed number of worker warps.  Either way the pieces of a
 * unit are merged in a fixed order, so results are bit-identical from run to run.  span_mass has one
 * row per sequence. */
int hook_attn_decode(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream);

/* One step of a serving loop that holds both a decode batch and prefill chunks (chunked prefill, the
 * usual shape of a served step): the work of hook_attn_decode(decode) and hook_attn_prefill(prefill), same
 * arguments, outputs, results and error behaviour, issued together.  (Section 2: the hooks act inside the
 * engine's forward pass, whatever mix of requests a step carries; Section 2.1: the worker runs them per
 * execute_model call.)  When both halves have head_dim 128, the prefill half has at least 128 rows and the
 * decode half at most 512 sequences, one launch carries both -- a part of the SMs streams the decode batch
 * at HBM speed while the rest runs the prefill tiles on the tensor cores -- followed by the merge of the
 * decode partials; otherwise the two calls are issued one after the other.  `decode->workspace` must hold
 * hook_attn_workspace_bytes(decode, 2) bytes.  Either half may be empty (num_seqs = 0).  The two halves must
 * not write overlapping outputs. */
int hook_attn_mixed(hook_attn_handle* handle, const hook_attn_params* prefill, const hook_attn_params* decode,
                    void* cuda_stream);

/* Decode for callers that can neither allocate device memory nor hand over scratch.
 * (The paper has no counterpart; this is a convenience of the library.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a serving loop whose
 * memory budget is already committed to the KV cache, a plug-in that only receives the hooked
 * layer's tensors, or a latency-critical path where an allocation (and the synchronisation it
 * implies) must never happen.  Such a caller cannot size and keep the `workspace` of
 * hook_attn_decode, so here the split-K partials go into a fixed array of
 * HOOK_ATTN_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds that much memory until the process exits.
 *
 * Same arguments, outputs and results as hook_attn_decode; `workspace` and `workspace_bytes` are
 * ignored.  The call allocates nothing and frees nothing.  A batch whose partials do not fit the
 * array (hook_attn_workspace_bytes(p, 1) > HOOK_ATTN_STATIC_SCRATCH_BYTES) is refused with
 * HOOK_ATTN_ERR_WORKSPACE and nothing is launched.  The handle's device must be the current
 * device, otherwise HOOK_ATTN_ERR_INVALID_ARG.
 *
 * The first call on each device looks up the device address of the array; make that first call
 * outside of any stream capture.  All calls on a device share the one array, which keeps whatever
 * the previous call left in it: the kernels never read an entry they have not written in the
 * same call, so nothing needs clearing -- but two calls whose work overlaps on the GPU (different
 * streams, or concurrent host threads) race on it.  Issue them on one stream, or order them. */
#define HOOK_ATTN_STATIC_SCRATCH_BYTES (16u << 20)
int hook_attn_decode_static_scratch(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream);

/* Analyzer reduction over span masses (Section 2.2: the analyzer turns the re-assembled attention of
 * the important heads and the configured token ranges into a score, attn_func "sum_normalize";
 * Section 3: focus score of the instruction, per-passage relevance scores).  The analyzer's body is
 * not printed in the paper, so the two reductions are this library's reading of its words:
 *   HOOK_SCORE_MEAN            scores[r][j] = mean over probed heads p of span_mass[r][p][j]
 *   HOOK_SCORE_SUM_NORMALIZE   scores[r][j] = mean over p of span_mass[r][p][j] / sum_j' span_mass[r][p][j']
 *                              (a head whose masses sum to zero contributes zero); with the two spans
 *                              (instruction, data) scores[r][0] is instruction / (instruction + data).
 * span_mass: device fp32 [rows][num_probed][num_spans] as written by prefill / decode; scores: device
 * fp32 [rows][num_spans].  Only this small result has to leave the GPU. */
enum { HOOK_SCORE_MEAN = 0, HOOK_SCORE_SUM_NORMALIZE = 1 };
int hook_attn_score(hook_attn_handle* handle, const float* span_mass, int32_t rows, int32_t num_probed,
                    int32_t num_spans, int32_t mode, float* scores, void* cuda_stream);

/* Residual-stream activation steering (Section 1 "Model Steering", Section 3: a steering vector is
 * injected into a layer of the deployed model): hidden[t][:] += alpha * steer_vec[:] for every token
 * row t, in place.  hidden: device bf16, num_tokens rows of hidden_size elements, row_stride elements
 * apart (multiples of 8, 16-byte aligned); steer_vec: device fp32 [hidden_size].  The add is done in
 * fp32 and rounded once to bf16.  alpha = 0 changes nothing. */
int hook_steer_residual(hook_attn_handle* handle, void* hidden, const float* steer_vec, float alpha,
                        int64_t num_tokens, int32_t hidden_size, int64_t row_stride, void* cuda_stream);

/* Raw q/k capture (Section 2.1: the worker's hook keeps, per hooked attention module, the queries of the
 * last or of all tokens and the keys of all tokens; Section 2.2: the analyzer recomputes attention from
 * them).  For analyzers that need the raw states rather than span masses.  Reads q, k_cache, block_table,
 * seq_lens, cu_q_lens (prefill), head_mask (host) and probe_rows of `p`; spans, steering, out and
 * workspace are ignored.  With P probed heads in ascending order:
 *   q_out  device bf16 [rows][P][D], rows = total_q (all_tokens) or num_seqs (last_token / decode; a
 *          sequence without rows in the call gets zeros);               may be NULL
 *   k_out  device bf16 [sum L_s][P][D]: key t of sequence s at row cu_k_lens[s] + t, taken from the KV
 *          head of the probed query head;                               may be NULL
 *   cu_k_lens  device int32 [num_seqs + 1], prefix sums of seq_lens (caller-computed).
 * Byte-exact copies; block ids are bounds-checked like in the attention calls. */
int hook_capture_qk(hook_attn_handle* handle, const hook_attn_params* p, int is_decode, void* q_out, void* k_out,
                    const int32_t* cu_k_lens, void* cuda_stream);

/* Self-test of the kernels' bounded waits (the paper has no counterpart; it backs the failure
 * behaviour stated above).  Launches one small kernel that waits on a barrier nothing ever signals.
 * After `limit_ns` (1 .. 1e9) the wait gives up, the kernel writes HOOK_ATTN_ERR_TIMEOUT into the
 * device word `status` (zeroed by the caller), stores the time it waited into the optional device
 * word `waited_ns`, and returns normally: no trap, no hang, the context stays usable. */
int hook_attn_selftest_wait_limit(hook_attn_handle* handle, int32_t* status, uint64_t limit_ns, uint64_t* waited_ns,
                                  void* cuda_stream);

/* Human-readable name of a return / status code. */
const char* hook_attn_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* HOOK_ATTN_H_ */
