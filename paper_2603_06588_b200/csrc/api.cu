// C ABI of the hooked paged-attention library: argument validation, workspace sizing, dispatch.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "common.cuh"

namespace hook_attn {
// decode.cu
cudaError_t configure_decode();
cudaError_t launch_decode(const KernelArgs& a, const HeadCfg& hc, int head_dim, int num_sms, cudaStream_t st);
size_t decode_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim, int max_keys);
// prefill_mma.cu
cudaError_t configure_prefill_mma();
cudaError_t launch_prefill_mma(const KernelArgs& a, const HeadCfg& hc, int head_dim, cudaStream_t st);
int prefill_mma_tiles_upper_bound(int total_q, int num_seqs);
// prefill_tc.cu
cudaError_t configure_prefill_tc();
bool prefill_tc_supported(const KernelArgs& a, int head_dim);
cudaError_t launch_prefill_tc(const KernelArgs& a, const HeadCfg& hc, void* tmap_cache, int num_sms, cudaStream_t st);
void* tmap_cache_create();
void tmap_cache_destroy(void* cache);
cudaError_t launch_wait_selftest(int32_t* status, uint64_t limit_ns, uint64_t* waited_ns, cudaStream_t st);
// mixed.cu
cudaError_t configure_mixed();
bool mixed_supported(const KernelArgs& apf, int head_dim_pf, const KernelArgs& adec, int head_dim_dec);
size_t mixed_decode_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim);
cudaError_t launch_mixed(const KernelArgs& apf, const HeadCfg& hpf, const KernelArgs& adec, const HeadCfg& hdec, void* tmap_cache,
                         int num_sms, int forced_dec_ctas, cudaStream_t st);
// extras.cu
cudaError_t launch_score(const float* mass, float* scores, int rows, int P, int S, int mode, cudaStream_t st);
cudaError_t launch_steer_residual(__nv_bfloat16* hidden, const float* vec, float alpha, int64_t tokens, int hidden_size,
                                  int64_t row_stride, int num_sms, cudaStream_t st);
cudaError_t launch_capture(const KernelArgs& a, const HeadCfg& hc, int head_dim, bool decode, __nv_bfloat16* q_out,
                           __nv_bfloat16* k_out, const int32_t* cu_k, cudaStream_t st);
}  // namespace hook_attn

using namespace hook_attn;

struct hook_attn_handle {
    int device;
    int num_sms;
    int cc_major, cc_minor;
    bool prefer_tc;   // head_dim-128 prefill goes to the tcgen05 kernel (HOOK_ATTN_PREFILL_KERNEL=mma turns it off)
    void* tmap_cache; // TMA descriptors of the prefill kernel, keyed by base pointer, shape and strides
    int mixed_dec_ctas; // HOOK_ATTN_MIXED_DECODE_CTAS: CTAs in the decode role of the one-launch mixed step (0 = from the shapes)
};

namespace {

int validate_common(const hook_attn_params* p, bool decode)
{
    if (!p) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->num_seqs < 0 || p->total_q < 0 || p->num_q_heads <= 0 || p->num_kv_heads <= 0 || p->head_dim <= 0 ||
        p->page_size <= 0 || p->num_blocks < 0 || p->max_blocks_per_seq < 0 || p->num_spans < 0 || p->max_seq_len < 0)
        return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->num_q_heads % p->num_kv_heads != 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if (decode && p->total_q != p->num_seqs) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->probe_rows != HOOK_PROBE_ROWS_ALL && p->probe_rows != HOOK_PROBE_ROWS_LAST) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->head_dim != 64 && p->head_dim != 128) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (p->page_size != kPage) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (p->num_q_heads > kMaxHeads) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (p->num_q_heads / p->num_kv_heads > kMaxGroup) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (p->num_spans > kMaxSpans) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (p->num_seqs > 65535) return HOOK_ATTN_ERR_UNSUPPORTED;
    return HOOK_ATTN_OK;
}

bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

// Longest sequence the call may hold: the caller's hint when given, never more than the table can address.
int max_keys_of(const hook_attn_params* p)
{
    long long cap = (long long)p->max_blocks_per_seq * p->page_size;
    if (cap > 0x7fffffffLL) cap = 0x7fffffffLL;
    if (p->max_seq_len > 0 && p->max_seq_len < cap) cap = p->max_seq_len;
    return (int)cap;
}

// Calls that launch need the handle's device to be the current one: the launch goes to the current
// device, and the kernels' shared-memory opt-in was made on the handle's.
int check_handle(const hook_attn_handle* handle)
{
    if (!handle) return HOOK_ATTN_ERR_INVALID_ARG;
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess) { (void)cudaGetLastError(); return HOOK_ATTN_ERR_CUDA; }
    return current == handle->device ? HOOK_ATTN_OK : HOOK_ATTN_ERR_INVALID_ARG;
}

// Fills the kernel arguments; returns a HOOK_ATTN_* code.
int prepare(const hook_attn_params* p, bool decode, KernelArgs& a, HeadCfg& hc)
{
    int rc = validate_common(p, decode);
    if (rc != HOOK_ATTN_OK) return rc;
    if (p->num_seqs == 0 || p->total_q == 0) return HOOK_ATTN_OK;   // nothing to do (caller checks total_q)
    if (!p->q || !p->k_cache || !p->v_cache || !p->block_table || !p->seq_lens || !p->out) return HOOK_ATTN_ERR_INVALID_ARG;
    if (!decode && !p->cu_q_lens) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->kv_block_stride <= 0 || p->kv_token_stride <= 0 || p->kv_head_stride <= 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if ((p->kv_block_stride | p->kv_token_stride | p->kv_head_stride) & 7) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (!aligned16(p->q) || !aligned16(p->k_cache) || !aligned16(p->v_cache) || !aligned16(p->out)) return HOOK_ATTN_ERR_UNSUPPORTED;

    memset(&hc, 0, sizeof hc);
    int probed = 0;
    bool any_steer = false;
    for (int h = 0; h < kMaxHeads; ++h) hc.slot[h] = -1;
    for (int h = 0; h < p->num_q_heads; ++h) {
        if (p->head_mask && p->head_mask[h]) hc.slot[h] = (int8_t)probed++;
        if (p->alpha && p->alpha[h] != 0.0f) {
            if (!isfinite(p->alpha[h])) return HOOK_ATTN_ERR_INVALID_ARG;
            hc.alpha[h] = p->alpha[h];
            any_steer = true;
        }
    }
    const bool any_probe = probed > 0 && p->num_spans > 0;
    if (any_probe && (!p->spans || !p->span_mass)) return HOOK_ATTN_ERR_INVALID_ARG;
    if (any_steer && !p->steer_vec) return HOOK_ATTN_ERR_INVALID_ARG;
    if (!any_probe) for (int h = 0; h < kMaxHeads; ++h) hc.slot[h] = -1;

    memset(&a, 0, sizeof a);
    a.q = static_cast<const __nv_bfloat16*>(p->q);
    a.k = static_cast<const __nv_bfloat16*>(p->k_cache);
    a.v = static_cast<const __nv_bfloat16*>(p->v_cache);
    a.bs = p->kv_block_stride; a.ts = p->kv_token_stride; a.hs = p->kv_head_stride;
    a.block_table = p->block_table; a.seq_lens = p->seq_lens; a.cu_q_lens = p->cu_q_lens;
    a.spans = p->spans; a.steer = p->steer_vec;
    a.out = static_cast<__nv_bfloat16*>(p->out);
    a.mass = p->span_mass;
    a.ws = static_cast<float*>(p->workspace);
    a.status = p->status;
    a.num_seqs = p->num_seqs; a.total_q = p->total_q; a.Hq = p->num_q_heads; a.Hkv = p->num_kv_heads;
    a.G = p->num_q_heads / p->num_kv_heads;
    a.num_blocks = p->num_blocks; a.max_blocks = p->max_blocks_per_seq;
    a.max_keys = max_keys_of(p);
    a.S = any_probe ? p->num_spans : 0; a.P = probed; a.probe_rows = p->probe_rows;
    const float scale = (p->scale > 0.f) ? p->scale : 1.0f / sqrtf((float)p->head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;
    a.any_probe = any_probe; a.any_steer = any_steer;
    return HOOK_ATTN_OK;
}

}  // namespace

extern "C" {

int hook_attn_create(hook_attn_handle** handle, int device)
{
    if (!handle) return HOOK_ATTN_ERR_INVALID_ARG;
    *handle = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return HOOK_ATTN_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return HOOK_ATTN_ERR_CUDA;
    if (prop.major != 10) return HOOK_ATTN_ERR_UNSUPPORTED;
    int prev = 0;
    cudaGetDevice(&prev);
    if (cudaSetDevice(device) != cudaSuccess) return HOOK_ATTN_ERR_CUDA;
    cudaError_t e = configure_decode();
    if (e == cudaSuccess) e = configure_prefill_mma();
    if (e == cudaSuccess) e = configure_prefill_tc();
    if (e == cudaSuccess) e = configure_mixed();
    cudaSetDevice(prev);
    if (e != cudaSuccess) return HOOK_ATTN_ERR_CUDA;
    hook_attn_handle* h = new hook_attn_handle;
    h->device = device;
    h->num_sms = prop.multiProcessorCount;
    h->cc_major = prop.major;
    h->cc_minor = prop.minor;
    const char* pk = getenv("HOOK_ATTN_PREFILL_KERNEL");
    h->prefer_tc = !(pk && strcmp(pk, "mma") == 0);
    h->tmap_cache = tmap_cache_create();
    const char* md = getenv("HOOK_ATTN_MIXED_DECODE_CTAS");
    h->mixed_dec_ctas = md ? atoi(md) : 0;
    *handle = h;
    return HOOK_ATTN_OK;
}

int hook_attn_destroy(hook_attn_handle* handle)
{
    if (handle) tmap_cache_destroy(handle->tmap_cache);
    delete handle;
    return HOOK_ATTN_OK;
}

size_t hook_attn_workspace_bytes(const hook_attn_params* p, int is_decode)
{
    if (validate_common(p, is_decode != 0) != HOOK_ATTN_OK) return 0;
    if (!is_decode) return 0;
    const int G = p->num_q_heads / p->num_kv_heads;
    const size_t alone = decode_workspace_bytes(p->num_seqs, p->num_kv_heads, G, p->head_dim, max_keys_of(p));
    if (is_decode != 2) return alone;
    // the decode half of hook_attn_mixed: the one-launch path cuts by page shares whatever the unit count,
    // the fallback is the stand-alone call
    const size_t shared = mixed_decode_workspace_bytes(p->num_seqs, p->num_kv_heads, G, p->head_dim);
    return alone > shared ? alone : shared;
}

int hook_attn_prefill(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream)
{
    KernelArgs a;
    HeadCfg hc;
    int rc = prepare(p, false, a, hc);     // argument errors are reported before anything else
    if (rc != HOOK_ATTN_OK) return rc;
    if ((rc = check_handle(handle)) != HOOK_ATTN_OK) return rc;
    if (p->num_seqs == 0 || p->total_q == 0) return HOOK_ATTN_OK;
    cudaError_t e;
    if (handle->prefer_tc && prefill_tc_supported(a, p->head_dim)) {
        e = launch_prefill_tc(a, hc, handle->tmap_cache, handle->num_sms, static_cast<cudaStream_t>(cuda_stream));
    } else {
        a.total_tiles = prefill_mma_tiles_upper_bound(p->total_q, p->num_seqs);
        e = launch_prefill_mma(a, hc, p->head_dim, static_cast<cudaStream_t>(cuda_stream));
    }
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_attn_decode(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream)
{
    KernelArgs a;
    HeadCfg hc;
    int rc = prepare(p, true, a, hc);
    if (rc != HOOK_ATTN_OK) return rc;
    if (p->num_seqs > 0 && p->max_blocks_per_seq == 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->num_seqs == 0) return handle ? HOOK_ATTN_OK : HOOK_ATTN_ERR_INVALID_ARG;
    const size_t need = decode_workspace_bytes(p->num_seqs, p->num_kv_heads, a.G, p->head_dim, a.max_keys);
    if (!p->workspace || p->workspace_bytes < need) return HOOK_ATTN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(p->workspace) & 255u) return HOOK_ATTN_ERR_WORKSPACE;
    if ((rc = check_handle(handle)) != HOOK_ATTN_OK) return rc;
    cudaError_t e = launch_decode(a, hc, p->head_dim, handle->num_sms, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_attn_mixed(hook_attn_handle* handle, const hook_attn_params* prefill, const hook_attn_params* decode, void* cuda_stream)
{
    KernelArgs apf, adec;
    HeadCfg hpf, hdec;
    int rc = prepare(prefill, false, apf, hpf);
    if (rc != HOOK_ATTN_OK) return rc;
    if ((rc = prepare(decode, true, adec, hdec)) != HOOK_ATTN_OK) return rc;
    const bool has_pf = prefill->num_seqs > 0 && prefill->total_q > 0, has_dec = decode->num_seqs > 0;
    if (has_dec && decode->max_blocks_per_seq == 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if (has_dec) {
        const size_t need = hook_attn_workspace_bytes(decode, 2);
        if (!decode->workspace || decode->workspace_bytes < need) return HOOK_ATTN_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(decode->workspace) & 255u) return HOOK_ATTN_ERR_WORKSPACE;
    }
    if ((rc = check_handle(handle)) != HOOK_ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (has_pf && has_dec && handle->prefer_tc && mixed_supported(apf, prefill->head_dim, adec, decode->head_dim)) {
        cudaError_t e = launch_mixed(apf, hpf, adec, hdec, handle->tmap_cache, handle->num_sms, handle->mixed_dec_ctas, st);
        return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
    }
    // shapes the one-launch kernel does not take (or an empty half): the two calls, one after the other
    if (has_dec && (rc = hook_attn_decode(handle, decode, cuda_stream)) != HOOK_ATTN_OK) return rc;
    if (has_pf && (rc = hook_attn_prefill(handle, prefill, cuda_stream)) != HOOK_ATTN_OK) return rc;
    return HOOK_ATTN_OK;
}

// ---- decode without any caller-provided or allocated scratch --------------------------------
//
// Some callers cannot allocate device memory at the point where they run attention: code inside
// a memory-pool-managed serving loop that has handed its whole budget to the KV cache, plug-ins
// that are only given the tensors of the layer they hook, and callers that must not trigger an
// allocation (and the implicit synchronisation it brings) on their hot path.  For them the
// split-K partials live in this fixed array, which every GPU that loads the library holds until
// the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HOOK_ATTN_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal
bool g_static_scratch_ready[kMaxDevices];
std::mutex g_static_scratch_mutex;

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address the kernels can use has to be asked for, once per device, with that device current.
int static_scratch_address(int device, float** out)
{
    if (device < 0 || device >= kMaxDevices) return HOOK_ATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ready[device]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return HOOK_ATTN_ERR_CUDA;
        }
        g_static_scratch_ptr[device] = static_cast<float*>(ptr);
        g_static_scratch_ready[device] = true;
    }
    *out = g_static_scratch_ptr[device];
    return HOOK_ATTN_OK;
}
}  // namespace

int hook_attn_decode_static_scratch(hook_attn_handle* handle, const hook_attn_params* p, void* cuda_stream)
{
    KernelArgs a;
    HeadCfg hc;
    int rc = prepare(p, true, a, hc);
    if (rc != HOOK_ATTN_OK) return rc;
    if (p->num_seqs > 0 && p->max_blocks_per_seq == 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if (p->num_seqs == 0) return handle ? HOOK_ATTN_OK : HOOK_ATTN_ERR_INVALID_ARG;
    const size_t need = decode_workspace_bytes(p->num_seqs, p->num_kv_heads, a.G, p->head_dim, a.max_keys);
    if (need > HOOK_ATTN_STATIC_SCRATCH_BYTES) return HOOK_ATTN_ERR_WORKSPACE;   // batch too large for the fixed array
    if ((rc = check_handle(handle)) != HOOK_ATTN_OK) return rc;                  // the handle's device must be current
    float* scratch = nullptr;
    rc = static_scratch_address(handle->device, &scratch);
    if (rc != HOOK_ATTN_OK) return rc;
    a.ws = scratch;   // every partial the merge reads is written by the streaming kernel of the same call:
                      // nothing in the array has to start at zero, stale contents are never read
    cudaError_t e = launch_decode(a, hc, p->head_dim, handle->num_sms, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_attn_score(hook_attn_handle* handle, const float* span_mass, int32_t rows, int32_t num_probed, int32_t num_spans,
                    int32_t mode, float* scores, void* cuda_stream)
{
    if (rows < 0 || num_probed <= 0 || num_spans <= 0) return HOOK_ATTN_ERR_INVALID_ARG;
    if (mode != HOOK_SCORE_MEAN && mode != HOOK_SCORE_SUM_NORMALIZE) return HOOK_ATTN_ERR_INVALID_ARG;
    if (num_spans > kMaxSpans) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (rows > 0 && (!span_mass || !scores)) return HOOK_ATTN_ERR_INVALID_ARG;
    int rc = check_handle(handle);
    if (rc != HOOK_ATTN_OK) return rc;
    if (rows == 0) return HOOK_ATTN_OK;
    cudaError_t e = launch_score(span_mass, scores, rows, num_probed, num_spans, mode, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_steer_residual(hook_attn_handle* handle, void* hidden, const float* steer_vec, float alpha, int64_t num_tokens,
                        int32_t hidden_size, int64_t row_stride, void* cuda_stream)
{
    if (num_tokens < 0 || hidden_size <= 0 || row_stride < hidden_size || !isfinite(alpha)) return HOOK_ATTN_ERR_INVALID_ARG;
    if ((hidden_size & 7) || (row_stride & 7)) return HOOK_ATTN_ERR_UNSUPPORTED;
    if (num_tokens > 0 && (!hidden || !steer_vec)) return HOOK_ATTN_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(steer_vec)) return HOOK_ATTN_ERR_UNSUPPORTED;
    int rc = check_handle(handle);
    if (rc != HOOK_ATTN_OK) return rc;
    if (num_tokens == 0 || alpha == 0.0f) return HOOK_ATTN_OK;   // alpha = 0 leaves every bit in place
    cudaError_t e = launch_steer_residual(static_cast<__nv_bfloat16*>(hidden), steer_vec, alpha, num_tokens, hidden_size,
                                          row_stride, handle->num_sms, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_capture_qk(hook_attn_handle* handle, const hook_attn_params* p, int is_decode, void* q_out, void* k_out,
                    const int32_t* cu_k_lens, void* cuda_stream)
{
    KernelArgs a;
    HeadCfg hc;
    hook_attn_params q = {};
    if (p) {
        q = *p;
        q.out = const_cast<void*>(p->q);   // the capture writes no attention output; keep the shared checks satisfied
        q.num_spans = 0;                   // spans play no role here
    }
    int rc = prepare(p ? &q : nullptr, is_decode != 0, a, hc);
    if (rc != HOOK_ATTN_OK) return rc;
    if ((rc = check_handle(handle)) != HOOK_ATTN_OK) return rc;
    if (p->num_seqs == 0 || p->total_q == 0) return HOOK_ATTN_OK;
    int probed = 0;
    for (int h = 0; h < p->num_q_heads; ++h)
        if (p->head_mask && p->head_mask[h]) hc.slot[h] = (int8_t)probed++; else hc.slot[h] = -1;
    if (probed == 0) return HOOK_ATTN_OK;   // nothing is hooked
    a.P = probed;
    if (k_out && !cu_k_lens) return HOOK_ATTN_ERR_INVALID_ARG;
    if ((q_out && !aligned16(q_out)) || (k_out && !aligned16(k_out))) return HOOK_ATTN_ERR_UNSUPPORTED;
    cudaError_t e = launch_capture(a, hc, p->head_dim, is_decode != 0, static_cast<__nv_bfloat16*>(q_out),
                                   static_cast<__nv_bfloat16*>(k_out), cu_k_lens, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

int hook_attn_selftest_wait_limit(hook_attn_handle* handle, int32_t* status, uint64_t limit_ns, uint64_t* waited_ns,
                                  void* cuda_stream)
{
    if (!status || limit_ns == 0 || limit_ns > 1000000000ull) return HOOK_ATTN_ERR_INVALID_ARG;
    int rc = check_handle(handle);
    if (rc != HOOK_ATTN_OK) return rc;
    cudaError_t e = launch_wait_selftest(status, limit_ns, waited_ns, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HOOK_ATTN_OK : HOOK_ATTN_ERR_CUDA;
}

const char* hook_attn_strerror(int code)
{
    switch (code) {
        case HOOK_ATTN_OK: return "ok";
        case HOOK_ATTN_ERR_INVALID_ARG: return "invalid argument";
        case HOOK_ATTN_ERR_UNSUPPORTED: return "unsupported shape, layout or device";
        case HOOK_ATTN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case HOOK_ATTN_ERR_CUDA: return "CUDA call failed";
        case HOOK_ATTN_ERR_TIMEOUT: return "bounded wait ran out on the device";
        case HOOK_ATTN_ERR_BOUNDS: return "block id or sequence length out of range";
        default: return "unknown code";
    }
}

}  // extern "C"
