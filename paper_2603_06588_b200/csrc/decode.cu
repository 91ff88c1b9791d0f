// Split-K decode of the hooked paged attention: one query row per sequence.
//
// The first kernel reduces pieces of each (sequence, KV head) unit to partials (m, l, o[D], s[S]),
// the second merges the partials of a unit.  Two ways of cutting the pieces, chosen per call from
// the batch shape:
//
// * decode_splitk (many units): one CTA per (key chunk, KV head, sequence) with a fixed chunk length;
//   its four warps take the chunk's pages in turn and are merged in shared memory.  With hundreds of
//   units the hardware's CTA dispatch keeps every SM busy and evens out their speeds.
// * decode_stream (few units, long sequences): fixed chunks would mean either too few CTAs or many
//   short ones and a large merge.  Here the 16-key pages of all units form one flat list
//   (sequence-major, then KV head, then page) and every warp of a grid of three CTAs per SM takes an
//   equal, contiguous share of it, found from the sequence lengths on the device.  A warp walks its
//   share unit by unit and writes one partial per unit it touches to slot `unit + warp` (both grow
//   along the walk, so the slot is unique).  When the shares of the four warps of a CTA all lie inside one
//   unit (the common case with long sequences) the CTA folds them in shared memory first and writes a
//   single partial to the slot of its first warp, which quarters the work of the merge.
//
// Inside a unit the G <= 8 query heads that share the KV head are processed together with
// warp-level tensor-core tiles in the transposed orientation: a 16-key page is the M dimension, the
// query heads are the N = 8 dimension (S^T = K Q^T, O^T = V^T P^T), so no padding work is spent on
// the single query row.  A warp streams pages through a private multi-stage cp.async pipeline
// (16-byte copies, zero-filled past the end of the sequence), keeps an online softmax per head, and
// carries the span masses of the probe as extra accumulators in the same frame as the running sum.
//
// decode_merge: one CTA per (query head, sequence) folds the unit's partials in a fixed order
// (run-to-run bit-identical), normalises, applies the steering add and stores.
#include "decode_device.cuh"

namespace hook_attn {

template <int HD, int NS>
__global__ void __launch_bounds__(kDecWarps * 32) decode_stream_kernel(const KernelArgs a, const HeadCfg hc)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ DecStreamShared<kDecWarps> sh;
    decode_stream_cta<HD, NS, kDecWarps>(a, hc, smem, blockIdx.x, sh);
}

template <int HD, int NS>
__global__ void __launch_bounds__(kDecWarps * 32) decode_splitk_kernel(const KernelArgs a, const HeadCfg hc)
{
    constexpr int TILEB = kPage * HD * 2;   // bytes per 16-key tile
    constexpr int KS = HD / 16;

    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ int sh_span[kDecWarps][2 * kMaxSpans];
    __shared__ DecFold sh_fold;

    const int s = blockIdx.z, kvh = blockIdx.y, c = blockIdx.x;
    const int warp = threadIdx.x >> 5;
    const int G = a.G;

    // launched with programmatic serialization: the merge of the call before this one on the stream may still be
    // running (it reads the workspace this grid writes, and may be writing the q this grid reads)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int L = a.seq_lens[s];
    if (L <= 0 || L > a.max_keys) return;   // reported and zero-filled by the merge kernel
    const int start = c * a.chunk;
    if (start >= L) return;
    const int end = min(L, start + a.chunk);
    const int ntiles = (end - start + kPage - 1) / kPage;

    // the four warps take contiguous quarters of the chunk's pages
    const int per = (ntiles + kDecWarps - 1) / kDecWarps;
    const int first = min(warp * per, ntiles);
    const int seg = min(per, ntiles - first);
    const uint32_t wbase = smem_u32(smem) + warp * (kDecStages * 2 * TILEB);

    float m0, m1, l0, l1, o[KS][4], sm[NS > 0 ? NS : 1][2];
    decode_segment<HD, NS>(a, hc, s, kvh, start / kPage + first, seg, L, wbase, sh_span[warp], m0, m1, l0, l1, o, sm);

    const size_t pstride = decode_partial_stride(HD);
    float* part = a.ws + (((size_t)s * a.Hkv + kvh) * a.max_chunks + c) * G * pstride;
    decode_fold_cta<HD, NS>(part, G, reinterpret_cast<float*>(smem), sh_fold, 1, m0, m1, l0, l1, o, sm);
}

constexpr int kMergeMaxWarps = 16;   // warps of the merge kernel when a unit may have many partials (4 otherwise)

// One CTA per (query head, sequence).  It finds the unit's partials -- the chunks of the sequence, or
// the worker warps and whole CTAs of the streaming kernel that covered the unit (the same arithmetic as
// there, from the page-count prefix that kernel left) -- then warp w folds the partials w, w + nwarps, ... with an
// online rescale (all loads of a partial are independent of the previous one's arithmetic, so several
// are in flight); the warps are then combined in warp order by the first 128 threads.  The order of
// every floating-point sum is fixed by (partial, warp) indices only: run-to-run bit-identical.
template <int HD, bool STREAM>
__global__ void __launch_bounds__(kMergeMaxWarps * 32) decode_merge_kernel(const KernelArgs a, const HeadCfg hc)
{
    constexpr int EPL = HD / 32;                       // output elements per lane
    __shared__ float sh_acc[kMergeMaxWarps][HD];
    __shared__ float sh_small[kMergeMaxWarps][2 + kMaxSpans];   // M, l, s[0..7]

    const int h = blockIdx.x, s = blockIdx.y;
    const int G = a.G, kvh = h / G, gi = h % G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    __nv_bfloat16* orow = a.out + ((int64_t)s * a.Hq + h) * HD;
    const int slot = hc.slot[h];
    float* mrow = (slot >= 0 && a.S > 0) ? a.mass + ((int64_t)s * a.P + slot) * a.S : nullptr;

    // the first-stage kernel of the next call on the stream may be scheduled from here on: it waits for this grid
    // before it touches the workspace or q
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // what does not come from the first-stage kernel is fetched while that kernel still runs
    const int L = a.seq_lens[s];
    const float al = hc.alpha[h];
    const float steer_d = (al != 0.f && (int)threadIdx.x < HD) ? al * a.steer[(int64_t)h * HD + threadIdx.x] : 0.f;
    // the partials are written by the kernel launched just before on the same stream
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int np = decode_pages(L, a.max_keys);
    if (np == 0) {
        if (threadIdx.x == 0) report(a.status, L <= 0 ? HOOK_ATTN_ERR_INVALID_ARG : HOOK_ATTN_ERR_BOUNDS);
        if ((int)threadIdx.x < HD) orow[threadIdx.x] = __float2bfloat16(0.f);
        if (mrow && (int)threadIdx.x < a.S) mrow[threadIdx.x] = 0.f;
        return;
    }
    const size_t pstride = decode_partial_stride(HD);
    const size_t cstride = (size_t)G * pstride;
    // Streaming kernel: in the order of its pages the unit's partials are the warps of a first CTA that the
    // unit shares with its neighbour (one partial each, slot = warp), then whole CTAs (one folded partial
    // each, in the slot of their first warp), then the warps of a last shared CTA.
    int nchunks, n_head = 0, n_mid = 0, n_tail = 0, head_w = 0, mid_c = 0, tail_w = 0;
    const float* part;
    if (STREAM) {
        const int* prefix = reinterpret_cast<const int*>(a.ws);
        const long long flat_total = (long long)prefix[a.num_seqs] * a.Hkv;
        const long long share = decode_share(flat_total, a.workers);
        const long long f0 = (long long)prefix[s] * a.Hkv + (long long)kvh * np, f1 = f0 + np;   // the unit's pages in the flat list
        const int w_first = (int)(f0 / share), w_last = (int)((f1 - 1) / share);
        const int c_first = w_first / kDecWarps, c_last = w_last / kDecWarps;
        auto whole = [&](int c) {   // the CTA's pages lie inside the unit: it wrote one folded partial
            const long long b = (long long)c * kDecWarps * share, e = min(b + kDecWarps * share, flat_total);
            return b >= f0 && e <= f1;
        };
        head_w = w_first;
        if (c_first == c_last) {
            if (whole(c_first)) { n_mid = 1; mid_c = c_first; }
            else n_head = w_last - w_first + 1;
        } else {
            const bool fw = whole(c_first), lw = whole(c_last);
            n_head = fw ? 0 : (c_first + 1) * kDecWarps - w_first;
            mid_c = fw ? c_first : c_first + 1;
            n_mid = (lw ? c_last : c_last - 1) - mid_c + 1;
            tail_w = c_last * kDecWarps;
            n_tail = lw ? 0 : w_last - tail_w + 1;
        }
        nchunks = n_head + n_mid + n_tail;
        part = reinterpret_cast<const float*>(reinterpret_cast<const char*>(a.ws) + decode_prefix_bytes(a.num_seqs)) +
               (((size_t)s * a.Hkv + kvh) * G + gi) * pstride;
    } else {
        nchunks = (L + a.chunk - 1) / a.chunk;
        part = a.ws + ((((size_t)s * a.Hkv + kvh) * a.max_chunks) * G + gi) * pstride;
    }
    // slot of the unit's i-th partial, relative to `part`
    auto slot_of = [&](int i) {
        if (!STREAM) return i;
        if (i < n_head) return head_w + i;
        if (i < n_head + n_mid) return (mid_c + (i - n_head)) * kDecWarps;
        return tail_w + (i - n_head - n_mid);
    };
    const bool want_mass = mrow != nullptr;

    float M = -INFINITY, lsum = 0.f, sacc = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
#pragma unroll 4
    for (int c = warp; c < nchunks; c += nwarps) {
        const float* pc = part + (size_t)slot_of(c) * cstride;
        const float mc = pc[HD], lc = pc[HD + 1];
        float oc[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) oc[e] = pc[lane + 32 * e];
        const float sc = (want_mass && lane < a.S) ? pc[HD + 2 + lane] : 0.f;
        const float Mn = fmaxf(M, mc);
        const float fo = fast_exp2(M - Mn), fc = fast_exp2(mc - Mn);   // M = -inf on the first chunk: fo = 0
        M = Mn;
        lsum = lsum * fo + lc * fc;
        sacc = sacc * fo + sc * fc;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = acc[e] * fo + oc[e] * fc;
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sh_acc[warp][lane + 32 * e] = acc[e];
    if (lane == 0) { sh_small[warp][0] = M; sh_small[warp][1] = lsum; }
    if (lane < kMaxSpans) sh_small[warp][2 + lane] = sacc;
    __syncthreads();

    const int d = threadIdx.x;
    if (d >= 128) return;
    const int used = min(nwarps, nchunks);             // warps that folded at least one chunk
    float Mg = sh_small[0][0];
    for (int w = 1; w < used; ++w) Mg = fmaxf(Mg, sh_small[w][0]);
    float ltot = 0.f, val = 0.f, mm = 0.f;
    for (int w = 0; w < used; ++w) {
        const float f = fast_exp2(sh_small[w][0] - Mg);
        ltot += f * sh_small[w][1];
        if (d < HD) val += f * sh_acc[w][d];
        if (d < kMaxSpans) mm += f * sh_small[w][2 + d];
    }
    const float inv = 1.f / ltot;
    if (d < HD) {
        val = val * inv + steer_d;
        orow[d] = __float2bfloat16(val);
    }
    if (mrow && d < a.S) mrow[d] = mm * inv;
}

// ------------------------------------------------------------------------------------------
// How a call is cut into pieces, from host-known bounds only (the lengths live on the device).
struct DecodePlan {
    bool stream;      // streaming kernel (few units) or fixed chunks
    int chunk;        // fixed chunks: keys per chunk, the largest power of two in 256..2048 that still
    int max_chunks;   //   leaves at least eight CTAs per SM in the grid; chunks per sequence
};

// The rule is evaluated for the SM count of a B200 whatever the device, so that the workspace size a caller
// asks for without a handle always matches the launch; only the streaming grid follows the device.
static DecodePlan decode_plan(int num_seqs, int Hkv, int max_keys)
{
    DecodePlan p = {};
    p.stream = (long)num_seqs * Hkv < kDecStreamUnits;
    p.chunk = 2048;
    while (p.chunk > 256) {
        const long ctas = (long)num_seqs * Hkv * (((long)max_keys + p.chunk - 1) / p.chunk);
        if (ctas >= 8L * kDecMaxSMs) break;
        p.chunk >>= 1;
    }
    p.max_chunks = (int)(((long)max_keys + p.chunk - 1) / p.chunk);
    if (p.max_chunks < 1) p.max_chunks = 1;
    return p;
}

// The merge is launched with programmatic stream serialization: its launch overlaps the drain of the
// first kernel, and it waits (griddepcontrol.wait) until that kernel's writes are visible.  `parts` is an
// estimate of the partials per unit and sizes the block.
template <int HD>
static cudaError_t launch_merge(const KernelArgs& a, const HeadCfg& hc, bool stream, long parts, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.Hq, a.num_seqs);
    cfg.blockDim = dim3((parts > 8 ? kMergeMaxWarps : 4) * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return stream ? cudaLaunchKernelEx(&cfg, decode_merge_kernel<HD, true>, a, hc)
                  : cudaLaunchKernelEx(&cfg, decode_merge_kernel<HD, false>, a, hc);
}

// Partials per unit when `ctas` streaming CTAs of `warps` warps share the pages of the call (half-full
// sequences assumed): whole groups of four warps inside a long unit, plus the warps of its two shared groups.
static long stream_parts_estimate(const KernelArgs& a, int ctas, int warps)
{
    const long max_pages = ((long)a.max_keys + kPage - 1) / kPage;
    const long groups = (long)ctas * warps / kDecWarps;
    const long est_group = ((long)a.num_seqs * a.Hkv * max_pages / 2 + groups - 1) / (groups > 0 ? groups : 1);
    return max_pages / (est_group > 0 ? est_group : 1) + 2 * kDecWarps;
}

template <int HD, int NS>
static cudaError_t launch_decode_t(KernelArgs a, const HeadCfg& hc, int num_sms, cudaStream_t st)
{
    const DecodePlan plan = decode_plan(a.num_seqs, a.Hkv, a.max_keys);
    a.chunk = plan.chunk;
    a.max_chunks = plan.max_chunks;
    long parts;   // partials per unit, to size the merge block
    // Programmatic serialization for the first kernel of the fixed-chunk cut as well: back-to-back decode calls on a
    // stream overlap its launch with the merge of the call before (which releases its successor at once): decode
    // batch 104.8 -> 102.3 us, mixed-batch decode 389.6 -> 384.2 us.  The one-wave streaming grid is launched in
    // stream order: with the attribute its step got slower (94.8 -> 100.2 us with hooks, 92.7 -> 94.0 without).
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kDecWarps * 32);
    cfg.dynamicSmemBytes = decode_smem_bytes<HD>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = plan.stream ? 0 : 1;
    cudaError_t e;
    if (plan.stream) {
        const int ctas = kDecCtasPerSM * (num_sms < kDecMaxSMs ? (num_sms > 0 ? num_sms : 1) : kDecMaxSMs);
        a.workers = ctas * kDecWarps;
        cfg.gridDim = dim3(ctas);
        e = cudaLaunchKernelEx(&cfg, decode_stream_kernel<HD, NS>, a, hc);
        parts = stream_parts_estimate(a, ctas, kDecWarps);
    } else {
        cfg.gridDim = dim3(plan.max_chunks, a.Hkv, a.num_seqs);
        e = cudaLaunchKernelEx(&cfg, decode_splitk_kernel<HD, NS>, a, hc);
        parts = plan.max_chunks;
    }
    if (e != cudaSuccess) return e;
    return launch_merge<HD>(a, hc, plan.stream, parts, st);
}

template <int HD, int NS>
static cudaError_t configure_one()
{
    cudaError_t e = cudaFuncSetAttribute(decode_splitk_kernel<HD, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         decode_smem_bytes<HD>());
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(decode_stream_kernel<HD, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                decode_smem_bytes<HD>());
}

// Opt in to the dynamic shared memory the first-stage kernels use (per device; called with the
// device current when a handle is created).
cudaError_t configure_decode()
{
    cudaError_t e;
#define HOOK_CFG(HD, NS) if ((e = configure_one<HD, NS>()) != cudaSuccess) return e;
    HOOK_CFG(64, 0) HOOK_CFG(64, 2) HOOK_CFG(64, 4) HOOK_CFG(64, 8)
    HOOK_CFG(128, 0) HOOK_CFG(128, 2) HOOK_CFG(128, 4) HOOK_CFG(128, 8)
#undef HOOK_CFG
    return cudaSuccess;
}

// Fixed chunks: one partial per (unit, chunk).  Streaming: the page-count prefix, then one partial
// per (unit, worker warp) pair that meets; the slot `unit + warp` is below units + workers.
size_t decode_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim, int max_keys)
{
    const DecodePlan plan = decode_plan(num_seqs, Hkv, max_keys);
    const size_t per_part = (size_t)G * decode_partial_stride(head_dim) * sizeof(float);
    if (plan.stream) return decode_prefix_bytes(num_seqs) + ((size_t)num_seqs * Hkv + kDecMaxWorkers) * per_part;
    return (size_t)num_seqs * Hkv * plan.max_chunks * per_part;
}

// For the kernel that runs decode CTAs of `warps` warps next to prefill CTAs in one launch: the workspace of
// the streaming cut whatever the unit count, and the merge that follows it.
size_t decode_stream_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim)
{
    const size_t per_part = (size_t)G * decode_partial_stride(head_dim) * sizeof(float);
    return decode_prefix_bytes(num_seqs) + ((size_t)num_seqs * Hkv + kDecMaxWorkers) * per_part;
}

cudaError_t launch_decode_stream_merge(const KernelArgs& a, const HeadCfg& hc, int ctas, int warps, cudaStream_t st)
{
    return launch_merge<128>(a, hc, true, stream_parts_estimate(a, ctas, warps), st);
}

cudaError_t launch_decode(const KernelArgs& a, const HeadCfg& hc, int head_dim, int num_sms, cudaStream_t st)
{
    const int ns = !a.any_probe ? 0 : (a.S <= 2 ? 2 : (a.S <= 4 ? 4 : 8));
#define HOOK_DISPATCH(HD)                                                         \
    switch (ns) {                                                                 \
        case 0: return launch_decode_t<HD, 0>(a, hc, num_sms, st);                \
        case 2: return launch_decode_t<HD, 2>(a, hc, num_sms, st);                \
        case 4: return launch_decode_t<HD, 4>(a, hc, num_sms, st);                \
        default: return launch_decode_t<HD, 8>(a, hc, num_sms, st);               \
    }
    if (head_dim == 128) { HOOK_DISPATCH(128) }
    HOOK_DISPATCH(64)
#undef HOOK_DISPATCH
}

}  // namespace hook_attn
