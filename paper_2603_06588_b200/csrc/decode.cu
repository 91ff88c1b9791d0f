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
#include "common.cuh"

namespace hook_attn {

constexpr int kDecWarps = 4;
// Two stages of one page (K and V) per warp: 64 KB per CTA, three CTAs per SM.  A warp needs well over
// a thousand cycles per page (dependent MMA chains, the exponentials, the transposes), so twelve warps
// per SM with one page in flight each stream faster than eight with two (measured: decode batch 104.4
// against 108.4 us per step; four warps with five pages in flight each: 145.6 us).
constexpr int kDecStages = 2;
constexpr int kDecCtasPerSM = 3;
constexpr int kDecMaxSMs = 148;                       // SMs of a B200; a device with fewer gets a smaller streaming grid
constexpr int kDecStreamUnits = 2 * kDecMaxSMs;       // the streaming kernel is picked for fewer units than this
constexpr int kDecMaxWorkers = kDecCtasPerSM * kDecMaxSMs * kDecWarps;   // most warps that share the flat page list
constexpr int kScanSeqs = 512;                        // most sequences the streaming kernel is picked for (a power of two)
constexpr int kPartPad = 16;   // floats after o[D] in a partial: m, l, s[0..7], padding
static_assert(kDecStreamUnits <= kScanSeqs, "the streaming kernel scans all sequences in one pass");

template <int HD>
constexpr int decode_smem_bytes()
{
    return kDecWarps * kDecStages * 2 * kPage * HD * 2;
}

__host__ __device__ inline size_t decode_partial_stride(int head_dim) { return (size_t)head_dim + kPartPad; }

// Pages that hold keys of a sequence; lengths that are not positive or exceed the block table
// count as empty here (the merge kernel reports them and zero-fills their rows).
__device__ __forceinline__ int decode_pages(int L, int max_keys)
{
    return (L > 0 && L <= max_keys) ? (L + kPage - 1) / kPage : 0;
}

// Pages of the flat list per worker warp.
__device__ __forceinline__ long long decode_share(long long flat_total, int workers)
{
    return (flat_total + workers - 1) / workers;
}

// Bytes at the start of the streaming kernel's workspace that hold the page-count prefix of the
// sequences (num_seqs + 1 ints, written by its first CTA for the merge kernel).
__host__ __device__ inline size_t decode_prefix_bytes(int num_seqs) { return (((size_t)num_seqs + 1) * 4 + 255) & ~(size_t)255; }


// One 16-key page of a unit: scores of the page against the G query heads, online softmax, span
// accumulators, P V.  Thread layout of the warp-level MMA: lane = 4 g + tq holds keys g and g + 8 of the
// page for the heads 2 tq and 2 tq + 1.  The softmax keeps a reference maximum per head that is only
// raised when a score exceeds it by more than 2^8: probabilities, running sum, span accumulators and the
// output all live in that frame (the reference cancels in o / l and s_j / l, so the result is exact),
// and the common page needs neither the shuffles of a row maximum nor a rescale of the accumulators.
constexpr float kDecRaise = 8.0f;   // log2 units

template <int HD, int NS>
__device__ __forceinline__ void decode_page(uint32_t kt, uint32_t vt, int key0, int L, float scale_log2, bool probe,
                                            const int* span, const uint32_t (&qb)[HD / 16][2], float& m0, float& m1,
                                            float& l0, float& l1, float (&o)[HD / 16][4], float (&sm)[NS > 0 ? NS : 1][2])
{
    constexpr int ROWB = HD * 2;
    constexpr int KS = HD / 16;
    const int lane = threadIdx.x & 31, g = lane >> 2;
    float sca[4] = {0.f, 0.f, 0.f, 0.f}, scb[4] = {0.f, 0.f, 0.f, 0.f};   // two chains: half the dependent depth
#pragma unroll
    for (int ks = 0; ks < KS; ks += 2) {
        uint32_t af[4], bf[4];
        ldmatrix_x4(af, kt + swz<ROWB>((lane & 7) + ((lane >> 3) & 1) * 8, 2 * ks + (lane >> 4)));
        ldmatrix_x4(bf, kt + swz<ROWB>((lane & 7) + ((lane >> 3) & 1) * 8, 2 * (ks + 1) + (lane >> 4)));
        mma_bf16_16816(sca, af, qb[ks][0], qb[ks][1]);
        mma_bf16_16816(scb, bf, qb[ks + 1][0], qb[ks + 1][1]);
    }
    const int t0 = key0 + g, t1 = t0 + 8;
    const float x0 = (t0 < L) ? (sca[0] + scb[0]) * scale_log2 : -INFINITY;   // (key t0, head 2tq)
    const float x1 = (t0 < L) ? (sca[1] + scb[1]) * scale_log2 : -INFINITY;   // (key t0, head 2tq+1)
    const float x2 = (t1 < L) ? (sca[2] + scb[2]) * scale_log2 : -INFINITY;   // (key t1, head 2tq)
    const float x3 = (t1 < L) ? (sca[3] + scb[3]) * scale_log2 : -INFINITY;   // (key t1, head 2tq+1)
    float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
    if (__any_sync(0xffffffffu, mx0 > m0 + kDecRaise || mx1 > m1 + kDecRaise)) {   // always on a unit's first page
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, d));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, d));
        }
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);   // finite: key0 < L
        const float c0 = fast_exp2(m0 - mn0), c1 = fast_exp2(m1 - mn1);
        m0 = mn0; m1 = mn1;
        l0 *= c0; l1 *= c1;
#pragma unroll
        for (int i = 0; i < KS; ++i) { o[i][0] *= c0; o[i][1] *= c1; o[i][2] *= c0; o[i][3] *= c1; }
        if (NS > 0) {
#pragma unroll
            for (int j = 0; j < (NS > 0 ? NS : 1); ++j) { sm[j][0] *= c0; sm[j][1] *= c1; }
        }
    }
    const float p0 = fast_exp2(x0 - m0), p1 = fast_exp2(x1 - m1);
    const float p2 = fast_exp2(x2 - m0), p3 = fast_exp2(x3 - m1);
    l0 += p0 + p2;
    l1 += p1 + p3;

    if (NS > 0 && probe) {
#pragma unroll
        for (int j = 0; j < (NS > 0 ? NS : 1); ++j) {
            const int sa = span[2 * j], sb = span[2 * j + 1];
            if (sb > key0 && sa < key0 + kPage) {
                const bool in0 = (t0 >= sa) && (t0 < sb), in1 = (t1 >= sa) && (t1 < sb);
                sm[j][0] += (in0 ? p0 : 0.f) + (in1 ? p2 : 0.f);
                sm[j][1] += (in0 ? p1 : 0.f) + (in1 ? p3 : 0.f);
            }
        }
    }

    // P^T as the B operand (k = key, n = head): transpose the two 8x8 blocks across lanes.
    const uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1));
    const uint32_t pb1 = movmatrix_trans(pack_bf16(p2, p3));
#pragma unroll
    for (int i = 0; i < KS; ++i) {
        uint32_t af[4];
        ldmatrix_x4_trans(af, vt + swz<ROWB>((lane & 7) + (lane >> 4) * 8, 2 * i + ((lane >> 3) & 1)));
        mma_bf16_16816(o[i], af, pb0, pb1);
    }
}

// Shared memory of the fold of a CTA's four warps into one partial.
struct DecFold {
    float m[kDecWarps][8];
    float small[kDecWarps][8][2 + kMaxSpans];
};

// A warp's pages [pg, pg + seg) of unit (s, kvh): streamed through its private cp.async stages and
// reduced to (m, l, o, span sums) per query head of the group, in the thread layout of decode_page.
// l and the span sums come back summed over the warp; seg = 0 leaves the empty state (m = -inf).
template <int HD, int NS>
__device__ __forceinline__ void decode_segment(const KernelArgs& a, const HeadCfg& hc, int s, int kvh, int pg, int seg, int L,
                                               uint32_t wbase, int* span, float& m0, float& m1, float& l0, float& l1,
                                               float (&o)[HD / 16][4], float (&sm)[NS > 0 ? NS : 1][2])
{
    constexpr int ROWB = HD * 2;            // bytes per K/V row
    constexpr int TILEB = kPage * ROWB;     // bytes per 16-key tile
    constexpr int CPR = HD / 8;             // 16-byte chunks per row
    constexpr int RPI = 32 / CPR;           // rows covered by one warp-wide copy instruction
    constexpr int KS = HD / 16;             // k-steps of the score product / d-blocks of the output
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int G = a.G;

    m0 = -INFINITY; m1 = -INFINITY; l0 = 0.f; l1 = 0.f;
#pragma unroll
    for (int i = 0; i < KS; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
#pragma unroll
    for (int j = 0; j < (NS > 0 ? NS : 1); ++j) sm[j][0] = sm[j][1] = 0.f;
    if (seg <= 0) return;

    const int32_t* bt = a.block_table + (int64_t)s * a.max_blocks + pg;
    const int key_base = pg * kPage;

    bool probe = false;
    if constexpr (NS > 0) {
        for (int i = 0; i < G; ++i) probe |= (hc.slot[kvh * G + i] >= 0);
        __syncwarp();
        if (lane < 2 * NS) {
            const int j = lane >> 1;
            span[lane] = (probe && j < a.S) ? a.spans[((int64_t)s * a.S + j) * 2 + (lane & 1)] : 0;
        }
        __syncwarp();
    }

    // block ids of 32 consecutive pages, one per lane; the next 32 are fetched a window ahead
    int btw = 0, btw_next = (lane < seg) ? bt[lane] : 0;
    auto issue = [&](int it) {
        if (it < seg) {
            if ((it & 31) == 0) {
                btw = btw_next;
                btw_next = (it + 32 + lane < seg) ? bt[it + 32 + lane] : 0;
            }
            int page = __shfl_sync(0xffffffffu, btw, it & 31);
            const bool page_ok = (page >= 0 && page < a.num_blocks);
            if (!page_ok) { if (lane == 0) report(a.status, HOOK_ATTN_ERR_BOUNDS); page = 0; }
            const int key0 = key_base + it * kPage;
            const uint32_t kdst = wbase + (it % kDecStages) * (2 * TILEB);
            const uint32_t vdst = kdst + TILEB;
            const int64_t base = (int64_t)page * a.bs + (int64_t)kvh * a.hs;
#pragma unroll
            for (int i = 0; i < kPage / RPI; ++i) {
                const int r = i * RPI + lane / CPR;
                const int cc = lane % CPR;
                const bool ok = page_ok && (key0 + r < L);
                const int64_t off = base + (int64_t)r * a.ts + cc * 8;
                cp_async16(kdst + swz<ROWB>(r, cc), a.k + off, ok);
                cp_async16(vdst + swz<ROWB>(r, cc), a.v + off, ok);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int i = 0; i < kDecStages - 1; ++i) issue(i);

    // B fragments of Q^T (k = d, n = head): head g of the group, zero for padding heads.
    uint32_t qb[KS][2];
    {
        const __nv_bfloat16* qrow = a.q + ((int64_t)s * a.Hq + kvh * G + g) * HD;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qb[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 2 * tq) : 0u;
            qb[ks][1] = (g < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8 + 2 * tq) : 0u;
        }
    }

    for (int it = 0; it < seg; ++it) {
        issue(it + kDecStages - 1);
        cp_async_wait<kDecStages - 1>();
        __syncwarp();

        const int key0 = key_base + it * kPage;
        const uint32_t kt = wbase + (it % kDecStages) * (2 * TILEB);
        const uint32_t vt = kt + TILEB;

        decode_page<HD, NS>(kt, vt, key0, L, a.scale_log2, probe, span, qb, m0, m1, l0, l1, o, sm);
        __syncwarp();
    }
    cp_async_wait<0>();

    // per-thread partial sums -> per-warp sums (lanes with the same tq hold the same heads)
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, d);
        l1 += __shfl_xor_sync(0xffffffffu, l1, d);
        if (NS > 0) {
#pragma unroll
            for (int j = 0; j < NS; ++j) {
                sm[j][0] += __shfl_xor_sync(0xffffffffu, sm[j][0], d);
                sm[j][1] += __shfl_xor_sync(0xffffffffu, sm[j][1], d);
            }
        }
    }
}

// One warp's result as a partial of its own.
template <int HD, int NS>
__device__ __forceinline__ void decode_store_warp_partial(float* part, int G, float m0, float m1, float l0, float l1,
                                                          const float (&o)[HD / 16][4], const float (&sm)[NS > 0 ? NS : 1][2])
{
    constexpr int KS = HD / 16;
    const int lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
    const size_t pstride = decode_partial_stride(HD);
    const int h0 = 2 * tq, h1 = 2 * tq + 1;
    float* r0 = part + h0 * pstride;
    float* r1 = part + h1 * pstride;
#pragma unroll
    for (int i = 0; i < KS; ++i) {
        if (h0 < G) { r0[16 * i + g] = o[i][0]; r0[16 * i + 8 + g] = o[i][2]; }
        if (h1 < G) { r1[16 * i + g] = o[i][1]; r1[16 * i + 8 + g] = o[i][3]; }
    }
    if (g == 0) {
        if (h0 < G) {
            r0[HD] = m0; r0[HD + 1] = l0;
#pragma unroll
            for (int j = 0; j < NS; ++j) r0[HD + 2 + j] = sm[j][0];
        }
        if (h1 < G) {
            r1[HD] = m1; r1[HD + 1] = l1;
#pragma unroll
            for (int j = 0; j < NS; ++j) r1[HD + 2 + j] = sm[j][1];
        }
    }
}

// The four warps of a CTA hold pieces of one unit: fold them, in warp order, into one partial.  Called by
// every thread of the CTA; `red` is the CTA's stage memory, free once every warp has drained its pipeline.
template <int HD, int NS>
__device__ __forceinline__ void decode_fold_cta(float* part, int G, float* red, DecFold& fold, float m0, float m1, float l0,
                                                float l1, const float (&o)[HD / 16][4], const float (&sm)[NS > 0 ? NS : 1][2])
{
    constexpr int KS = HD / 16;
    constexpr int OSTR = HD + 4;            // padded row of the cross-warp reduction buffer
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    if (g == 0) { fold.m[warp][2 * tq] = m0; fold.m[warp][2 * tq + 1] = m1; }
    __syncthreads();   // also: every warp has drained its pipeline, the stage buffers are free
    float M0 = fold.m[0][2 * tq], M1 = fold.m[0][2 * tq + 1];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) { M0 = fmaxf(M0, fold.m[w][2 * tq]); M1 = fmaxf(M1, fold.m[w][2 * tq + 1]); }
    // a warp without pages has m = -inf and contributes zero; M is finite because the unit has keys
    const float f0 = (m0 == -INFINITY) ? 0.f : fast_exp2(m0 - M0), f1 = (m1 == -INFINITY) ? 0.f : fast_exp2(m1 - M1);

#pragma unroll
    for (int i = 0; i < KS; ++i) {
        float* r0 = red + (warp * 8 + 2 * tq) * OSTR;
        r0[16 * i + g] = o[i][0] * f0;
        r0[OSTR + 16 * i + g] = o[i][1] * f1;
        r0[16 * i + 8 + g] = o[i][2] * f0;
        r0[OSTR + 16 * i + 8 + g] = o[i][3] * f1;
    }
    if (g == 0) {
        fold.small[warp][2 * tq][0] = M0;
        fold.small[warp][2 * tq + 1][0] = M1;
        fold.small[warp][2 * tq][1] = l0 * f0;
        fold.small[warp][2 * tq + 1][1] = l1 * f1;
        if (NS > 0) {
#pragma unroll
            for (int j = 0; j < NS; ++j) {
                fold.small[warp][2 * tq][2 + j] = sm[j][0] * f0;
                fold.small[warp][2 * tq + 1][2 + j] = sm[j][1] * f1;
            }
        }
    }
    __syncthreads();

    const size_t pstride = decode_partial_stride(HD);
    for (int idx = threadIdx.x; idx < G * HD; idx += kDecWarps * 32) {
        const int h = idx / HD, d = idx % HD;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) acc += red[(w * 8 + h) * OSTR + d];
        part[h * pstride + d] = acc;
    }
    for (int idx = threadIdx.x; idx < G * (2 + NS); idx += kDecWarps * 32) {
        const int h = idx / (2 + NS), e = idx % (2 + NS);
        float val;
        if (e == 0) {
            val = fold.small[0][h][0];
        } else {
            val = 0.f;
#pragma unroll
            for (int w = 0; w < kDecWarps; ++w) val += fold.small[w][h][e];
        }
        part[h * pstride + HD + e] = val;
    }
}

template <int HD, int NS>
__global__ void __launch_bounds__(kDecWarps * 32) decode_stream_kernel(const KernelArgs a, const HeadCfg hc)
{
    constexpr int TILEB = kPage * HD * 2;   // bytes per 16-key tile
    constexpr int KS = HD / 16;
    constexpr int EPT = kScanSeqs / (kDecWarps * 32);   // scan entries per thread

    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ int sh_ex[kScanSeqs];                 // page counts of the sequences, then their exclusive prefix
    __shared__ int sh_wsum[kDecWarps];
    __shared__ int sh_span[kDecWarps][2 * kMaxSpans];
    __shared__ DecFold sh_fold;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = a.G;

    // ---- exclusive prefix of the page counts (the host only picks this kernel for fewer than
    //      kScanSeqs sequences); a thread owns EPT consecutive entries ----
    for (int i = threadIdx.x; i < kScanSeqs; i += kDecWarps * 32)
        sh_ex[i] = (i < a.num_seqs) ? decode_pages(a.seq_lens[i], a.max_keys) : 0;
    __syncthreads();
    int v[EPT], run = 0;
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        v[e] = sh_ex[threadIdx.x * EPT + e];
        run += v[e];
    }
    int incl = run;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += t;
    }
    if (lane == 31) sh_wsum[warp] = incl;
    __syncthreads();
    int off = incl - run, total_pages = 0;
#pragma unroll
    for (int w = 0; w < kDecWarps; ++w) {
        if (w < warp) off += sh_wsum[w];
        total_pages += sh_wsum[w];
    }
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
        sh_ex[threadIdx.x * EPT + e] = off;
        off += v[e];
    }
    __syncthreads();
    // the merge kernel may be scheduled from here on; it waits for this grid's writes itself
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0) {   // the merge kernel sizes up its unit from this table
        int* prefix = reinterpret_cast<int*>(a.ws);
        for (int i = threadIdx.x; i < a.num_seqs; i += kDecWarps * 32) prefix[i] = sh_ex[i];
        if (threadIdx.x == 0) prefix[a.num_seqs] = total_pages;
    }
    const long long flat_total = (long long)total_pages * a.Hkv;
    const long long share = decode_share(flat_total, a.workers);
    const int W = blockIdx.x * kDecWarps + warp;
    const long long c_begin = (long long)blockIdx.x * kDecWarps * share;           // the CTA's pages
    const long long c_end = min(c_begin + kDecWarps * share, flat_total);
    if (c_begin >= c_end) return;                                                  // the whole CTA is idle
    const long long f_begin = min((long long)W * share, flat_total);               // this warp's pages
    const long long f_end = min(f_begin + share, flat_total);

    // the unit that holds flat page f: the last sequence whose prefix, counted in pages of all its KV
    // heads, does not exceed it; then KV head and page inside the sequence
    auto locate = [&](long long f, int& s, int& kvh, int& pg, int& np, int& L) {
        const long long target = f / a.Hkv;
        int lo = 0, hi = a.num_seqs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (sh_ex[mid] <= target) lo = mid; else hi = mid - 1;
        }
        s = lo;
        L = a.seq_lens[s];
        np = decode_pages(L, a.max_keys);
        const long long r = f - (long long)sh_ex[s] * a.Hkv;   // offset inside the units of sequence s
        kvh = (int)(r / np);
        pg = (int)(r % np);
    };

    const uint32_t wbase = smem_u32(smem) + warp * (kDecStages * 2 * TILEB);
    const size_t pstride = decode_partial_stride(HD);
    float* parts = reinterpret_cast<float*>(reinterpret_cast<char*>(a.ws) + decode_prefix_bytes(a.num_seqs));

    float m0, m1, l0, l1, o[KS][4], sm[NS > 0 ? NS : 1][2];

    // ---- all pages of the CTA in one unit: every warp reduces its piece, the CTA writes one partial ----
    int s, kvh, pg, np, L;
    locate(c_begin, s, kvh, pg, np, L);
    if (c_end - c_begin <= (long long)(np - pg)) {        // uniform over the CTA
        const int seg = (int)(f_end - f_begin);
        decode_segment<HD, NS>(a, hc, s, kvh, pg + (int)(f_begin - c_begin), seg, L, wbase, sh_span[warp], m0, m1, l0, l1, o, sm);
        float* part = parts + ((size_t)s * a.Hkv + kvh + blockIdx.x * kDecWarps) * G * pstride;
        decode_fold_cta<HD, NS>(part, G, reinterpret_cast<float*>(smem), sh_fold, m0, m1, l0, l1, o, sm);
        return;
    }

    // ---- otherwise the warps are independent: each walks its share unit by unit, one partial per unit ----
    if (f_begin >= f_end) return;
    locate(f_begin, s, kvh, pg, np, L);
    long long rem = f_end - f_begin;
    while (rem > 0) {
        const int seg = (int)min((long long)(np - pg), rem);   // pages of unit (s, kvh) this warp handles
        decode_segment<HD, NS>(a, hc, s, kvh, pg, seg, L, wbase, sh_span[warp], m0, m1, l0, l1, o, sm);
        decode_store_warp_partial<HD, NS>(parts + ((size_t)s * a.Hkv + kvh + W) * G * pstride, G, m0, m1, l0, l1, o, sm);

        // ---- next unit ----
        rem -= seg;
        pg = 0;
        if (rem > 0 && ++kvh == a.Hkv) {
            kvh = 0;
            do {
                if (++s >= a.num_seqs) return;     // cannot happen while rem > 0; keeps every access in bounds
                L = a.seq_lens[s];
                np = decode_pages(L, a.max_keys);
            } while (np == 0);
        }
    }
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
    decode_fold_cta<HD, NS>(part, G, reinterpret_cast<float*>(smem), sh_fold, m0, m1, l0, l1, o, sm);
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

    // the partials are written by the kernel launched just before on the same stream
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int L = a.seq_lens[s];
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
        val *= inv;
        const float al = hc.alpha[h];
        if (al != 0.f) val += al * a.steer[(int64_t)h * HD + d];
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

template <int HD, int NS>
static cudaError_t launch_decode_t(KernelArgs a, const HeadCfg& hc, int num_sms, cudaStream_t st)
{
    const DecodePlan plan = decode_plan(a.num_seqs, a.Hkv, a.max_keys);
    a.chunk = plan.chunk;
    a.max_chunks = plan.max_chunks;
    long parts;   // partials per unit, to size the merge block
    if (plan.stream) {
        const int ctas = kDecCtasPerSM * (num_sms < kDecMaxSMs ? (num_sms > 0 ? num_sms : 1) : kDecMaxSMs);
        a.workers = ctas * kDecWarps;
        decode_stream_kernel<HD, NS><<<ctas, kDecWarps * 32, decode_smem_bytes<HD>(), st>>>(a, hc);
        // pages of a CTA if the sequences are half as long as they may be; a long unit then has about
        // max pages / that many folded partials, plus the warps of its two shared CTAs
        const long max_pages = ((long)a.max_keys + kPage - 1) / kPage;
        const long est_cta = ((long)a.num_seqs * a.Hkv * max_pages / 2 + ctas - 1) / ctas;
        parts = max_pages / (est_cta > 0 ? est_cta : 1) + 2 * kDecWarps;
    } else {
        decode_splitk_kernel<HD, NS><<<dim3(plan.max_chunks, a.Hkv, a.num_seqs), kDecWarps * 32, decode_smem_bytes<HD>(), st>>>(a, hc);
        parts = plan.max_chunks;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // The merge is launched with programmatic stream serialization: its launch overlaps the drain of
    // the first kernel, and it waits (griddepcontrol.wait) until that kernel's writes are visible.
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
    return plan.stream ? cudaLaunchKernelEx(&cfg, decode_merge_kernel<HD, true>, a, hc)
                       : cudaLaunchKernelEx(&cfg, decode_merge_kernel<HD, false>, a, hc);
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
