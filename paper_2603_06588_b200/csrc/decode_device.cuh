// Device code of the split-K decode shared by the stand-alone decode kernels and by the kernel that runs a
// decode batch and prefill chunks in one launch: the per-page routine, a warp's walk over a run of pages, the
// fold of four warps into one partial, and the body of a streaming CTA.
#pragma once

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

// Four consecutive warps (a CTA of the stand-alone kernels, a third of a twelve-warp CTA elsewhere)
// hold pieces of one unit: fold them, in warp order, into one partial.  Called by the 128 threads of the
// group, which meet at named barrier `bar_id`; `red` is the group's stage memory, free once each of its
// warps has drained its pipeline.
template <int HD, int NS>
__device__ __forceinline__ void decode_fold_cta(float* part, int G, float* red, DecFold& fold, int bar_id, float m0, float m1,
                                                float l0, float l1, const float (&o)[HD / 16][4],
                                                const float (&sm)[NS > 0 ? NS : 1][2])
{
    constexpr int KS = HD / 16;
    constexpr int OSTR = HD + 4;            // padded row of the cross-warp reduction buffer
    const int warp = (threadIdx.x >> 5) & (kDecWarps - 1), lane = threadIdx.x & 31;
    const int t128 = threadIdx.x & (kDecWarps * 32 - 1);
    const int g = lane >> 2, tq = lane & 3;
    if (g == 0) { fold.m[warp][2 * tq] = m0; fold.m[warp][2 * tq + 1] = m1; }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");   // also: every warp has drained its pipeline, the stage buffers are free
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
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");

    const size_t pstride = decode_partial_stride(HD);
    for (int idx = t128; idx < G * HD; idx += kDecWarps * 32) {
        const int h = idx / HD, d = idx % HD;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) acc += red[(w * 8 + h) * OSTR + d];
        part[h * pstride + d] = acc;
    }
    for (int idx = t128; idx < G * (2 + NS); idx += kDecWarps * 32) {
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

// Shared memory of a streaming CTA of NW warps (groups of four warps fold on their own).
template <int NW>
struct DecStreamShared {
    static constexpr int kEPT = (kScanSeqs + NW * 32 - 1) / (NW * 32);   // scan entries per thread
    int ex[kEPT * NW * 32];          // page counts of the sequences, then their exclusive prefix
    int wsum[NW];
    int span[NW][2 * kMaxSpans];
    DecFold fold[NW / kDecWarps];
};

// The work of streaming CTA `cta` (of a grid whose warps add up to a.workers): NW warps, each with
// kDecStages * 2 page buffers in `smem`.  Every thread of the CTA calls it.
template <int HD, int NS, int NW>
__device__ __forceinline__ void decode_stream_cta(const KernelArgs& a, const HeadCfg& hc, uint8_t* smem, int cta,
                                                  DecStreamShared<NW>& sh)
{
    constexpr int TILEB = kPage * HD * 2;   // bytes per 16-key tile
    constexpr int KS = HD / 16;
    constexpr int EPT = DecStreamShared<NW>::kEPT;
    constexpr int NT = NW * 32;
    int* sh_ex = sh.ex;
    int* sh_wsum = sh.wsum;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int quad = warp / kDecWarps;             // group of four warps: the unit of folding
    const int G = a.G;

    // ---- exclusive prefix of the page counts (the host only picks this kernel for fewer than
    //      kScanSeqs sequences); a thread owns EPT consecutive entries ----
    for (int i = threadIdx.x; i < EPT * NT; i += NT)
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
    for (int w = 0; w < NW; ++w) {
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
    // Launched with programmatic serialization, this grid may have started while the merge of the call before it
    // on the stream was still running (that merge lets its successor go at once); everything up to here read the
    // sequence lengths only.  From here on the grid writes the workspace, which that merge may be reading, and reads
    // q, which may be what that merge wrote: wait for it.  (Without such a predecessor the wait returns at once.)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (cta == 0) {   // the merge kernel sizes up its unit from this table
        int* prefix = reinterpret_cast<int*>(a.ws);
        for (int i = threadIdx.x; i < a.num_seqs; i += NT) prefix[i] = sh_ex[i];
        if (threadIdx.x == 0) prefix[a.num_seqs] = total_pages;
    }
    const long long flat_total = (long long)total_pages * a.Hkv;
    const long long share = decode_share(flat_total, a.workers);
    const int W = cta * NW + warp;
    const long long c_begin = (long long)(W - (warp & (kDecWarps - 1))) * share;   // the pages of this group of four warps
    const long long c_end = min(c_begin + kDecWarps * share, flat_total);
    if (c_begin >= c_end) return;                                                  // the whole group is idle
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

    // ---- all pages of the group in one unit: every warp reduces its piece, the group writes one partial ----
    int s, kvh, pg, np, L;
    locate(c_begin, s, kvh, pg, np, L);
    if (c_end - c_begin <= (long long)(np - pg)) {        // uniform over the group
        const int seg = (int)(f_end - f_begin);
        decode_segment<HD, NS>(a, hc, s, kvh, pg + (int)(f_begin - c_begin), seg, L, wbase, sh.span[warp], m0, m1, l0, l1, o, sm);
        float* part = parts + ((size_t)s * a.Hkv + kvh + (W - (warp & (kDecWarps - 1)))) * G * pstride;
        float* red = reinterpret_cast<float*>(smem + (size_t)quad * kDecWarps * kDecStages * 2 * TILEB);
        decode_fold_cta<HD, NS>(part, G, red, sh.fold[quad], 1 + quad, m0, m1, l0, l1, o, sm);
        return;
    }

    // ---- otherwise the warps are independent: each walks its share unit by unit, one partial per unit ----
    if (f_begin >= f_end) return;
    locate(f_begin, s, kvh, pg, np, L);
    long long rem = f_end - f_begin;
    while (rem > 0) {
        const int seg = (int)min((long long)(np - pg), rem);   // pages of unit (s, kvh) this warp handles
        decode_segment<HD, NS>(a, hc, s, kvh, pg, seg, L, wbase, sh.span[warp], m0, m1, l0, l1, o, sm);
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

}  // namespace hook_attn
