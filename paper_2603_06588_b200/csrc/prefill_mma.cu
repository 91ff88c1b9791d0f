// Prefill / chunked prefill of the hooked paged attention, warp-level tensor-core version.
//
// One CTA handles 64 query rows of one (sequence, query head): four warps of 16 rows each.  Key
// tiles of 64 keys (four pages) are gathered through the block table with 16-byte cp.async copies
// into a double-buffered, XOR-swizzled shared-memory tile (rows past the end of the sequence are
// zero-filled, pages past it are never touched).  Scores and the PV product use
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate) with the usual register reuse of the probability
// tile as the A operand.  The probe's span masses are extra per-row accumulators in the frame of
// the running sum: a key tile that lies completely inside a span adds the tile's row sum, a tile
// that straddles a span edge adds a masked row sum, a disjoint tile adds nothing.  The epilogue
// normalises, applies the steering add in fp32 and rounds once to bf16.
//
// This kernel serves every supported shape (head_dim 64 and 128, any group size); the
// tcgen05/TMEM kernel takes over the large head_dim-128 shapes.
#include "common.cuh"

namespace hook_attn {

constexpr int kPfBM = 64;   // query rows per CTA
constexpr int kPfBN = 64;   // keys per tile

template <int HD>
constexpr int prefill_mma_smem_bytes()
{
    return kPfBM * HD * 2 + 2 * 2 * kPfBN * HD * 2;
}

template <int HD, int NS>
__global__ void __launch_bounds__(128) prefill_mma_kernel(const KernelArgs a, const HeadCfg hc)
{
    constexpr int ROWB = HD * 2;
    constexpr int CPR = HD / 8;
    constexpr int KS = HD / 16;
    constexpr int QB = kPfBM * ROWB;        // Q tile bytes
    constexpr int TB = kPfBN * ROWB;        // K or V tile bytes

    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ int sh_span[2 * kMaxSpans];

    const int h = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;
    const int kvh = h / a.G;

    // last-token mode: a sequence without rows in this call gets zeros in its span_mass row
    if (NS > 0 && blockIdx.x == 0 && blockIdx.y == 0 && a.probe_rows == HOOK_PROBE_ROWS_LAST) {
        const int per = a.P * a.S;
        for (int sq = warp; sq < a.num_seqs; sq += 4) {
            if (a.cu_q_lens[sq + 1] - a.cu_q_lens[sq] > 0) continue;
            for (int i = lane; i < per; i += 32) a.mass[(int64_t)sq * per + i] = 0.f;
        }
    }

    // locate (sequence, query tile); later tiles of a sequence (more keys) are scheduled first
    int t = blockIdx.x, s = 0, n = 0;
    for (; s < a.num_seqs; ++s) {
        n = a.cu_q_lens[s + 1] - a.cu_q_lens[s];
        const int nt = (n + kPfBM - 1) / kPfBM;
        if (t < nt) { t = nt - 1 - t; break; }
        t -= nt;
    }
    if (s >= a.num_seqs) return;
    const int L = a.seq_lens[s];
    const int row0 = t * kPfBM;
    const int rows = min(kPfBM, n - row0);
    const int64_t grow0 = (int64_t)a.cu_q_lens[s] + row0;
    const int slot = (NS > 0) ? hc.slot[h] : -1;
    const bool probe = (NS > 0) && slot >= 0;

    if (n > L || L > a.max_keys) {
        // inconsistent lengths: report, write zeros for this tile, touch nothing else
        if (threadIdx.x == 0) report(a.status, n > L ? HOOK_ATTN_ERR_INVALID_ARG : HOOK_ATTN_ERR_BOUNDS);
        for (int idx = threadIdx.x; idx < rows * HD; idx += 128)
            a.out[((grow0 + idx / HD) * a.Hq + h) * HD + idx % HD] = __float2bfloat16(0.f);
        if (probe) {
            const bool last_only = (a.probe_rows == HOOK_PROBE_ROWS_LAST);
            for (int idx = threadIdx.x; idx < rows * a.S; idx += 128) {
                const int r = idx / a.S, js = idx % a.S;
                if (last_only && row0 + r != n - 1) continue;
                const int64_t mrow = last_only ? (int64_t)s : grow0 + r;
                a.mass[(mrow * a.P + slot) * a.S + js] = 0.f;
            }
        }
        return;
    }
    const int first_pos = L - n + row0;                 // position of the tile's first row
    const int pos_max = first_pos + rows - 1;
    const int ntiles = pos_max / kPfBN + 1;

    if (NS > 0 && (int)threadIdx.x < 2 * NS) {
        const int j = threadIdx.x >> 1;
        sh_span[threadIdx.x] = (probe && j < a.S) ? a.spans[((int64_t)s * a.S + j) * 2 + (threadIdx.x & 1)] : 0;
    }

    const uint32_t sq = smem_u32(smem);
    const uint32_t skv = sq + QB;
    const int32_t* bt = a.block_table + (int64_t)s * a.max_blocks;

    // Q tile -> shared (rows past the end of the sequence chunk are zero)
    for (int idx = threadIdx.x; idx < kPfBM * CPR; idx += 128) {
        const int r = idx / CPR, cc = idx % CPR;
        const bool ok = r < rows;
        const __nv_bfloat16* src = a.q + ((grow0 + (ok ? r : 0)) * a.Hq + h) * HD + cc * 8;
        cp_async16(sq + swz<ROWB>(r, cc), src, ok);
    }
    cp_async_commit();

    auto load_kv = [&](int j) {
        const uint32_t kd = skv + (j & 1) * (2 * TB);
        const uint32_t vd = kd + TB;
        for (int idx = threadIdx.x; idx < kPfBN * CPR; idx += 128) {
            const int r = idx / CPR, cc = idx % CPR;
            const int key = j * kPfBN + r;
            bool ok = key < L;
            int page = 0;
            if (ok) {
                page = bt[key / kPage];
                if (page < 0 || page >= a.num_blocks) { report(a.status, HOOK_ATTN_ERR_BOUNDS); ok = false; page = 0; }
            }
            const int64_t off = (int64_t)page * a.bs + (int64_t)(key % kPage) * a.ts + (int64_t)kvh * a.hs + cc * 8;
            cp_async16(kd + swz<ROWB>(r, cc), a.k + off, ok);
            cp_async16(vd + swz<ROWB>(r, cc), a.v + off, ok);
        }
        cp_async_commit();
    };

    load_kv(0);
    cp_async_wait<1>();      // Q has landed
    __syncthreads();

    uint32_t qa[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
        ldmatrix_x4(qa[ks], sq + swz<ROWB>(16 * warp + (lane & 7) + ((lane >> 3) & 1) * 8, 2 * ks + (lane >> 4)));

    // positions of this thread's two rows (clamped for padding rows, whose results are dropped)
    const int pr0 = min(first_pos + 16 * warp + g, L - 1);
    const int pr1 = min(first_pos + 16 * warp + g + 8, L - 1);

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[HD / 8][4];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float sm[NS > 0 ? NS : 1][2];
#pragma unroll
    for (int j = 0; j < (NS > 0 ? NS : 1); ++j) sm[j][0] = sm[j][1] = 0.f;

    for (int j = 0; j < ntiles; ++j) {
        if (j + 1 < ntiles) { load_kv(j + 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
        __syncthreads();
        const uint32_t kt = skv + (j & 1) * (2 * TB);
        const uint32_t vt = kt + TB;
        const int k0 = j * kPfBN;

        float sc[kPfBN / 8][4];
#pragma unroll
        for (int i = 0; i < kPfBN / 8; ++i) sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
#pragma unroll
        for (int np = 0; np < kPfBN / 16; ++np) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t kb[4];
                ldmatrix_x4(kb, kt + swz<ROWB>(16 * np + (lane & 7) + (lane >> 4) * 8, 2 * ks + ((lane >> 3) & 1)));
                mma_bf16_16816(sc[2 * np], qa[ks], kb[0], kb[1]);
                mma_bf16_16816(sc[2 * np + 1], qa[ks], kb[2], kb[3]);
            }
        }

        // scale, causal mask (select, never additive), row maxima
        const bool need_mask = (k0 + kPfBN - 1 > first_pos + 16 * warp) ;   // tile reaches past the warp's first row
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int i = 0; i < kPfBN / 8; ++i) {
            const int key = k0 + 8 * i + 2 * tq;
            float x0 = sc[i][0] * a.scale_log2, x1 = sc[i][1] * a.scale_log2;
            float x2 = sc[i][2] * a.scale_log2, x3 = sc[i][3] * a.scale_log2;
            if (need_mask) {
                if (key > pr0) x0 = -INFINITY;
                if (key + 1 > pr0) x1 = -INFINITY;
                if (key > pr1) x2 = -INFINITY;
                if (key + 1 > pr1) x3 = -INFINITY;
            }
            sc[i][0] = x0; sc[i][1] = x1; sc[i][2] = x2; sc[i][3] = x3;
            mx0 = fmaxf(mx0, fmaxf(x0, x1));
            mx1 = fmaxf(mx1, fmaxf(x2, x3));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // a row can be fully masked only in tiles beyond its position; keep its state unchanged then
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float c0 = fast_exp2(m0 - ms0), c1 = fast_exp2(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
        for (int i = 0; i < kPfBN / 8; ++i) {
            sc[i][0] = fast_exp2(sc[i][0] - ms0);
            sc[i][1] = fast_exp2(sc[i][1] - ms0);
            sc[i][2] = fast_exp2(sc[i][2] - ms1);
            sc[i][3] = fast_exp2(sc[i][3] - ms1);
            rs0 += sc[i][0] + sc[i][1];
            rs1 += sc[i][2] + sc[i][3];
        }
        l0 = l0 * c0 + rs0;
        l1 = l1 * c1 + rs1;
#pragma unroll
        for (int i = 0; i < HD / 8; ++i) { o[i][0] *= c0; o[i][1] *= c0; o[i][2] *= c1; o[i][3] *= c1; }

        if (NS > 0 && probe) {
#pragma unroll
            for (int js = 0; js < NS; ++js) {
                const int sa = sh_span[2 * js], sb = sh_span[2 * js + 1];
                float add0 = 0.f, add1 = 0.f;
                if (sb > k0 && sa < k0 + kPfBN) {
                    if (sa <= k0 && sb >= k0 + kPfBN) {
                        add0 = rs0; add1 = rs1;          // the whole tile lies inside the span
                    } else {
#pragma unroll
                        for (int i = 0; i < kPfBN / 8; ++i) {
                            const int key = k0 + 8 * i + 2 * tq;
                            const bool in_a = (key >= sa) && (key < sb), in_b = (key + 1 >= sa) && (key + 1 < sb);
                            add0 += (in_a ? sc[i][0] : 0.f) + (in_b ? sc[i][1] : 0.f);
                            add1 += (in_a ? sc[i][2] : 0.f) + (in_b ? sc[i][3] : 0.f);
                        }
                    }
                }
                sm[js][0] = sm[js][0] * c0 + add0;
                sm[js][1] = sm[js][1] * c1 + add1;
            }
        }

        // O += P V
#pragma unroll
        for (int kk = 0; kk < kPfBN / 16; ++kk) {
            uint32_t pa[4];
            pa[0] = pack_bf16(sc[2 * kk][0], sc[2 * kk][1]);
            pa[1] = pack_bf16(sc[2 * kk][2], sc[2 * kk][3]);
            pa[2] = pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]);
            pa[3] = pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
#pragma unroll
            for (int dp = 0; dp < HD / 16; ++dp) {
                uint32_t vb[4];
                ldmatrix_x4_trans(vb, vt + swz<ROWB>(16 * kk + (lane & 7) + ((lane >> 3) & 1) * 8, 2 * dp + (lane >> 4)));
                mma_bf16_16816(o[2 * dp], pa, vb[0], vb[1]);
                mma_bf16_16816(o[2 * dp + 1], pa, vb[2], vb[3]);
            }
        }
        __syncthreads();   // the tile may be overwritten by the next load
    }

    // ---- epilogue ----
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float inv0 = 1.f / l0, inv1 = 1.f / l1;
    const int r0 = 16 * warp + g, r1 = r0 + 8;
    const float al = hc.alpha[h];
    const float* sv = (al != 0.f) ? a.steer + (int64_t)h * HD : nullptr;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
        const int d = 8 * i + 2 * tq;
        float s0 = 0.f, s1 = 0.f;
        if (sv) { s0 = al * sv[d]; s1 = al * sv[d + 1]; }
        if (r0 < rows)
            *reinterpret_cast<uint32_t*>(a.out + ((grow0 + r0) * a.Hq + h) * HD + d) =
                pack_bf16(o[i][0] * inv0 + s0, o[i][1] * inv0 + s1);
        if (r1 < rows)
            *reinterpret_cast<uint32_t*>(a.out + ((grow0 + r1) * a.Hq + h) * HD + d) =
                pack_bf16(o[i][2] * inv1 + s0, o[i][3] * inv1 + s1);
    }
    if (NS > 0 && probe) {
#pragma unroll
        for (int js = 0; js < NS; ++js) {
            sm[js][0] += __shfl_xor_sync(0xffffffffu, sm[js][0], 1);
            sm[js][0] += __shfl_xor_sync(0xffffffffu, sm[js][0], 2);
            sm[js][1] += __shfl_xor_sync(0xffffffffu, sm[js][1], 1);
            sm[js][1] += __shfl_xor_sync(0xffffffffu, sm[js][1], 2);
        }
        if (tq == 0) {
            const bool last_only = (a.probe_rows == HOOK_PROBE_ROWS_LAST);
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                const int r = rr ? r1 : r0;
                if (r >= rows) continue;
                int64_t mrow;
                if (last_only) {
                    if (row0 + r != n - 1) continue;
                    mrow = s;
                } else {
                    mrow = grow0 + r;
                }
                float* dst = a.mass + (mrow * a.P + slot) * a.S;
                const float inv = rr ? inv1 : inv0;
#pragma unroll
                for (int js = 0; js < NS; ++js)
                    if (js < a.S) dst[js] = sm[js][rr] * inv;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
template <int HD, int NS>
static cudaError_t launch_prefill_mma_t(const KernelArgs& a, const HeadCfg& hc, cudaStream_t st)
{
    dim3 grid(a.total_tiles, a.Hq);
    prefill_mma_kernel<HD, NS><<<grid, 128, prefill_mma_smem_bytes<HD>(), st>>>(a, hc);
    return cudaGetLastError();
}

template <int HD, int NS>
static cudaError_t configure_one()
{
    return cudaFuncSetAttribute(prefill_mma_kernel<HD, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                prefill_mma_smem_bytes<HD>());
}

cudaError_t configure_prefill_mma()
{
    cudaError_t e;
#define HOOK_CFG(HD, NS) if ((e = configure_one<HD, NS>()) != cudaSuccess) return e;
    HOOK_CFG(64, 0) HOOK_CFG(64, 2) HOOK_CFG(64, 4) HOOK_CFG(64, 8)
    HOOK_CFG(128, 0) HOOK_CFG(128, 2) HOOK_CFG(128, 4) HOOK_CFG(128, 8)
#undef HOOK_CFG
    return cudaSuccess;
}

int prefill_mma_tiles_upper_bound(int total_q, int num_seqs)
{
    // sum over sequences of ceil(n_s / 64) <= floor(total_q / 64) + num_seqs
    return total_q / kPfBM + num_seqs;
}

cudaError_t launch_prefill_mma(const KernelArgs& a, const HeadCfg& hc, int head_dim, cudaStream_t st)
{
    const int ns = !a.any_probe ? 0 : (a.S <= 2 ? 2 : (a.S <= 4 ? 4 : 8));
#define HOOK_DISPATCH(HD)                                                         \
    switch (ns) {                                                                 \
        case 0: return launch_prefill_mma_t<HD, 0>(a, hc, st);                    \
        case 2: return launch_prefill_mma_t<HD, 2>(a, hc, st);                    \
        case 4: return launch_prefill_mma_t<HD, 4>(a, hc, st);                    \
        default: return launch_prefill_mma_t<HD, 8>(a, hc, st);                   \
    }
    if (head_dim == 128) { HOOK_DISPATCH(128) }
    HOOK_DISPATCH(64)
#undef HOOK_DISPATCH
}

}  // namespace hook_attn
