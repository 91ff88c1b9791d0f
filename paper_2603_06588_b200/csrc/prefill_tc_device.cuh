// Prefill / chunked prefill of the hooked paged attention on the 5th-generation tensor cores
// (head_dim 128): TMA-staged K/V pages, tcgen05.mma with accumulators in tensor memory.
//
// One CTA owns two consecutive 128-row query tiles ("A" and "B") of one (sequence, query head)
// and walks the 128-key tiles they need.  Roles (12 warps, three warpgroups):
//   warps 0-3  softmax of tile A: one thread per query row, reads the scores S_A from tensor
//              memory, keeps the online softmax and the span-mass accumulators, writes the bf16
//              probabilities P_A back over S_A, rescales the output accumulator O_A when the
//              running reference maximum moves, and runs the epilogue of tile A;
//   warps 4-7  the same for tile B;
//   warp  8    producer: resolves pages through the block table and issues one TMA box load per
//              (page, 64-wide half of the head) into 128B-swizzled K and V stages; it also zeroes the
//              value rows past the end of the sequence in the last tile;
//   warp  9    owns tensor memory and walks the issue loop as a whole, converged; one elected lane
//              of it issues the MMAs: S = Q K^T (both operands K-major in shared memory) and
//              O += P V (P from tensor memory, V as the MN-major B operand), ordered
//              PV(A,j) QK(A,j+1) PV(B,j) QK(B,j+1) so that one tile's softmax overlaps the other
//              tile's tensor work.  The pipe's queue of issued MMAs is shallow, so every cycle this
//              warp spends on anything else is a cycle the pipe may run dry: it does nothing but
//              wait and issue (plus one commit per step that hands the V stage back to the producer
//              as soon as the step's last P V has completed; the K stage is handed back by a softmax
//              thread of the later tile, which sees the completion of QK(.,j) anyway), and P V of a
//              tile is issued in two halves of 64 keys, the first as soon as the softmax has stored it.
// Tensor memory (512 columns): S_A/P_A at 0, S_B/P_B at 128, O_A at 256, O_B at 384.
//
// The softmax keeps a *reference* maximum that is only raised when a tile's maximum exceeds it by
// more than 2^8; probabilities, the running sum and the span accumulators all live in that frame,
// so the result is exact (the reference cancels in o / l and s_j / l) while most tiles need no
// rescale of the accumulator.  Span masses are added from the fp32 probabilities, before the
// rounding to bf16: a key tile inside a span adds its row sum to a running sum kept per set of
// covering spans (flushed to the per-span sums, which live in shared memory, when the set changes);
// a tile that straddles a span edge adds sums of the 32-key chunks inside the span plus a masked
// sum of the one or two chunks on an edge; a disjoint tile adds nothing.  The probabilities are
// handed to the MMA warp before any of this span work starts.
//
// Every wait on an mbarrier is bounded; when one runs out the role raises the CTA's abort flag (every
// other wait of the CTA polls it and gives up too), the CTA reports HOOK_ATTN_ERR_TIMEOUT through the
// status word, stamps a launch-wide word so that the CTAs of the same launch that have not started yet
// return at once, releases tensor memory and returns.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace hook_attn {

namespace tc {

constexpr int kBM = 128;             // query rows per tile
constexpr int kBN = 128;             // keys per tile
constexpr int kHD = 128;             // head dim
constexpr int kThreads = 384;            // three warpgroups: softmax A, softmax B, {producer, MMA, 2 idle warps}
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;
constexpr int kTileBytes = kBM * kHD * 2;       // 32 KB: one Q, K or V tile
constexpr int kHalfBytes = kTileBytes / 2;      // 16 KB: 128 rows x 64 elements
constexpr int kStages = 2;
constexpr int kSmemBytes = 2 * kTileBytes + 2 * kStages * kTileBytes + 1024;   // Q(A,B) + K,V stages + alignment slack
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;       // log2 units
constexpr int kMaskTiles = 1024;                // key tiles with a precomputed span classification

// Which spans does key tile [k0, k0 + 128) touch?  Low byte: spans that contain the whole tile;
// high byte: spans that straddle it (their masked row sum is needed).
__device__ __forceinline__ uint32_t classify_tile(const int* span, int ns, int k0)
{
    uint32_t m = 0;
    for (int js = 0; js < ns; ++js) {
        const int sa = span[2 * js], sb = span[2 * js + 1];
        if (sb > k0 && sa < k0 + kBN && sb > sa) m |= (sa <= k0 && sb >= k0 + kBN) ? (1u << js) : (0x100u << js);
    }
    return m;
}

// ---- mbarrier / TMA / tcgen05 wrappers --------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after `limit_ns` (two seconds unless stated otherwise), or as soon as another
// role of the CTA has given up (`abort_flag`, in shared memory).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag = nullptr,
                                          uint64_t limit_ns = 2000000000ull)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u) {
            if (abort_flag && *abort_flag) return false;
            if (global_timer_ns() - t0 > limit_ns) {
                if (abort_flag) *abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void tc_mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void tc_mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v)   // v: 32 consecutive values (registers)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float (&v)[32])
{
    const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t* r)   // r: 16 consecutive values (registers)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Wait for outstanding tensor-memory loads and tie the 32 loaded values to the wait, so that no use
// of them can be scheduled ahead of it.
__device__ __forceinline__ void tc_wait_ld_dep(float* v)
{
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :
                 : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Move the start-address field (units of 16 bytes) of a descriptor; the field never overflows here.
__device__ __forceinline__ uint64_t desc_advance(uint64_t d, uint32_t units16)
{
    return ((uint64_t)(uint32_t)(d >> 32) << 32) | (uint64_t)((uint32_t)d + units16);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128; b_mn = 1 for an MN-major B operand.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t b_mn)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}

// Set by a CTA whose wait ran out: the id of its launch and the time (globaltimer, ns).  CTAs of the same
// launch that start within the next seconds return at once instead of sitting out waits of their own, so
// that a wedged launch of thousands of CTAs ends after one wait limit and not after thousands.
struct LaunchAbort {
    unsigned long long when_ns;
    unsigned int launch_id;
};
static __device__ LaunchAbort g_launch_abort;
constexpr unsigned long long kAbortWindowNs = 5000000000ull;

template <bool B>
struct ProbedTag {
    static constexpr bool value = B;
};

struct Barriers {
    uint64_t q_full[2];
    uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
    uint64_t s_full[2], p_half[2], p_full[2], o_full[2];   // p_half: the first 64 keys of P are in tensor memory
    uint64_t v_tail;          // the producer has zeroed the value rows past the end of the sequence
    uint32_t tmem_base;
    int abort_flag;
};

}  // namespace tc

using namespace tc;

// The work of one CTA: the pair of query tiles `pair_index` (counted over the sequences of the call) of query
// head `h`.  Every thread of the CTA calls it; `smem_raw` is the CTA's dynamic shared memory (kSmemBytes).
template <int NS>
__device__ __forceinline__ void prefill_tc_cta(const KernelArgs& a, const HeadCfg& hc, const unsigned int launch_id,
                                               const CUtensorMap* map_q_ptr, const CUtensorMap* map_k_ptr,
                                               const CUtensorMap* map_v_ptr, const int h, const int pair_index, uint8_t* smem_raw)
{
    __shared__ Barriers bars;
    __shared__ int sh_span[2 * kMaxSpans];
    __shared__ uint16_t sh_tile_mask[kMaskTiles];   // per key tile: bits 0-7 spans covering it, bits 8-15 spans straddling it
    __shared__ __align__(16) float sh_steer[kHD];    // alpha[h] * steer_vec[h][:] of a steered head
    __shared__ float sh_sm[NS > 0 ? 2 : 1][NS > 0 ? kMaxSpans : 1][NS > 0 ? kBM : 1];   // span sums of tile x, span j, row r

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kvh = h / a.G;

    // The loads a CTA needs before it can start anything are issued side by side, not one after the other: a
    // CTA lives for a few dozen microseconds, and every dependent trip to global memory at its start is half a
    // microsecond in which its SM does nothing.
    const volatile LaunchAbort* ab = &g_launch_abort;
    const unsigned int ab_id = ab->launch_id;
    const unsigned long long ab_when = ab->when_ns;

    // ---- locate (sequence, pair of query tiles); later pairs of a sequence (more keys) come first ----
    // Every warp scans the sequences 32 at a time: a lane loads the row range and the length of its sequence, a
    // prefix sum over the lanes' pair counts finds the sequence that holds pair `pair_index`.
    int t = pair_index, s = -1, n = 0, L = 0;
    int64_t grow_seq = 0;
    for (int base = 0; base < a.num_seqs; base += 32) {
        const int sq = base + lane;
        int c0 = 0, c1 = 0, len = 0;
        if (sq < a.num_seqs) {
            c0 = a.cu_q_lens[sq];
            c1 = a.cu_q_lens[sq + 1];
            len = a.seq_lens[sq];
        }
        const int np = max(0, (c1 - c0 + 2 * kBM - 1) / (2 * kBM));
        int incl = np;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (t < total) {
            const int src = __ffs(__ballot_sync(0xffffffffu, t < incl)) - 1;   // first lane whose range ends past t
            const int before = __shfl_sync(0xffffffffu, incl - np, src);
            const int npair = __shfl_sync(0xffffffffu, np, src);
            s = base + src;
            n = __shfl_sync(0xffffffffu, c1 - c0, src);
            L = __shfl_sync(0xffffffffu, len, src);
            grow_seq = __shfl_sync(0xffffffffu, c0, src);
            t = npair - 1 - (t - before);
            break;
        }
        t -= total;
    }
    // last-token mode: a sequence without rows in this call gets zeros in its span_mass row
    if (NS > 0 && h == 0 && pair_index == 0 && a.probe_rows == HOOK_PROBE_ROWS_LAST) {
        const int per = a.P * a.S;
        for (int sq = warp; sq < a.num_seqs; sq += kThreads / 32) {
            if (a.cu_q_lens[sq + 1] - a.cu_q_lens[sq] > 0) continue;
            for (int i = lane; i < per; i += 32) a.mass[(int64_t)sq * per + i] = 0.f;
        }
    }
    if (s < 0) return;
    // once any CTA of this launch has given up on a wait, the rest of the grid does not start
    if (ab_id == launch_id && global_timer_ns() - ab_when < kAbortWindowNs) {
        if (threadIdx.x == 0) report(a.status, HOOK_ATTN_ERR_TIMEOUT);
        return;
    }
    const int row0[2] = {2 * t * kBM, (2 * t + 1) * kBM};
    int rows[2], first_pos[2], ntiles[2];
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        rows[x] = max(0, min(kBM, n - row0[x]));
        first_pos[x] = L - n + row0[x];
        ntiles[x] = rows[x] > 0 ? (first_pos[x] + rows[x] - 1) / kBN + 1 : 0;
    }
    if (n > L || L > a.max_keys) {
        if (threadIdx.x == 0) report(a.status, n > L ? HOOK_ATTN_ERR_INVALID_ARG : HOOK_ATTN_ERR_BOUNDS);
        const int nrows = rows[0] + rows[1];
        for (int idx = threadIdx.x; idx < nrows * kHD; idx += kThreads)
            a.out[((grow_seq + row0[0] + idx / kHD) * a.Hq + h) * kHD + idx % kHD] = __float2bfloat16(0.f);
        const int slot_bad = (NS > 0) ? hc.slot[h] : -1;
        if (NS > 0 && slot_bad >= 0) {   // the probed rows of this tile pair: zeros as well
            const bool last_only = (a.probe_rows == HOOK_PROBE_ROWS_LAST);
            for (int idx = threadIdx.x; idx < nrows * a.S; idx += kThreads) {
                const int r = row0[0] + idx / a.S, js = idx % a.S;
                if (last_only && r != n - 1) continue;
                const int64_t mrow = last_only ? (int64_t)s : grow_seq + r;
                a.mass[(mrow * a.P + slot_bad) * a.S + js] = 0.f;
            }
        }
        return;
    }
    const int nmax = max(ntiles[0], ntiles[1]);
    const int slot = (NS > 0) ? hc.slot[h] : -1;
    // in last-token mode only the pair of tiles that holds the sequence's last row carries the probe
    const bool probe = (NS > 0) && slot >= 0 &&
                       (a.probe_rows == HOOK_PROBE_ROWS_ALL || (n - 1 >= row0[0] && n - 1 < row0[0] + 2 * kBM));

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ[2] = {smem_base, smem_base + kTileBytes};
    const uint32_t sK = smem_base + 2 * kTileBytes;
    const uint32_t sV = sK + kStages * kTileBytes;

    // ---- set-up: barriers, spans, tensor memory ----
    // The producer warp initialises the barriers and at once starts the loads of Q and of the first
    // K/V tile, so that their latency runs under the rest of the set-up.
    if (warp == kProducerWarp && lane == 0) {
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&bars.q_full[x]), 1);
            mbar_init(smem_u32(&bars.s_full[x]), 1);
            mbar_init(smem_u32(&bars.p_half[x]), 128);
            mbar_init(smem_u32(&bars.p_full[x]), 128);
            mbar_init(smem_u32(&bars.o_full[x]), 1);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(smem_u32(&bars.k_full[i]), 1);
            mbar_init(smem_u32(&bars.k_empty[i]), 1);
            mbar_init(smem_u32(&bars.v_full[i]), 1);
            mbar_init(smem_u32(&bars.v_empty[i]), 1);
        }
        mbar_init(smem_u32(&bars.v_tail), 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    bool ok = true;   // false once a bounded wait ran out
    volatile int* abort_flag = &bars.abort_flag;
    const int32_t* bt = a.block_table + (int64_t)s * a.max_blocks;
    // producer: the loads of key tile j (K then V), one TMA box per (page, 64-wide half of the head)
    auto produce = [&](int j) {
        const int st = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        const int pages = min(kBN / kPage, (L - j * kBN + kPage - 1) / kPage);   // pages that hold keys < L
        int blk = 0;
        const int pg = lane >> 1, half = lane & 1;
        if (lane < 16 && pg < pages) {
            blk = bt[j * (kBN / kPage) + pg];
            if (blk < 0 || blk >= a.num_blocks) { report(a.status, HOOK_ATTN_ERR_BOUNDS); blk = 0; }
        }
#pragma unroll
        for (int kv = 0; kv < 2; ++kv) {
            const uint32_t full = smem_u32(kv ? &bars.v_full[st] : &bars.k_full[st]);
            const uint32_t empty = smem_u32(kv ? &bars.v_empty[st] : &bars.k_empty[st]);
            ok = __all_sync(0xffffffffu, mbar_wait(empty, ph ^ 1u, abort_flag));
            if (!ok) break;
            if (lane == 0) mbar_expect_tx(full, (uint32_t)pages * 2u * (kPage * 128u));
            __syncwarp();
            if (lane < 16 && pg < pages) {
                const uint32_t dst = (kv ? sV : sK) + st * kTileBytes + half * kHalfBytes + pg * (kPage * 128);
                tma_load_4d(dst, kv ? map_v_ptr : map_k_ptr, full, half * 64, kvh, 0, blk);
            }
        }
    };
    if (warp == kProducerWarp) {
        __syncwarp();
        if (lane == 0) {
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (ntiles[x] > 0) {
                    const uint32_t bar = smem_u32(&bars.q_full[x]);
                    mbar_expect_tx(bar, kTileBytes);
                    tma_load_3d(sQ[x], map_q_ptr, bar, 0, h, (int)(grow_seq + row0[x]));
                    tma_load_3d(sQ[x] + kHalfBytes, map_q_ptr, bar, 64, h, (int)(grow_seq + row0[x]));
                }
            }
        }
        if (nmax > 0) produce(0);
    }
    if (hc.alpha[h] != 0.f && (int)threadIdx.x < kHD) sh_steer[threadIdx.x] = hc.alpha[h] * a.steer[(int64_t)h * kHD + threadIdx.x];
    if (NS > 0 && (int)threadIdx.x < 2 * NS) {
        const int j = threadIdx.x >> 1;
        sh_span[threadIdx.x] = (probe && j < a.S) ? a.spans[((int64_t)s * a.S + j) * 2 + (threadIdx.x & 1)] : 0;
    }
    if (NS > 0 && probe) {
        const int* gspan = a.spans + (int64_t)s * a.S * 2;
        for (int jj = threadIdx.x; jj < min(nmax, kMaskTiles); jj += kThreads)
            sh_tile_mask[jj] = (uint16_t)classify_tile(gspan, a.S, jj * kBN);
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;

    // Register split between the warpgroups: the softmax threads keep a whole 128-wide score row in
    // registers, the producer/MMA warpgroup needs few.  Launched with 168 per thread (384 x 168 =
    // 64512); after the split 128 x (208 + 208 + 72) = 62464, which fits the launch allocation.
    if (warp >= 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 72;" ::: "memory");
    }
    if (warp == kProducerWarp) {
        // ================================ producer ================================
        for (int j = 1; j < nmax && ok; ++j) produce(j);
        if (ok && nmax > 0 && nmax * kBN > L) {
            // value rows at keys >= L (page tails, pages that were never loaded) must not reach the
            // tensor cores: 0 * NaN would poison the accumulator.  Zero them in shared memory once the
            // last tile has landed, then tell the MMA warp.
            const int j = nmax - 1, st = j & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.v_full[st]), (j >> 1) & 1, abort_flag));
            if (ok) {
                const int r_first = L - j * kBN;
                const uint32_t vb = sV + st * kTileBytes;
                for (int idx = lane; idx < (kBN - r_first) * 16; idx += 32) {
                    const int r = r_first + (idx >> 4), c = idx & 15;
                    const uint32_t addr = vb + (c >> 3) * kHalfBytes + r * 128 + (c & 7) * 16;
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&bars.v_tail));
            }
        }
    } else if (warp == kMmaWarp) {
        // ================================ MMA issue ================================
        constexpr uint32_t idesc_qk = instr_desc(0), idesc_pv = instr_desc(1);
        const uint32_t tS[2] = {tmem, tmem + 128}, tO[2] = {tmem + 256, tmem + 384};
        // Descriptors are built once; per MMA only the start-address field moves (one 32-bit add), so
        // that the issuing lane keeps the tensor pipe fed.
        const uint64_t dQ[2] = {smem_desc(sQ[0], 16, 1024), smem_desc(sQ[1], 16, 1024)};
        const uint64_t dK[2] = {smem_desc(sK, 16, 1024), smem_desc(sK + kTileBytes, 16, 1024)};
        const uint64_t dV[2] = {smem_desc(sV, kHalfBytes, 1024), smem_desc(sV + kTileBytes, kHalfBytes, 1024)};
        auto issue_qk = [&](int x, int j) {
            const uint64_t dq = dQ[x], dk = (j & 1) ? dK[1] : dK[0];
#pragma unroll
            for (int ks = 0; ks < kHD / 16; ++ks) {
                const uint32_t off = ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;
                tc_mma_ss(tS[x], desc_advance(dq, off), desc_advance(dk, off), idesc_qk, ks > 0);
            }
            tc_commit(smem_u32(&bars.s_full[x]));
        };
        // P V in two halves of 64 keys each: the first half starts as soon as its probabilities are in tensor
        // memory, while the softmax threads still work on the second
        auto issue_pv_half = [&](int x, int j, int half) {
            const uint64_t dv = (j & 1) ? dV[1] : dV[0];
#pragma unroll
            for (int kk = 0; kk < kBN / 32; ++kk) {
                const int ks = half * (kBN / 32) + kk;
                tc_mma_ts(tO[x], tS[x] + ks * 8, desc_advance(dv, (ks * 16 * 128) >> 4), idesc_pv, (ks > 0) || (j > 0));
            }
        };
        // The whole warp walks the issue loop in step -- every lane looks at the barriers, so loop counters,
        // descriptors and branch conditions stay warp-uniform -- and one elected lane issues the MMAs and
        // commits.  (A loop run by a single thread inside a divergent branch costs that thread several
        // times the instructions per MMA; the tensor pipe's queue is shallow, so every cycle the issuing
        // thread spends on anything else is a cycle the pipe idles.)  No votes: a lane whose wait runs out
        // raises the abort flag, which ends the other lanes' waits as well.
        uint32_t elected;
        asm volatile("{\n\t.reg .pred pe;\n\telect.sync _|pe, 0xffffffff;\n\tselp.u32 %0, 1, 0, pe;\n\t}" : "=r"(elected));
#pragma unroll
        for (int x = 0; x < 2; ++x)
            if (ok && ntiles[x] > 0) ok = mbar_wait(smem_u32(&bars.q_full[x]), 0, abort_flag);
        if (ok) ok = mbar_wait(smem_u32(&bars.k_full[0]), 0, abort_flag);
        if (ok) {
            tc_fence_after();
            if (elected) {
                if (ntiles[0] > 0) issue_qk(0, 0);
                if (ntiles[1] > 0) issue_qk(1, 0);
            }
        }
        for (int j = 0; j < nmax && ok; ++j) {
            const int st = j & 1;
            ok = mbar_wait(smem_u32(&bars.v_full[st]), (j >> 1) & 1, abort_flag);
            if (ok && j == nmax - 1 && (j + 1) * kBN > L) ok = mbar_wait(smem_u32(&bars.v_tail), 0, abort_flag);
            if (ok && j + 1 < nmax) ok = mbar_wait(smem_u32(&bars.k_full[(j + 1) & 1]), ((j + 1) >> 1) & 1, abort_flag);
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if (ok && j < ntiles[x]) {
                    ok = mbar_wait(smem_u32(&bars.p_half[x]), j & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (elected) issue_pv_half(x, j, 0);
                    ok = mbar_wait(smem_u32(&bars.p_full[x]), j & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (elected) {
                        issue_pv_half(x, j, 1);
                        // the step's last P V: once it has completed, V tile j is free for the producer
                        if (x == 1 || j >= ntiles[1]) tc_commit(smem_u32(&bars.v_empty[st]));
                        if (j + 1 < ntiles[x]) issue_qk(x, j + 1);
                        else tc_commit(smem_u32(&bars.o_full[x]));
                    }
                }
            }
        }
    } else if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;" ::: "memory");
        // ================================ softmax + epilogue ================================
        const int x = warp >> 2;                      // 0 = tile A, 1 = tile B
        const int nt = ntiles[x];
        if (nt > 0) {
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;
            const bool releases = (nt == nmax) && (x == 1 || ntiles[1] < nmax);   // the tile whose QK is issued last
            const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
            const uint32_t tS = tmem + x * 128 + lane_off;
            const uint32_t tO = tmem + 256 + x * 128 + lane_off;
            const int pos = min(first_pos[x] + row, L - 1);
            const float sl2 = a.scale_log2;
            float m_ref = -INFINITY, l = 0.f;
            // Span sums of the probe.  They live in shared memory (one column per thread, no bank conflicts)
            // and not in registers: consecutive key tiles are almost always covered by the same set of spans,
            // so their row sums collect in one running sum in a register, which is handed to the spans'
            // accumulators only when the set changes; tiles with a span edge add their masked sums directly.
            float* my_sm = &sh_sm[NS > 0 ? x : 0][0][NS > 0 ? row : 0];     // element of span j at my_sm[j * kBM]
            if (NS > 0 && probe)
                for (int js = 0; js < a.S; ++js) my_sm[js * kBM] = 0.f;
            float run_acc = 0.f;
            uint32_t run_mask = 0;
            auto flush_run = [&]() {
                for (uint32_t m = run_mask; m; m &= m - 1) my_sm[(__ffs(m) - 1) * kBM] += run_acc;
                run_acc = 0.f;
            };

            // The key loop exists twice: heads without a probe run the plain loop, whatever the call probes
            // elsewhere; probed heads carry the span sums.
            auto key_loop = [&](auto probed_c) {
                constexpr bool PROBED = decltype(probed_c)::value;
                // spans touching a key tile: low byte covering, high byte straddling; looked up one tile ahead
                auto tile_spans = [&](int j) -> uint32_t { return (j < kMaskTiles) ? sh_tile_mask[j] : classify_tile(sh_span, NS, j * kBN); };
                uint32_t tm_next = PROBED ? tile_spans(0) : 0u;
                for (int j = 0; j < nt && ok; ++j) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[x]), j & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    if (releases && (threadIdx.x & 127) == 0) {
                        // QK(., j) has completed, and with it every MMA issued before it: K tile j is free for
                        // the producer (V tiles are handed back by a commit of the MMA warp, which comes earlier)
                        mbar_arrive(smem_u32(&bars.k_empty[j & 1]));
                    }
                    const int k0 = j * kBN;
                    const bool need_mask = (k0 + kBN - 1 > first_pos[x]);

                    const uint32_t tm = tm_next;
                    if (PROBED && j + 1 < nt) tm_next = tile_spans(j + 1);

                    // the whole score row of this thread: four loads in flight, one wait
                    float sc[kBN];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tc_ld32(tS + 32 * c, sc + 32 * c);
#pragma unroll
                    for (int c = 0; c < 4; ++c) tc_wait_ld_dep(sc + 32 * c);
                    if (need_mask) {
                        // causal / end-of-sequence mask as a select (stale or poisoned keys never propagate)
                        const int lim = pos - k0;
#pragma unroll
                        for (int i = 0; i < kBN; ++i) sc[i] = (i <= lim) ? sc[i] : -INFINITY;
                    }
                    float mxp[4];   // four independent chains keep the dependency depth short
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        float t = max3(sc[32 * q4], sc[32 * q4 + 1], sc[32 * q4 + 2]);
#pragma unroll
                        for (int i = 3; i + 1 < 32; i += 2) t = max3(t, sc[32 * q4 + i], sc[32 * q4 + i + 1]);
                        mxp[q4] = fmaxf(t, sc[32 * q4 + 31]);
                    }
                    const float mx = fmaxf(max3(mxp[0], mxp[1], mxp[2]), mxp[3]) * sl2;

                    // raise the reference maximum only when it is exceeded by more than the threshold
                    const bool raise = mx > m_ref + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, raise)) {
                        const float m_new = fmaxf(m_ref, mx);
                        const float f = (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - m_new);
                        m_ref = m_new;
                        l *= f;
                        if (PROBED) {
                            run_acc *= f;
                            for (int js = 0; js < a.S; ++js) my_sm[js * kBM] *= f;
                        }
                        if (j > 0) {
                            float v[32];
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                tc_ld32(tO + 32 * c, v);
                                tc_wait_ld_dep(v);
#pragma unroll
                                for (int i = 0; i < 32; ++i) v[i] *= f;
                                tc_st32(tO + 32 * c, v);
                            }
                            tc_wait_st();
                        }
                    }

                    // probabilities in the frame of the reference maximum: fp32 for the sums, bf16 pairs
                    // written over the scores for the tensor cores
                    const float2 sl2v = make_float2(sl2, sl2), nmv = make_float2(-m_ref, -m_ref);
                    float2 rs2[4];   // row sums of the four 32-key chunks
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t pk[16];
                        rs2[c] = make_float2(0.f, 0.f);
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int e = 32 * c + 2 * i;
                            const float2 xx = __ffma2_rn(make_float2(sc[e], sc[e + 1]), sl2v, nmv);
                            const float2 pp = make_float2(fast_exp2(xx.x), fast_exp2(xx.y));
                            if (PROBED) {   // kept for the masked sums of a tile with a span edge
                                sc[e] = pp.x;
                                sc[e + 1] = pp.y;
                            }
                            rs2[c] = __fadd2_rn(rs2[c], pp);
                            pk[i] = pack_bf16(pp.x, pp.y);
                        }
                        tc_st16(tS + 16 * c, pk);
                        if (c == 1) {   // the first 64 keys: the MMA warp may start on them
                            tc_wait_st();
                            tc_fence_before();
                            mbar_arrive(smem_u32(&bars.p_half[x]));
                        }
                    }
                    const float cs[4] = {rs2[0].x + rs2[0].y, rs2[1].x + rs2[1].y, rs2[2].x + rs2[2].y, rs2[3].x + rs2[3].y};
                    const float rs = (cs[0] + cs[1]) + (cs[2] + cs[3]);
                    l += rs;
                    // P is complete: hand it to the MMA warp first, the span sums need registers only
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&bars.p_full[x]));
                    if (PROBED) {
                        // a tile inside spans adds its row sum to them (through the running sum)
                        const uint32_t cover = tm & 0xffu;
                        if (cover != run_mask) { flush_run(); run_mask = cover; }
                        run_acc += rs;
                        if (tm & 0xff00u) {
                            // Spans with an edge inside the tile add prefix(hi) - prefix(lo), where prefix(t) is the
                            // sum of the tile's first t probabilities: whole 32-key chunks from their row sums, the
                            // chunk that holds the edge as a masked sum of the probabilities kept above.
                            auto prefix = [&](int t) -> float {
                                if (t <= 0) return 0.f;
                                if (t >= kBN) return rs;
                                const int c = t >> 5;
                                const uint32_t r = (uint32_t)(t & 31);
                                float acc[4] = {c > 0 ? cs[0] : 0.f, c > 1 ? cs[1] : 0.f, c > 2 ? cs[2] : 0.f, 0.f};
#define HOOK_MASKED_CHUNK(C)                                                                        \
    _Pragma("unroll") for (uint32_t i = 0; i < 32; ++i) acc[i & 3] += (i < r) ? sc[32 * (C) + i] : 0.f;
                                switch (c) {   // static register indices in every case
                                    case 0: HOOK_MASKED_CHUNK(0) break;
                                    case 1: HOOK_MASKED_CHUNK(1) break;
                                    case 2: HOOK_MASKED_CHUNK(2) break;
                                    default: HOOK_MASKED_CHUNK(3) break;
                                }
#undef HOOK_MASKED_CHUNK
                                return (acc[0] + acc[1]) + (acc[2] + acc[3]);
                            };
#pragma unroll 1
                            for (int js = 0; js < a.S; ++js) {
                                if (!((tm >> (8 + js)) & 1u)) continue;
                                my_sm[js * kBM] += prefix(sh_span[2 * js + 1] - k0) - prefix(sh_span[2 * js] - k0);
                            }
                        }
                    }
                }
                if (PROBED) flush_run();
            };
            if (NS > 0 && probe) key_loop(ProbedTag<true>{});
            else key_loop(ProbedTag<false>{});

            // ---- epilogue: normalise, steer, round once, store ----
            if (ok) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.o_full[x]), 0, abort_flag));
            const float inv = 1.f / l;
            const bool live = row < rows[x];
            const uint32_t stage = sQ[x];
            if (ok) {
                tc_fence_after();
                const float al = hc.alpha[h];
                // A thread holds one output row; stored from here, a warp would write 32 rows with 16
                // bytes each per instruction.  The tile goes through the shared memory of Q_x instead
                // (free: every MMA of this tile has completed), 16-byte chunks XOR-ed with the row so
                // that neither side has bank conflicts, and leaves it two whole rows per instruction.
                float v[32];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    tc_ld32(tO + 32 * c, v);
                    tc_wait_ld_dep(v);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int d = 32 * c + 8 * q4 + 2 * i;
                            float y0 = v[8 * q4 + 2 * i] * inv, y1 = v[8 * q4 + 2 * i + 1] * inv;
                            if (al != 0.f) { y0 += sh_steer[d]; y1 += sh_steer[d + 1]; }
                            w[i] = pack_bf16(y0, y1);
                        }
                        const uint32_t addr = stage + row * 256 + (((4 * c + q4) ^ (row & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
                    }
                }
            }
            // all four warps of the tile meet here, also one whose waits ran out (it reported that)
            asm volatile("bar.sync %0, 128;" ::"r"(1 + x) : "memory");
            if (ok) {
                {
                    const int t128 = threadIdx.x & 127;
                    __nv_bfloat16* otile = a.out + ((grow_seq + row0[x]) * a.Hq + h) * kHD;
#pragma unroll 4
                    for (int it = 0; it < 16; ++it) {
                        const int idx = it * 128 + t128, r = idx >> 4, c = idx & 15;
                        if (r < rows[x]) {
                            uint4 val;
                            const uint32_t addr = stage + r * 256 + ((c ^ (r & 7)) << 4);
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(addr));
                            *reinterpret_cast<uint4*>(otile + (int64_t)r * a.Hq * kHD + c * 8) = val;
                        }
                    }
                }
                if (NS > 0 && probe && live) {
                    const bool last_only = (a.probe_rows == HOOK_PROBE_ROWS_LAST);
                    if (!last_only || row0[x] + row == n - 1) {
                        const int64_t mrow = last_only ? (int64_t)s : grow_seq + row0[x] + row;
                        float* dst = a.mass + (mrow * a.P + slot) * a.S;
                        for (int js = 0; js < a.S; ++js) dst[js] = my_sm[js * kBM] * inv;
                    }
                }
            }
        }
    }

    // ---- teardown ----
    if (!ok) {
        if (lane == 0) {
            report(a.status, HOOK_ATTN_ERR_TIMEOUT);
            g_launch_abort.launch_id = launch_id;
            g_launch_abort.when_ns = global_timer_ns();
        }
        const uint64_t t0 = global_timer_ns();           // let copies that are still in flight land
        while (global_timer_ns() - t0 < 1000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace hook_attn
