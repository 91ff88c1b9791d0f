// Operations that sit next to the hooked attention: the analyzer's score reduction over span
// masses, residual-stream activation steering, and the raw q/k capture of the probed heads.
// All three are bandwidth-trivial or bandwidth-bound element movers; none needs tensor cores.
#include "common.cuh"

namespace hook_attn {

// ---- analyzer reduction: span_mass [R][P][S] -> scores [R][S] ------------------------------------
// One warp per row; lanes walk the probed heads, the per-span sums are reduced with shuffles in a
// fixed order (deterministic).  mode 1 divides each head's masses by that head's total first.
__global__ void __launch_bounds__(128) score_kernel(const float* __restrict__ mass, float* __restrict__ scores,
                                                    int rows, int P, int S, int mode)
{
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    float acc[kMaxSpans];
#pragma unroll
    for (int j = 0; j < kMaxSpans; ++j) acc[j] = 0.f;
    for (int p = lane; p < P; p += 32) {
        const float* m = mass + ((int64_t)row * P + p) * S;
        float v[kMaxSpans], tot = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxSpans; ++j) { v[j] = (j < S) ? m[j] : 0.f; tot += v[j]; }
        const float w = (mode == 0) ? 1.f : (tot > 0.f ? 1.f / tot : 0.f);
#pragma unroll
        for (int j = 0; j < kMaxSpans; ++j) acc[j] += v[j] * w;
    }
#pragma unroll
    for (int j = 0; j < kMaxSpans; ++j)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    if (lane == 0) {
        const float inv = 1.f / (float)P;
#pragma unroll
        for (int j = 0; j < kMaxSpans; ++j)
            if (j < S) scores[(int64_t)row * S + j] = acc[j] * inv;
    }
}

cudaError_t launch_score(const float* mass, float* scores, int rows, int P, int S, int mode, cudaStream_t st)
{
    score_kernel<<<(rows + 3) / 4, 128, 0, st>>>(mass, scores, rows, P, S, mode);
    return cudaGetLastError();
}

// ---- residual-stream steering: hidden[t][:] += alpha * vec[:] (bf16 in place, fp32 add) -----------
// 16-byte accesses, one 8-element packet per thread and step; grid-stride over packets.
__global__ void __launch_bounds__(256) steer_residual_kernel(__nv_bfloat16* __restrict__ hidden, const float* __restrict__ vec,
                                                             float alpha, int64_t tokens, int hidden_size, int64_t row_stride)
{
    const int packets_per_row = hidden_size >> 3;
    const int64_t total = tokens * packets_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i / packets_per_row;
        const int c = (int)(i - t * packets_per_row) << 3;
        uint4* ptr = reinterpret_cast<uint4*>(hidden + t * row_stride + c);
        uint4 raw = *ptr;
        const float4 v0 = *reinterpret_cast<const float4*>(vec + c), v1 = *reinterpret_cast<const float4*>(vec + c + 4);
        __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&raw);
        float2 a0 = __bfloat1622float2(hp[0]), a1 = __bfloat1622float2(hp[1]);
        float2 a2 = __bfloat1622float2(hp[2]), a3 = __bfloat1622float2(hp[3]);
        raw.x = pack_bf16(fmaf(alpha, v0.x, a0.x), fmaf(alpha, v0.y, a0.y));
        raw.y = pack_bf16(fmaf(alpha, v0.z, a1.x), fmaf(alpha, v0.w, a1.y));
        raw.z = pack_bf16(fmaf(alpha, v1.x, a2.x), fmaf(alpha, v1.y, a2.y));
        raw.w = pack_bf16(fmaf(alpha, v1.z, a3.x), fmaf(alpha, v1.w, a3.y));
        *ptr = raw;
    }
}

cudaError_t launch_steer_residual(__nv_bfloat16* hidden, const float* vec, float alpha, int64_t tokens, int hidden_size,
                                  int64_t row_stride, int num_sms, cudaStream_t st)
{
    const int64_t packets = tokens * (hidden_size >> 3);
    int64_t blocks = (packets + 255) / 256;
    const int64_t cap = (int64_t)num_sms * 16;    // grid-stride beyond that
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    steer_residual_kernel<<<(unsigned)blocks, 256, 0, st>>>(hidden, vec, alpha, tokens, hidden_size, row_stride);
    return cudaGetLastError();
}

// ---- raw q/k capture ----------------------------------------------------------------------------
// k: grid (key tiles of 64, sequences); a warp takes one key at a time.  The key's rows of all KV heads
// are contiguous in the cache and its rows of the P probed heads are contiguous in the output, so the warp
// looks the page up once and then moves 32 / (D / 8) rows per instruction with 16-byte accesses (several
// in flight): no per-row index arithmetic.  q: one (row, probed head) per 16 lanes.
template <int HD>
__global__ void __launch_bounds__(256) capture_k_kernel(const KernelArgs a, const HeadCfg hc, __nv_bfloat16* __restrict__ k_out,
                                                        const int32_t* __restrict__ cu_k)
{
    constexpr int LPR = HD / 8;                 // lanes per row (16-byte packets)
    constexpr int RPW = 32 / LPR;               // rows per warp instruction
    __shared__ int8_t sh_kvh[kMaxHeads];        // KV head of the probed head in slot i
    if ((int)threadIdx.x < a.Hq && hc.slot[threadIdx.x] >= 0) sh_kvh[hc.slot[threadIdx.x]] = (int8_t)(threadIdx.x / a.G);
    __syncthreads();
    const int s = blockIdx.y;
    const int L = a.seq_lens[s];
    if (L <= 0 || L > a.max_keys) {
        if (L > a.max_keys && threadIdx.x == 0 && blockIdx.x == 0) report(a.status, HOOK_ATTN_ERR_BOUNDS);
        return;
    }
    const int t0 = blockIdx.x * 64;
    if (t0 >= L) return;
    const int t1 = min(L, t0 + 64);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / LPR, part = lane % LPR;
    const int32_t* bt = a.block_table + (int64_t)s * a.max_blocks;
    const int64_t out0 = (int64_t)cu_k[s];
    for (int t = t0 + warp; t < t1; t += 8) {
        const int page = bt[t / kPage];
        if (page < 0 || page >= a.num_blocks) { if (lane == 0) report(a.status, HOOK_ATTN_ERR_BOUNDS); continue; }
        const __nv_bfloat16* src = a.k + (int64_t)page * a.bs + (int64_t)(t % kPage) * a.ts + part * 8;
        __nv_bfloat16* dst = k_out + (out0 + t) * a.P * HD + part * 8;
        for (int p0 = 0; p0 < a.P; p0 += 4 * RPW) {   // four instructions' worth of rows: loads first, then stores
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int pi = p0 + u * RPW + sub;
                if (pi < a.P) v[u] = *reinterpret_cast<const uint4*>(src + (int64_t)sh_kvh[pi] * a.hs);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int pi = p0 + u * RPW + sub;
                if (pi < a.P) *reinterpret_cast<uint4*>(dst + (int64_t)pi * HD) = v[u];
            }
        }
    }
}

template <int HD>
__global__ void __launch_bounds__(256) capture_q_kernel(const KernelArgs a, const HeadCfg hc, __nv_bfloat16* __restrict__ q_out,
                                                        int out_rows, bool last_only, bool decode)
{
    constexpr int LPR = HD / 8;
    __shared__ int8_t sh_heads[kMaxHeads];
    if (threadIdx.x < kMaxHeads) sh_heads[threadIdx.x] = 0;
    __syncthreads();
    if ((int)threadIdx.x < a.Hq && hc.slot[threadIdx.x] >= 0) sh_heads[hc.slot[threadIdx.x]] = (int8_t)threadIdx.x;
    __syncthreads();
    const int part = threadIdx.x % LPR;
    const int64_t total = (int64_t)out_rows * a.P;
    for (int64_t r = (int64_t)blockIdx.x * (256 / LPR) + threadIdx.x / LPR; r < total; r += (int64_t)gridDim.x * (256 / LPR)) {
        const int64_t orow = r / a.P;
        const int pi = (int)(r % a.P);
        int64_t src_row = orow;
        uint4 v = make_uint4(0, 0, 0, 0);
        bool have = true;
        if (last_only && !decode) {
            const int s = (int)orow;
            const int n = a.cu_q_lens[s + 1] - a.cu_q_lens[s];
            have = n > 0;
            src_row = (int64_t)a.cu_q_lens[s + 1] - 1;
        }
        if (have) v = *reinterpret_cast<const uint4*>(a.q + (src_row * a.Hq + sh_heads[pi]) * HD + part * 8);
        *reinterpret_cast<uint4*>(q_out + (orow * a.P + pi) * HD + part * 8) = v;
    }
}

cudaError_t launch_capture(const KernelArgs& a, const HeadCfg& hc, int head_dim, bool decode, __nv_bfloat16* q_out,
                           __nv_bfloat16* k_out, const int32_t* cu_k, cudaStream_t st)
{
    const bool last_only = decode || a.probe_rows == HOOK_PROBE_ROWS_LAST;
    const int out_rows = last_only ? a.num_seqs : a.total_q;
    const int key_tiles = (a.max_keys + 63) / 64;
    if (q_out && out_rows > 0) {
        const int64_t total = (int64_t)out_rows * a.P;
        int blocks = (int)((total + 15) / 16);
        if (blocks > 4096) blocks = 4096;
        if (head_dim == 128) capture_q_kernel<128><<<blocks, 256, 0, st>>>(a, hc, q_out, out_rows, last_only, decode);
        else capture_q_kernel<64><<<blocks, 256, 0, st>>>(a, hc, q_out, out_rows, last_only, decode);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (k_out && key_tiles > 0 && a.num_seqs > 0) {
        dim3 grid(key_tiles, a.num_seqs);
        if (head_dim == 128) capture_k_kernel<128><<<grid, 256, 0, st>>>(a, hc, k_out, cu_k);
        else capture_k_kernel<64><<<grid, 256, 0, st>>>(a, hc, k_out, cu_k);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

}  // namespace hook_attn
