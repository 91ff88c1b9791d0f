// Shared device helpers and launch-parameter structs of the hooked paged-attention kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hook_attn.h"

namespace hook_attn {

constexpr int kPage = 16;        // tokens per KV page (the only supported page size)
constexpr int kMaxHeads = 64;    // query heads per call
constexpr int kMaxSpans = 8;     // spans per sequence
constexpr int kMaxGroup = 8;     // query heads per KV head

// Per-head hook configuration, passed by value in the kernel parameters so that "hooks
// disabled" is a launch-time fact (no device memory is read to find out).
struct HeadCfg {
    float  alpha[kMaxHeads];   // 0 = not steered
    int8_t slot[kMaxHeads];    // index of the head in the compact span_mass layout, -1 = not probed
};

struct KernelArgs {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    int64_t bs, ts, hs;               // KV strides in elements: block, token, head
    const int32_t* block_table;
    const int32_t* seq_lens;
    const int32_t* cu_q_lens;
    const int32_t* spans;
    const float* steer;
    __nv_bfloat16* out;
    float* mass;
    float* ws;
    int32_t* status;
    int32_t num_seqs, total_q, Hq, Hkv, G, num_blocks, max_blocks, S, P, probe_rows;
    int32_t max_keys;                 // longest sequence the call may hold: the caller's hint, else max_blocks * page
    int32_t workers;                  // decode, equal shares: warps that share the flat page list
    int32_t chunk;                    // decode, fixed chunks: keys per chunk
    int32_t max_chunks;               // decode, fixed chunks: chunks per sequence the workspace is sized for
    int32_t total_tiles;              // prefill: upper bound on query tiles
    float scale_log2;                 // scale * log2(e)
    bool any_probe, any_steer;
};

// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid)
{
    // 16-byte asynchronous copy; when !valid nothing is read and the destination is zero-filled.
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<uint32_t*>(&t);
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Swizzled byte offset of 16-byte chunk `c` of row `r` in a tile whose rows are ROW_BYTES long
// (ROW_BYTES = 128 or 256): chunks are XOR-ed with the row index so that the eight rows an
// ldmatrix reads fall into distinct banks.
template <int ROW_BYTES>
__device__ __forceinline__ uint32_t swz(int r, int c)
{
    return static_cast<uint32_t>(r * ROW_BYTES + ((c ^ (r & 7)) << 4));
}

__device__ __forceinline__ void report(int32_t* status, int code)
{
    if (status) atomicMin(status, code);
}

}  // namespace hook_attn
