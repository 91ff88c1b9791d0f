// One launch for a serving step that holds both a decode batch and prefill chunks (the mixed chunked batch).
//
// The decode call is bound by HBM bandwidth and needs only a part of the SMs to saturate it; the prefill call
// is bound by the tensor cores.  Launched one after the other, or side by side on two streams, each kernel
// fills whatever SMs it gets and the two overlap only at their edges, because one SM cannot hold a CTA of
// each (three decode CTAs of 64 KB or one prefill CTA of 193 KB of shared memory).  Here one grid of
// 384-thread CTAs carries both: the first `dec_ctas` CTAs take the decode role -- twelve warps that stream an
// equal share of the flat page list each, exactly as the stand-alone streaming kernel does with four -- and
// stay for the whole step; the others take the prefill role, one pair of query tiles each, and are cycled
// through the remaining SMs by the hardware.  The split is chosen on the host from the two calls' bytes and
// flops.  The merge of the decode partials stays a second launch.
#include <stdlib.h>

#include "decode_device.cuh"
#include "prefill_tc_device.cuh"

namespace hook_attn {

using namespace tc;

// decode.cu
size_t decode_stream_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim);
cudaError_t launch_decode_stream_merge(const KernelArgs& a, const HeadCfg& hc, int ctas, int warps, cudaStream_t st);
// prefill_tc.cu
bool prefill_tc_maps(const KernelArgs& a, void* tmap_cache, CUtensorMap* mq, CUtensorMap* mk, CUtensorMap* mv);
int prefill_tc_pairs(const KernelArgs& a);
unsigned int prefill_tc_launch_id();
bool prefill_tc_supported(const KernelArgs& a, int head_dim);

constexpr int kMixWarps = kThreads / 32;   // twelve warps per CTA in either role
static_assert(kMixWarps % kDecWarps == 0, "decode warps fold in groups of four");
static_assert(kMixWarps * kDecStages * 2 * kPage * 128 * 2 + 1024 <= kSmemBytes, "the decode role's page buffers fit the prefill CTA's shared memory");

template <int NS_PF, int NS_DEC>
__global__ void __launch_bounds__(kThreads, 1)
mixed_kernel(const KernelArgs apf, const HeadCfg hpf, const KernelArgs adec, const HeadCfg hdec, const unsigned int launch_id,
             const int dec_ctas, const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
             const __grid_constant__ CUtensorMap map_v)
{
    extern __shared__ uint8_t smem_raw[];
    if ((int)blockIdx.x < dec_ctas) {
        __shared__ DecStreamShared<kMixWarps> sh;
        uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
        decode_stream_cta<128, NS_DEC, kMixWarps>(adec, hdec, base, blockIdx.x, sh);
    } else {
        const int idx = (int)blockIdx.x - dec_ctas;
        prefill_tc_cta<NS_PF>(apf, hpf, launch_id, &map_q, &map_k, &map_v, idx % apf.Hq, idx / apf.Hq, smem_raw);
    }
}

template <int NS_PF, int NS_DEC>
static cudaError_t launch_mixed_t(const KernelArgs& apf, const HeadCfg& hpf, const KernelArgs& adec, const HeadCfg& hdec,
                                  const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, int dec_ctas, long grid,
                                  cudaStream_t st)
{
    mixed_kernel<NS_PF, NS_DEC><<<(unsigned)grid, kThreads, kSmemBytes, st>>>(apf, hpf, adec, hdec, prefill_tc_launch_id(), dec_ctas,
                                                                            mq, mk, mv);
    return cudaGetLastError();
}

cudaError_t configure_mixed()
{
    cudaError_t e;
#define HOOK_CFG(A, B) if ((e = cudaFuncSetAttribute(mixed_kernel<A, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return e;
    HOOK_CFG(0, 0) HOOK_CFG(0, 4) HOOK_CFG(0, 8) HOOK_CFG(8, 0) HOOK_CFG(8, 4) HOOK_CFG(8, 8)
#undef HOOK_CFG
    return cudaSuccess;
}

// The fused launch serves head_dim 128 on both sides, a prefill call the tensor-core kernel can take and a
// decode batch the streaming body can scan in one pass.
bool mixed_supported(const KernelArgs& apf, int head_dim_pf, const KernelArgs& adec, int head_dim_dec)
{
    return head_dim_dec == 128 && adec.num_seqs <= kScanSeqs && prefill_tc_supported(apf, head_dim_pf);
}

size_t mixed_decode_workspace_bytes(int num_seqs, int Hkv, int G, int head_dim)
{
    return decode_stream_workspace_bytes(num_seqs, Hkv, G, head_dim);
}

// How many CTAs take the decode role.  The host knows bounds, not lengths: the decode call is taken to read
// 0.55 of the keys its bound allows and the prefill rows to see 0.8 of theirs.  An SM in the decode role is
// taken to stream 60 GB/s (52 GB/s when it probes; twelve warps with one 8 KB page in flight each; 75-90 GB/s were
// measured with few decode SMs, less once HBM fills up), an SM in the prefill role to
// sustain 5.7 TFLOP/s; the split equalises the two times.  Too many decode CTAs cost little -- their SMs go to
// prefill CTAs when they are done -- too few leave the decode as the long pole, so the result is rounded up.
int mixed_decode_ctas(const KernelArgs& apf, const KernelArgs& adec, int num_sms, int forced)
{
    int d;
    if (forced > 0) {
        d = forced;
    } else {
        const double bytes = 0.55 * (double)adec.num_seqs * adec.Hkv * adec.max_keys * 4.0 * 128;
        const double flops = 0.8 * (double)apf.total_q * apf.Hq * apf.max_keys * 4.0 * 128;
        // with span sums to carry, a decode SM streams less: measured optimum 72 CTAs against 64-67 without (0.585
        // against 0.596 ms at 67)
        const double t_dec1 = bytes / (adec.any_probe ? 52e9 : 60e9), t_pf1 = flops / 5.7e12;     // seconds on one SM
        d = (int)(num_sms * t_dec1 / (t_dec1 + t_pf1) + 0.999) + 2;
    }
    if (d > num_sms - 8) d = num_sms - 8;
    if (d * kMixWarps > 3 * 148 * kDecWarps) d = 3 * 148 * kDecWarps / kMixWarps;   // the workspace is sized for that many warps
    if (d < 1) d = 1;
    return d;
}

cudaError_t launch_mixed(const KernelArgs& apf, const HeadCfg& hpf, const KernelArgs& adec_in, const HeadCfg& hdec, void* tmap_cache,
                         int num_sms, int forced_dec_ctas, cudaStream_t st)
{
    CUtensorMap mq, mk, mv;
    if (!prefill_tc_maps(apf, tmap_cache, &mq, &mk, &mv)) return cudaErrorInvalidValue;
    KernelArgs adec = adec_in;
    const int dec_ctas = mixed_decode_ctas(apf, adec, num_sms, forced_dec_ctas);
    adec.workers = dec_ctas * kMixWarps;
    const long grid = (long)dec_ctas + (long)prefill_tc_pairs(apf) * apf.Hq;
    // the prefill role has two forms (no spans, up to 8); the decode role keeps its span sums in registers and has
    // one for up to 4 spans as well
    const bool ppf = apf.any_probe;
    const int nsd = !adec.any_probe ? 0 : (adec.S <= 4 ? 4 : 8);
    cudaError_t e;
    if (ppf && nsd == 8) e = launch_mixed_t<8, 8>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    else if (ppf && nsd == 4) e = launch_mixed_t<8, 4>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    else if (ppf) e = launch_mixed_t<8, 0>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    else if (nsd == 8) e = launch_mixed_t<0, 8>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    else if (nsd == 4) e = launch_mixed_t<0, 4>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    else e = launch_mixed_t<0, 0>(apf, hpf, adec, hdec, mq, mk, mv, dec_ctas, grid, st);
    if (e != cudaSuccess) return e;
    return launch_decode_stream_merge(adec, hdec, dec_ctas, kMixWarps, st);
}

}  // namespace hook_attn
