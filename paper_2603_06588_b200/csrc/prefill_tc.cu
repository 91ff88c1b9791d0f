// Prefill / chunked prefill of the hooked paged attention on the 5th-generation tensor cores: the kernel
// around the CTA routine of prefill_tc_device.cuh, its TMA descriptors and its launch.
#include <string.h>

#include <atomic>
#include <mutex>
#include <utility>
#include <vector>

#include "prefill_tc_device.cuh"

namespace hook_attn {

using namespace tc;

template <int NS>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const KernelArgs a, const HeadCfg hc, const unsigned int launch_id, const __grid_constant__ CUtensorMap map_q,
                  const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v)
{
    extern __shared__ uint8_t smem_raw[];
    prefill_tc_cta<NS>(a, hc, launch_id, &map_q, &map_k, &map_v, blockIdx.x, blockIdx.y, smem_raw);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

// What a descriptor is made from; descriptors are cached under it.
struct TmapKey {
    const void* base;
    uint32_t rank;
    uint32_t box[4];
    uint64_t dims[4];
    uint64_t strides[3];   // bytes
};

struct TmapCache {
    static constexpr size_t kEntries = 256;   // a model's layers times q/k/v; replaced round-robin beyond that
    std::mutex mu;
    std::vector<std::pair<TmapKey, CUtensorMap>> entries;
    size_t next = 0;
};

// The descriptor of a bf16 tensor with 128B-swizzled boxes: from the cache when the same base pointer,
// shape and strides were seen before (a serving loop re-issues the same layers), encoded otherwise.
bool tensor_map(TmapCache* cache, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                const cuuint64_t* strides_bytes, const cuuint32_t* box)
{
    TmapKey key;
    memset(&key, 0, sizeof key);
    key.base = base;
    key.rank = (uint32_t)rank;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides_bytes[i];
    if (cache) {
        std::lock_guard<std::mutex> lock(cache->mu);
        for (const auto& e : cache->entries)
            if (memcmp(&e.first, &key, sizeof key) == 0) { *map = e.second; return true; }
    }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes, box, ones,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (cache) {
        std::lock_guard<std::mutex> lock(cache->mu);
        if (cache->entries.size() < TmapCache::kEntries) cache->entries.emplace_back(key, *map);
        else { cache->entries[cache->next] = std::make_pair(key, *map); cache->next = (cache->next + 1) % TmapCache::kEntries; }
    }
    return true;
}

std::atomic<unsigned int> g_launch_counter{1};
}  // namespace
unsigned int prefill_tc_launch_id();
namespace {

template <int NS>
cudaError_t launch_t(const KernelArgs& a, const HeadCfg& hc, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     int pairs, cudaStream_t st)
{
    const unsigned int launch_id = prefill_tc_launch_id();
    prefill_tc_kernel<NS><<<dim3(a.Hq, pairs), kThreads, kSmemBytes, st>>>(a, hc, launch_id, mq, mk, mv);
    return cudaGetLastError();
}

template <int NS>
cudaError_t configure_one()
{
    return cudaFuncSetAttribute(prefill_tc_kernel<NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

}  // namespace

void* tmap_cache_create() { return new TmapCache; }
void tmap_cache_destroy(void* cache) { delete static_cast<TmapCache*>(cache); }

// Self-test of the bounded waits: one CTA waits on an mbarrier that nothing ever arrives at.  The
// wait must run out after `limit_ns`, the kernel must report HOOK_ATTN_ERR_TIMEOUT through the status
// word and return normally, leaving the context usable.
__global__ void wait_selftest_kernel(int32_t* status, uint64_t limit_ns, uint64_t* waited_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const uint64_t t0 = global_timer_ns();
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar), 0, nullptr, limit_ns));
    if (threadIdx.x == 0) {
        if (!ok) report(status, HOOK_ATTN_ERR_TIMEOUT);
        if (waited_ns) *waited_ns = global_timer_ns() - t0;
    }
}

cudaError_t launch_wait_selftest(int32_t* status, uint64_t limit_ns, uint64_t* waited_ns, cudaStream_t st)
{
    wait_selftest_kernel<<<1, 32, 0, st>>>(status, limit_ns, waited_ns);
    return cudaGetLastError();
}

cudaError_t configure_prefill_tc()
{
    cudaError_t e;
    if ((e = configure_one<0>()) != cudaSuccess) return e;
    return configure_one<kMaxSpans>();
}

// True when the tensor-core kernel can serve the call (head_dim 128, tensor maps encodable).
bool prefill_tc_supported(const KernelArgs& a, int head_dim)
{
    return head_dim == kHD && a.total_q >= kBM && a.num_blocks > 0 && encode_fn() != nullptr &&
           a.bs < (1ll << 38) && a.ts < (1ll << 38) && a.hs < (1ll << 38);
}

// The three TMA descriptors of a call (q: 3-D, k/v: 4-D over [d][kv head][slot][block] with the caller's strides).
bool prefill_tc_maps(const KernelArgs& a, void* tmap_cache, CUtensorMap* mq, CUtensorMap* mk, CUtensorMap* mv)
{
    TmapCache* cache = static_cast<TmapCache*>(tmap_cache);
    {
        const cuuint64_t dims[3] = {(cuuint64_t)kHD, (cuuint64_t)a.Hq, (cuuint64_t)a.total_q};
        const cuuint64_t strides[2] = {(cuuint64_t)kHD * 2, (cuuint64_t)a.Hq * kHD * 2};
        const cuuint32_t box[3] = {64, 1, (cuuint32_t)kBM};
        if (!tensor_map(cache, mq, a.q, 3, dims, strides, box)) return false;
    }
    const cuuint64_t dims[4] = {(cuuint64_t)kHD, (cuuint64_t)a.Hkv, (cuuint64_t)kPage, (cuuint64_t)a.num_blocks};
    const cuuint64_t strides[3] = {(cuuint64_t)a.hs * 2, (cuuint64_t)a.ts * 2, (cuuint64_t)a.bs * 2};
    const cuuint32_t box[4] = {64, 1, (cuuint32_t)kPage, 1};
    return tensor_map(cache, mk, a.k, 4, dims, strides, box) && tensor_map(cache, mv, a.v, 4, dims, strides, box);
}

// Pairs of query tiles of a call: sum over sequences of ceil(n_s / 256) <= floor(total_q / 256) + num_seqs.
int prefill_tc_pairs(const KernelArgs& a) { return a.total_q / (2 * kBM) + a.num_seqs; }

unsigned int prefill_tc_launch_id() { return g_launch_counter.fetch_add(1, std::memory_order_relaxed); }

cudaError_t launch_prefill_tc(const KernelArgs& a, const HeadCfg& hc, void* tmap_cache, int num_sms, cudaStream_t st)
{
    (void)num_sms;
    CUtensorMap mq, mk, mv;
    if (!prefill_tc_maps(a, tmap_cache, &mq, &mk, &mv)) return cudaErrorInvalidValue;
    const int pairs = prefill_tc_pairs(a);
    // two instantiations: without a probe, and with one (any number of spans: the span sums live in shared memory)
    return a.any_probe ? launch_t<kMaxSpans>(a, hc, mq, mk, mv, pairs, st) : launch_t<0>(a, hc, mq, mk, mv, pairs, st);
}

}  // namespace hook_attn
