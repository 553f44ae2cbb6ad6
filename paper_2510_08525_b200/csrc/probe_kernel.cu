// Measurement aid of librlkv: how fast this GPU delivers a read-only stream from HBM into shared memory
// with the mechanism the decode kernel's producer uses (bulk asynchronous copies completing on
// mbarriers, a ring of stages per SM, one persistent CTA per SM), with nobody consuming the data.
// The decode kernel cannot be faster than this on the bytes it must read, so the benchmark reports it
// beside the copy bandwidth (which moves every byte twice: one read, one write).
#include "rlkv_host.cuh"

namespace rlkv {
namespace {

constexpr int kProbeStages = 6;
constexpr int kProbeChunk = 32 * 1024;  // bytes per copy: a K tile and a V tile of head_dim 128

__device__ int g_probe_status;  // 0, or 1 when a wait ran out

__device__ __forceinline__ uint32_t probe_smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// One thread per CTA streams chunks blockIdx.x, blockIdx.x + gridDim.x, ... of `src` through the ring.
__global__ void __launch_bounds__(32, 1) read_stream_kernel(const unsigned char* src, long long n_chunks)
{
    extern __shared__ __align__(1024) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[kProbeStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kProbeStages; ++s)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(probe_smem_u32(bars + s)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    auto issue = [&](long long chunk, int s) {
        const uint32_t bar = probe_smem_u32(bars + s);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kProbeChunk) : "memory");
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
                probe_smem_u32(ring + (size_t)s * kProbeChunk)),
            "l"(src + chunk * kProbeChunk), "r"(kProbeChunk), "r"(bar), "l"(policy)
            : "memory");
    };
    long long next = blockIdx.x;
    int in_flight = 0;
    for (; in_flight < kProbeStages && next < n_chunks; ++in_flight, next += gridDim.x) issue(next, in_flight);
    // waits for the copy into stage s (about one second at most)
    auto landed = [&](int s, uint32_t parity) -> bool {
        const uint32_t bar = probe_smem_u32(bars + s);
        unsigned long long t0 = 0;
        for (uint32_t i = 0;; ++i) {
            uint32_t ok;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(ok)
                : "r"(bar), "r"(parity)
                : "memory");
            if (ok) return true;
            if (i < 1024) continue;
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > 1000000000ull) return false;
        }
    };
    int s = 0;
    uint32_t parity = 0;
    while (in_flight > 0) {
        if (!landed(s, parity)) {
            // record it, give the copies still in flight one more bounded wait each so that none lands
            // in shared memory after the CTA has retired, and leave
            atomicExch(&g_probe_status, 1);
            for (int j = 0; j < in_flight; ++j) {
                landed(s, parity);
                if (++s == kProbeStages) {
                    s = 0;
                    parity ^= 1u;
                }
            }
            return;
        }
        --in_flight;
        if (next < n_chunks) {
            issue(next, s);
            next += gridDim.x;
            ++in_flight;
        }
        if (++s == kProbeStages) {
            s = 0;
            parity ^= 1u;
        }
    }
}

// A stand-in for what a model runs between two attention calls (projections, MLP): it streams `n16`
// 16-byte pieces from src to dst -- work that depends on nothing, like the weights a GEMM reads --,
// then waits for the kernel before it (when launched to overlap), reads a word of `after` (the
// attention output it would consume) and copies `produce_n16` pieces to `produce` (the next call's q,
// k or v), so that those arrive at the very end of the kernel.
__global__ void __launch_bounds__(256) standin_kernel(uint4* dst, const uint4* src, size_t n16, const float* after,
                                                       uint4* produce, const uint4* produce_src, size_t produce_n16,
                                                       int overlap, float* sink)
{
    if (overlap) grid_dep_launch();
    const size_t stride = (size_t)gridDim.x * blockDim.x, first = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (size_t i = first; i < n16; i += stride) dst[i] = __ldcs(src + i);
    if (overlap) grid_dep_wait();
    if (after && first == 0) *sink = *reinterpret_cast<const volatile float*>(after);
    for (size_t i = first; i < produce_n16; i += stride) produce[i] = produce_src[i];
}

__device__ float g_standin_sink;

}  // namespace
}  // namespace rlkv

using namespace rlkv;

extern "C" int rlkv_debug_standin(void* dst, const void* src, size_t bytes, const void* after, void* produce,
                                  const void* produce_src, size_t produce_bytes, int overlap, void* stream)
{
    if ((bytes && (!dst || !src)) || (produce_bytes && (!produce || !produce_src)) || bytes % 16 || produce_bytes % 16 ||
        !aligned16(dst) || !aligned16(src) || !aligned16(produce) || !aligned16(produce_src))
        return RLKV_EINVAL;
    float* sink = nullptr;
    RLKV_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&sink), g_standin_sink));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(148 * 8);
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    RLKV_CUDA(cudaLaunchKernelEx(&cfg, standin_kernel, static_cast<uint4*>(dst), static_cast<const uint4*>(src), bytes / 16,
                                 static_cast<const float*>(after), static_cast<uint4*>(produce),
                                 static_cast<const uint4*>(produce_src), produce_bytes / 16, overlap ? 1 : 0, sink));
    return RLKV_OK;
}

extern "C" int rlkv_debug_read_bandwidth(const void* device_buf, size_t bytes, int launches, float* ms_out)
{
    if (!device_buf || !ms_out || launches < 1 || bytes < (size_t)kProbeChunk || !aligned16(device_buf)) return RLKV_EINVAL;
    int device = 0, sms = 0;
    RLKV_CUDA(cudaGetDevice(&device));
    RLKV_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    const size_t smem = (size_t)kProbeStages * kProbeChunk;
    RLKV_CUDA(cudaFuncSetAttribute(read_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int zero = 0;
    RLKV_CUDA(cudaMemcpyToSymbol(g_probe_status, &zero, sizeof zero));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    RLKV_CUDA(cudaEventCreate(&e0));
    cudaError_t e = cudaEventCreate(&e1);
    if (e != cudaSuccess) {
        cudaEventDestroy(e0);
        return cuda_fail(e, "cudaEventCreate");
    }
    const long long n_chunks = (long long)(bytes / kProbeChunk);
    read_stream_kernel<<<sms, 32, smem>>>(static_cast<const unsigned char*>(device_buf), n_chunks);  // warm-up
    cudaEventRecord(e0);
    for (int i = 0; i < launches; ++i)
        read_stream_kernel<<<sms, 32, smem>>>(static_cast<const unsigned char*>(device_buf), n_chunks);
    cudaEventRecord(e1);
    e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) e = cudaGetLastError();
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return cuda_fail(e, "read_stream_kernel");
    int status = 0;
    RLKV_CUDA(cudaMemcpyFromSymbol(&status, g_probe_status, sizeof status));
    if (status != 0) return RLKV_EKERNEL;
    *ms_out = ms / launches;
    return RLKV_OK;
}
