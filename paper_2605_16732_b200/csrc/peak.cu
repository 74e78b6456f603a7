// Tensor-pipe issue-rate probe: every SM issues back-to-back tcgen05.mma instructions on operands
// that already sit in shared memory (no TMA, no epilogue).  Used by the benchmark to measure the
// dense 8-bit (int8, E4M3) and bf16 MMA rates of the part the roofline fractions are quoted against.
#include "common.h"
#include "ptx.cuh"

namespace dirotq {
namespace {

constexpr int PEAK_THREADS = 128;
constexpr int PEAK_SMEM = 2 * (16384 + 32768) + 1024 + 64;

// kind: 0 = kind::i8 (s8 x s8 -> s32, K = 32 per instruction), 1 = kind::f16 (bf16 -> f32, K = 16),
//       2 = kind::f8f6f4 (E4M3 x E4M3 -> f32, K = 32)
__global__ void __launch_bounds__(PEAK_THREADS, 1) mma_peak_kernel(int kind, int iters, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar = base + 2 * (16384 + 32768);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + 2 * (16384 + 32768) + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 2 * (16384 + 32768) + 20);
    // operands: zeros are fine for an issue-rate probe
    for (int i = threadIdx.x; i < 2 * (16384 + 32768) / 16; i += PEAK_THREADS)
        reinterpret_cast<uint4*>(gen)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) {
        const uint32_t idesc = kind == 0 ? umma_idesc(2, 1, 128, 256) : (kind == 1 ? umma_idesc(1, 1, 128, 256) : umma_idesc(1, 0, 128, 256));
        for (int i = 0; i < iters; ++i) {
            const uint32_t st = base + (i & 1) * (16384 + 32768);
            const uint64_t adesc = umma_desc_sw128(st);
            const uint64_t bdesc = umma_desc_sw128(st + 16384);
            const uint32_t d = tmem_base + ((i >> 2) & 1) * 256;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (kind == 0) umma_i8(d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
                else if (kind == 1) umma_bf16(d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
                else umma_f8f6f4(d, adesc + 2 * k, bdesc + 2 * k, idesc, 1u);
            }
        }
        umma_commit(bar);
        mbar_wait(bar, 0, abort_flag, status, DEV_TIMEOUT_MMA);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// One warp waits, with the same bounded wait every kernel of the library uses, on a barrier nobody will ever arrive on:
// the wait gives up after `limit_ns`, records its code in the status word and the kernel returns normally.
__global__ void wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, DEV_TIMEOUT_SELFTEST, limit_ns);
    (void)ok;  // false: either this thread's clock ran out or it saw another thread's abort flag
}

}  // namespace
}  // namespace dirotq

using namespace dirotq;

extern "C" dirotq_status_t dirotq_wait_selftest(void* workspace, unsigned int limit_us, dirotq_stream_t stream) {
    if (!workspace || limit_us < 1 || limit_us > 100000) return DIROTQ_ERR_INVALID_ARG;
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int*>(workspace),
                                                                         static_cast<unsigned long long>(limit_us) * 1000ull);
    return cudaGetLastError() == cudaSuccess ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

extern "C" dirotq_status_t dirotq_mma_rate_probe(int kind, int iters, void* status_word, float* tera_ops_per_s,
                                                dirotq_stream_t stream) {
    if (kind < 0 || kind > 2 || iters < 1 || iters > (1 << 20) || !status_word || !tera_ops_per_s)
        return DIROTQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIROTQ_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DIROTQ_ERR_CUDA;
    if (major != 10) return DIROTQ_ERR_ARCH;
    static SmemOptIn<1> opt_in;
    if (!opt_in.ensure(mma_peak_kernel, 0, dev, PEAK_SMEM)) return DIROTQ_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return DIROTQ_ERR_CUDA;
    const int grid = sm_count(dev);
    mma_peak_kernel<<<grid, PEAK_THREADS, PEAK_SMEM, s>>>(kind, iters, static_cast<int*>(status_word));  // warm-up
    cudaEventRecord(e0, s);
    mma_peak_kernel<<<grid, PEAK_THREADS, PEAK_SMEM, s>>>(kind, iters, static_cast<int*>(status_word));
    cudaEventRecord(e1, s);
    cudaError_t e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess || ms <= 0.f) return DIROTQ_ERR_CUDA;
    const double k_per_instr = kind == 1 ? 16.0 : 32.0;
    const double ops = 2.0 * 128.0 * 256.0 * k_per_instr * 4.0 * iters * grid;
    *tera_ops_per_s = static_cast<float>(ops / (ms * 1e-3) / 1e12);
    return DIROTQ_OK;
}
