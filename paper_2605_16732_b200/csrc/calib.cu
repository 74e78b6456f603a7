// Calibration of the NVFP4 activations' per-tensor power-of-two scale (paper Sec. 5.1 / App. E: blocks of 16 with an
// FP8 scale each; the second-level scale of the format is taken as 2^e with e = ceil(log2(max|X| / (6 * 256))), so that
// the largest block scale lands in (128, 256] of E4M3's range).  Offline, outside the timed path: the largest
// low-precision coefficient of a batch of calibration tokens is found on the device and turned into e on the host.
//   * dense rotation: from the fp32 rotated activations that dirotq_rotate_quantize exports;
//   * projection form: x~_h = bf16(x U_hb), x~_l = (x H+- - x~_h V) / 8 with V = bf16(U_hb^T H+-) and H+- the +-1
//     Hadamard blocks of 64, from x and U_h alone (no layer exists yet: the exponent is an argument of the layer's
//     preparation).
#include "common.h"

#include <math.h>
#include <string.h>

namespace dirotq {
namespace {

__device__ __forceinline__ float bf16_round_f32(float v) {  // nearest even
    uint32_t u = __float_as_uint(v);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return __uint_as_float(u & 0xFFFF0000u);
}

__device__ __forceinline__ float load_uh_bf16(const void* Uh, int dtype, size_t idx) {
    // U_hb = bf16(U_h); the fp64 value goes through a single rounding (round to odd into fp32 first)
    if (dtype == DIROTQ_DTYPE_F64) {
        const double v = static_cast<const double*>(Uh)[idx];
        float f = __double2float_rz(v);
        uint32_t u = __float_as_uint(f);
        if (static_cast<double>(f) != v) u |= 1u;
        return bf16_round_f32(__uint_as_float(u));
    }
    return bf16_round_f32(static_cast<const float*>(Uh)[idx]);
}

__device__ __forceinline__ void block_max_to(unsigned int* out, float v, float* red) {
    // non-negative floats order like their bit patterns
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = 0.f;
        for (int w = 0; w < (blockDim.x + 31) / 32; ++w) m = fmaxf(m, red[w]);
        atomicMax(out, __float_as_uint(m));
    }
}

// max |xrot[m][c]| over c >= r
__global__ void __launch_bounds__(256) absmax_low_kernel(const float* xrot, int M, int K, int r, unsigned int* out) {
    __shared__ float red[8];
    const int m = blockIdx.x;
    float v = 0.f;
    for (int c = r + threadIdx.x; c < K; c += blockDim.x) v = fmaxf(v, fabsf(xrot[static_cast<size_t>(m) * K + c]));
    block_max_to(out, v, red);
}

// V[i][k] = bf16(sum_j (-1)^popc(j & c) U_hb[64 b + j][i]) for k = 64 b + c, as fp32 (the sum is exact in fp64)
__global__ void __launch_bounds__(128) projection_v_kernel(const void* Uh, int uh_dtype, int K, int r, float* V) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    const int b = k / 64, c = k % 64;
    for (int i = 0; i < r; ++i) {
        double acc = 0.0;
        for (int j = 0; j < 64; ++j) {
            const double u = static_cast<double>(load_uh_bf16(Uh, uh_dtype, static_cast<size_t>(64 * b + j) * r + i));
            acc += (__popc(j & c) & 1) ? -u : u;
        }
        float f = __double2float_rz(acc);  // one rounding into bf16: round to odd into fp32 first
        uint32_t u = __float_as_uint(f);
        if (static_cast<double>(f) != acc) u |= 1u;
        V[static_cast<size_t>(i) * K + k] = bf16_round_f32(__uint_as_float(u));
    }
}

// One CTA per token row.  Dynamic shared memory: K floats (x H+-, then the residual) after r floats (x~_h).
__global__ void __launch_bounds__(256) residual_absmax_kernel(const uint16_t* x, int M, int K, int r, const void* Uh, int uh_dtype,
                                                              const float* V, unsigned int* out) {
    extern __shared__ float sm[];
    __shared__ float red[8];
    float* xh = sm;       // [r]
    float* d = sm + r;    // [K]
    const int m = blockIdx.x;
    const uint16_t* xr = x + static_cast<size_t>(m) * K;
    for (int i = threadIdx.x; i < r; i += blockDim.x) {
        float acc = 0.f;
        for (int k = 0; k < K; ++k)
            acc = fmaf(__uint_as_float(static_cast<uint32_t>(xr[k]) << 16), load_uh_bf16(Uh, uh_dtype, static_cast<size_t>(k) * r + i), acc);
        xh[i] = bf16_round_f32(acc);
    }
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x) d[k] = __uint_as_float(static_cast<uint32_t>(xr[k]) << 16);
    __syncthreads();
    // x H+-, Hadamard blocks of 64: six butterfly stages in place
    for (int h = 1; h < 64; h <<= 1) {
        for (int p = threadIdx.x; p < K / 2; p += blockDim.x) {
            const int blk = p / 32, q = p % 32;              // pair q of block blk
            const int j = (q / h) * 2 * h + (q % h);         // lower index of the pair at this stage
            float* b = d + blk * 64;
            const float a0 = b[j], a1 = b[j + h];
            b[j] = a0 + a1;
            b[j + h] = a0 - a1;
        }
        __syncthreads();
    }
    float v = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        float acc = 0.f;
        for (int i = 0; i < r; ++i) acc = fmaf(xh[i], V[static_cast<size_t>(i) * K + k], acc);
        v = fmaxf(v, fabsf(d[k] - acc) * 0.125f);
    }
    block_max_to(out, v, red);
}

dirotq_status_t finish(unsigned int* device_word, cudaStream_t s, int* act_scale_log2) {
    unsigned int bits = 0;
    cudaError_t e = cudaMemcpyAsync(&bits, device_word, sizeof bits, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return DIROTQ_ERR_CUDA;
    float amax;
    memcpy(&amax, &bits, sizeof amax);
    if (!(amax > 0.f)) { *act_scale_log2 = 0; return DIROTQ_OK; }
    *act_scale_log2 = static_cast<int>(ceil(log2(static_cast<double>(amax) / 1536.0)));
    return DIROTQ_OK;
}

}  // namespace
}  // namespace dirotq

using namespace dirotq;

extern "C" dirotq_status_t dirotq_act_scale_log2_from_rotated(const float* xrot_f32, int M, int K, int r, void* device_word,
                                                             int* act_scale_log2, dirotq_stream_t stream) {
    if (!xrot_f32 || !device_word || !act_scale_log2 || M < 1 || K < 1 || r < 0 || r >= K) return DIROTQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(device_word, 0, 4, s) != cudaSuccess) return DIROTQ_ERR_CUDA;
    absmax_low_kernel<<<M, 256, 0, s>>>(xrot_f32, M, K, r, static_cast<unsigned int*>(device_word));
    if (cudaGetLastError() != cudaSuccess) return DIROTQ_ERR_CUDA;
    return finish(static_cast<unsigned int*>(device_word), s, act_scale_log2);
}

extern "C" dirotq_status_t dirotq_act_scale_log2_ph(const void* x, int M, const void* Uh, int uh_dtype, int K, int r,
                                                   void* scratch, size_t scratch_bytes, int* act_scale_log2,
                                                   dirotq_stream_t stream) {
    if (!x || !Uh || !scratch || !act_scale_log2 || M < 1 || K < 64 || K % 64 != 0 || r < 1 || r >= K)
        return DIROTQ_ERR_INVALID_ARG;
    if (scratch_bytes < 16 + static_cast<size_t>(r) * K * sizeof(float)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    void* device_word = scratch;
    float* V = reinterpret_cast<float*>(static_cast<char*>(scratch) + 16);
    if (uh_dtype != DIROTQ_DTYPE_F64 && uh_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    const size_t smem = static_cast<size_t>(K + r) * sizeof(float);
    if (smem > 200 * 1024) return DIROTQ_ERR_UNSUPPORTED_SHAPE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIROTQ_ERR_CUDA;
    static SmemOptIn<1> opt_in;
    if (!opt_in.ensure(residual_absmax_kernel, 0, dev, 200 * 1024)) return DIROTQ_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(device_word, 0, 4, s) != cudaSuccess) return DIROTQ_ERR_CUDA;
    projection_v_kernel<<<(K + 127) / 128, 128, 0, s>>>(Uh, uh_dtype, K, r, V);
    if (cudaGetLastError() != cudaSuccess) return DIROTQ_ERR_CUDA;
    residual_absmax_kernel<<<M, 256, smem, s>>>(static_cast<const uint16_t*>(x), M, K, r, Uh, uh_dtype, V,
                                                static_cast<unsigned int*>(device_word));
    if (cudaGetLastError() != cudaSuccess) return DIROTQ_ERR_CUDA;
    return finish(static_cast<unsigned int*>(device_word), s, act_scale_log2);
}
