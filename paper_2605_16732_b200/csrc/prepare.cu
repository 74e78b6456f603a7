// Offline part (paper Eq. 5, right factor): fold the rotation into the weight, split at row r,
// quantize the low rows to INT4 per (group, output column) with round-to-nearest, pack, and lay
// everything out the way the two online kernels read it.  Plain CUDA cores, fp64: this runs once
// per layer and is not on the timed path.
//
// Packed weight-code layout, row n of u8 [N][K_lp/2] (K-major): codes are taken 32 at a time
// (16 bytes, four 32-bit words); word j of such a piece holds codes 8*j .. 8*j + 7.  In the grouped INT4
// formats a code is stored as sign + 3-bit magnitude, codes 8j..8j+3 in bits 7, 2..0 of the word's bytes and
// codes 8j+4..8j+7 four bit positions further up (signmag_nibble_bits in common.h), so that the online unpack of a
// word is a mask, a rotate and a mask, and the resulting byte s0000mmm read as E4M3 is q * 2^-9 exactly (see
// w4a4_gemm.cu).  The W4A8 format keeps the nibble u = q + 8 (code 8j + b in the low, 8j + 4 + b in the high nibble
// of byte 4j + b), which its own kernel turns into the int8 value 16 q.
#include "common.h"

#include <cuda_bf16.h>

namespace dirotq {
namespace {

// fp64 -> bf16, nearest, ties to even, with a single rounding: round to odd into fp32 first.
__device__ __forceinline__ uint16_t f64_to_bf16(double v) {
    float f = __double2float_rz(v);
    uint32_t u = __float_as_uint(f);
    if (static_cast<double>(f) != v && (u & 0x7F800000u) != 0x7F800000u) u |= 1u;  // sticky bit
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0;                             // NaN
    u += 0x7FFFu + ((u >> 16) & 1u);
    return static_cast<uint16_t>(u >> 16);
}

__device__ __forceinline__ double bf16_to_f64(uint16_t h) {
    return static_cast<double>(__uint_as_float(static_cast<uint32_t>(h) << 16));
}

__device__ __forceinline__ double load_q(const void* Q, int q_dtype, int K, int k, int j) {
    const size_t i = static_cast<size_t>(k) * K + j;
    return q_dtype == DIROTQ_DTYPE_F64 ? static_cast<const double*>(Q)[i]
                                       : static_cast<double>(static_cast<const float*>(Q)[i]);
}

__device__ __forceinline__ double load_w(const void* W, int w_dtype, int w_layout, int K, int N, int k, int n) {
    const size_t i = w_layout == DIROTQ_LAYOUT_KN ? static_cast<size_t>(k) * N + n : static_cast<size_t>(n) * K + k;
    return w_dtype == DIROTQ_DTYPE_F32 ? static_cast<double>(static_cast<const float*>(W)[i])
                                       : bf16_to_f64(static_cast<const uint16_t*>(W)[i]);
}

// Wt[i][n] = sum_k Q[k][i] * W[k][n]     (64 x 64 output tile, 4 x 4 per thread, fp64)
__global__ void __launch_bounds__(256) fold_kernel(const void* Q, int q_dtype, const void* W, int w_dtype, int w_layout,
                                                   double* Wt, int K, int N) {
    __shared__ double sq[16][64 + 1];
    __shared__ double sw[16][64 + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int i0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    double acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int e = threadIdx.x; e < 16 * 64; e += 256) {
            const int kk = e >> 6, c = e & 63;
            sq[kk][c] = (i0 + c < K) ? load_q(Q, q_dtype, K, k0 + kk, i0 + c) : 0.0;
            sw[kk][c] = (n0 + c < N) ? load_w(W, w_dtype, w_layout, K, N, k0 + kk, n0 + c) : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = sq[kk][ty * 4 + u]; b[u] = sw[kk][tx * 4 + u]; }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
    for (int u = 0; u < 4; ++u)
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * 4 + u, n = n0 + tx * 4 + v;
            if (i < K && n < N) Wt[static_cast<size_t>(i) * N + n] = acc[u][v];
        }
}

__host__ __device__ __forceinline__ int packed_byte_index(int k) {  // byte of code k inside its row
    const int w = k & 31;
    return (k >> 5) * 16 + (w >> 3) * 4 + (w & 3);
}
__host__ __device__ __forceinline__ int packed_is_high(int k) { return (k >> 2) & 1; }

// One thread per (group, output column): Eq. 1 with z = 0, s = bf16(max|w|/7), ties to even.
__global__ void quantize_weights_kernel(const double* Wt, uint8_t* wpacked, float* wscale, uint16_t* wh, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int grp = blockIdx.y;
    if (n >= g.N) return;
    const int j0 = grp * g.G;
    const int len = min(g.G, g.K_l - j0);
    const double* col = Wt + static_cast<size_t>(g.r + j0) * g.N + n;
    double a = 0.0;
    for (int j = 0; j < len; ++j) a = fmax(a, fabs(col[static_cast<size_t>(j) * g.N]));
    const uint16_t sb = (a == 0.0) ? 0 : f64_to_bf16(a / 7.0);
    const double s = bf16_to_f64(sb);
    wscale[wscale_index(g.N, grp, n)] = static_cast<float>(s) * kWScaleFold;  // a power of two times a bf16 value: exact
    uint8_t* row = wpacked + static_cast<size_t>(n) * (g.K_lp / 2);
    int csum = 0;
    for (int jb = 0; jb < g.G; jb += 8) {
        // codes j0+jb .. j0+jb+7 share four bytes
        uint32_t word = 0;
        for (int t = 0; t < 8; ++t) {
            const int j = jb + t;
            int q = 0;
            if (j < len && s != 0.0) {
                double qq = rint(col[static_cast<size_t>(j) * g.N] / s);
                qq = fmin(7.0, fmax(-7.0, qq));
                q = static_cast<int>(qq);
            }
            csum += q;
            word |= signmag_nibble_bits(t, q);
        }
        *reinterpret_cast<uint32_t*>(row + packed_byte_index(j0 + jb)) = word;
    }
    if (g.fmt == 2) {
        // zero-point term of asymmetric activations: d = s_w * sum(q_w) (at most 17 significant bits), stored as three
        // bf16 pieces that add up to it exactly, in the extra columns of the rank-r weight operand
        double rem = s * static_cast<double>(csum);
        uint16_t* ext = wh + static_cast<size_t>(n) * g.r_pad + g.r_pad0;
        for (int piece = 0; piece < 3; ++piece) {
            const uint16_t pb = f64_to_bf16(rem);
            ext[piece * g.n_g + grp] = pb;
            rem -= bf16_to_f64(pb);
        }
    }
}

// Residual weights rounded by the caller (GPTQ or any other offline rounding): codes [K_l][N] int8 and bf16 scales
// [n_g][N] go into the same packed layout as the library's own round-to-nearest codes.
__global__ void pack_codes_kernel(const int8_t* codes, const uint16_t* scales, uint8_t* wpacked, float* wscale,
                                  uint16_t* wh, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int grp = blockIdx.y;
    if (n >= g.N) return;
    const int j0 = grp * g.G;
    const int len = min(g.G, g.K_l - j0);
    const double s = bf16_to_f64(scales[static_cast<size_t>(grp) * g.N + n]);
    wscale[wscale_index(g.N, grp, n)] = static_cast<float>(s) * kWScaleFold;
    const int8_t* col = codes + static_cast<size_t>(j0) * g.N + n;
    uint8_t* row = wpacked + static_cast<size_t>(n) * (g.K_lp / 2);
    int csum = 0;
    for (int jb = 0; jb < g.G; jb += 8) {
        uint32_t word = 0;
        for (int t = 0; t < 8; ++t) {
            const int j = jb + t;
            const int q = j < len ? max(-7, min(7, static_cast<int>(col[static_cast<size_t>(j) * g.N]))) : 0;
            csum += q;
            word |= signmag_nibble_bits(t, q);
        }
        *reinterpret_cast<uint32_t*>(row + packed_byte_index(j0 + jb)) = word;
    }
    if (g.fmt == 2) {
        double rem = s * static_cast<double>(csum);
        uint16_t* ext = wh + static_cast<size_t>(n) * g.r_pad + g.r_pad0;
        for (int piece = 0; piece < 3; ++piece) {
            const uint16_t pb = f64_to_bf16(rem);
            ext[piece * g.n_g + grp] = pb;
            rem -= bf16_to_f64(pb);
        }
    }
}

// wh[n][i] = bf16(Wt[i][n]) for i < r, zero up to r_pad.
__global__ void high_rows_kernel(const double* Wt, uint16_t* wh, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= g.N) return;
    for (int i = 0; i < g.r_pad; ++i)
        wh[static_cast<size_t>(n) * g.r_pad + i] = i < g.r ? f64_to_bf16(Wt[static_cast<size_t>(i) * g.N + n]) : 0;
}

// qt[c'][k] = bf16(Q[k][col(c')]) with the low-precision columns first (tiled transpose).
__global__ void rotation_kernel(const void* Q, int q_dtype, uint16_t* qt, Geometry g) {
    __shared__ uint16_t tile[32][33];
    const int k0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    for (int dy = threadIdx.y; dy < 32; dy += blockDim.y) {
        const int k = k0 + dy, cp = c0 + threadIdx.x;  // read Q[k][col(cp)], coalesced along cp
        if (k < g.K && cp < g.K) {
            const int col = cp < g.K_l ? cp + g.r : cp - g.K_l;
            tile[dy][threadIdx.x] = f64_to_bf16(load_q(Q, q_dtype, g.K, k, col));
        }
    }
    __syncthreads();
    for (int dy = threadIdx.y; dy < 32; dy += blockDim.y) {
        const int cp = c0 + dy, k = k0 + threadIdx.x;
        if (cp < g.K && k < g.K) qt[static_cast<size_t>(cp) * g.K + k] = tile[threadIdx.x][dy];
    }
}

__global__ void bias_kernel(const uint16_t* bias, float* out, int N) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n < N) out[n] = bias ? __uint_as_float(static_cast<uint32_t>(bias[n]) << 16) : 0.f;
}

// ---------------------------------------------------------------- exports (parity checks)

__global__ void export_wcodes_kernel(const uint8_t* wpacked, int8_t* wcodes, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = blockIdx.y;
    if (n >= g.N || j >= g.K_l) return;
    const uint8_t* row = wpacked + static_cast<size_t>(n) * (g.K_lp / 2);
    if (g.fmt == 3) {  // W4A8: nibble = q + 8
        const uint8_t byte = row[packed_byte_index(j)];
        const int nib = packed_is_high(j) ? (byte >> 4) : (byte & 0xF);
        wcodes[static_cast<size_t>(j) * g.N + n] = static_cast<int8_t>(nib - 8);
    } else {           // grouped formats: sign + magnitude, see signmag_nibble_bits
        const uint32_t word = *reinterpret_cast<const uint32_t*>(row + packed_byte_index(j & ~7));
        wcodes[static_cast<size_t>(j) * g.N + n] = static_cast<int8_t>(signmag_nibble_decode(word, j & 7));
    }
}

// Group scales back in plain order as bf16: [rows][N].  `grouped`: stored permuted and times 2^18 (wscale_index).
__global__ void export_wscales_kernel(const float* wscale, uint16_t* out, int rows, int N, bool grouped) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int grp = blockIdx.y;
    if (n >= N || grp >= rows) return;
    const float v = grouped ? wscale[wscale_index(N, grp, n)] * (1.0f / kWScaleFold) : wscale[static_cast<size_t>(grp) * N + n];
    out[static_cast<size_t>(grp) * N + n] = static_cast<uint16_t>(__float_as_uint(v) >> 16);  // values are bf16-exact
}

__global__ void export_wh_kernel(const uint16_t* wh, uint16_t* out, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    if (n < g.N && i < g.r) out[static_cast<size_t>(i) * g.N + n] = wh[static_cast<size_t>(n) * g.r_pad + i];
}

__global__ void export_q_kernel(const uint16_t* qt, uint16_t* out, Geometry g) {
    __shared__ uint16_t tile[32][33];
    const int k0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    for (int dy = threadIdx.y; dy < 32; dy += blockDim.y) {
        const int cp = c0 + dy, k = k0 + threadIdx.x;
        if (cp < g.K && k < g.K) tile[dy][threadIdx.x] = qt[static_cast<size_t>(cp) * g.K + k];
    }
    __syncthreads();
    for (int dy = threadIdx.y; dy < 32; dy += blockDim.y) {
        const int k = k0 + dy, cp = c0 + threadIdx.x;
        if (k < g.K && cp < g.K) {
            const int col = cp < g.K_l ? cp + g.r : cp - g.K_l;
            out[static_cast<size_t>(k) * g.K + col] = tile[threadIdx.x][dy];
        }
    }
}

__global__ void export_workspace_kernel(const int8_t* codes, const float* xscale, const uint16_t* xh_pad, int M, int ldm,
                                        Geometry g, uint16_t* xh, int8_t* codes_out, uint16_t* scales) {
    const int m = blockIdx.y;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < g.K_l; c += gridDim.x * blockDim.x)
        if (codes_out) {
            const int sm = static_cast<uint8_t>(codes[static_cast<size_t>(m) * g.K_lp + c]);  // sign-magnitude byte
            codes_out[static_cast<size_t>(m) * g.K_l + c] =
                kI8Path ? static_cast<int8_t>(sm) : static_cast<int8_t>((sm & 0x80) ? -(sm & 7) : (sm & 7));
        }
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < g.r; i += blockDim.x)
            if (xh) xh[static_cast<size_t>(m) * g.r + i] = xh_pad[static_cast<size_t>(m) * g.r_pad + i];
        for (int gi = threadIdx.x; gi < g.n_g; gi += blockDim.x)
            if (scales)
                scales[static_cast<size_t>(m) * g.n_g + gi] =
                    static_cast<uint16_t>(__float_as_uint(xscale[static_cast<size_t>(gi) * ldm + m]) >> 16);
    }
}

// fmt 2: codes are plain bytes 0..15; the zero-points sit in the extra columns of x~_h.
__global__ void export_workspace_asym_kernel(const uint8_t* codes, const float* xscale, const uint16_t* xh_pad, int M, int ldm,
                                             Geometry g, uint16_t* xh, uint8_t* codes_out, uint16_t* scales, uint16_t* zeros) {
    const int m = blockIdx.y;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < g.K_l; c += gridDim.x * blockDim.x)
        if (codes_out) codes_out[static_cast<size_t>(m) * g.K_l + c] = codes[static_cast<size_t>(m) * g.K_lp + c];
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < g.r; i += blockDim.x)
            if (xh) xh[static_cast<size_t>(m) * g.r + i] = xh_pad[static_cast<size_t>(m) * g.r_pad + i];
        for (int gi = threadIdx.x; gi < g.n_g; gi += blockDim.x) {
            if (scales)
                scales[static_cast<size_t>(m) * g.n_g + gi] =
                    static_cast<uint16_t>(__float_as_uint(xscale[static_cast<size_t>(gi) * ldm + m]) >> 16);
            if (zeros) zeros[static_cast<size_t>(m) * g.n_g + gi] = xh_pad[static_cast<size_t>(m) * g.r_pad + g.r_pad0 + gi];
        }
    }
}

__global__ void export_zero_term_kernel(const uint16_t* wh, float* d, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int grp = blockIdx.y;
    if (n >= g.N) return;
    const uint16_t* ext = wh + static_cast<size_t>(n) * g.r_pad + g.r_pad0;
    double v = 0.0;
    for (int piece = 2; piece >= 0; --piece) v += bf16_to_f64(ext[piece * g.n_g + grp]);
    d[static_cast<size_t>(grp) * g.N + n] = static_cast<float>(v);  // 17 significant bits: exact
}

// Debug entry of the group GEMM: two's-complement codes [M][K_lp] -> the sign-magnitude bytes the kernel reads, and
// unit scales (one thread per token and group).
__global__ void debug_codes_kernel(const int8_t* in, uint8_t* out, float* xscale, int M, int ldm, Geometry g) {
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    const int grp = blockIdx.y;
    if (m >= M) return;
    for (int j = 0; j < g.G; ++j) {
        const size_t idx = static_cast<size_t>(m) * g.K_lp + grp * g.G + j;
        const int q = in[idx];
        out[idx] = kI8Path ? static_cast<uint8_t>(q) : static_cast<uint8_t>((q < 0 ? 0x80 : 0) | (q < 0 ? -q : q));
    }
    xscale[static_cast<size_t>(grp) * ldm + m] = 1.0f;
}

// ================================================================ W4A8 (paper Sec. 5.1: per-channel 4-bit weights, per-token 8-bit activations)

// One thread per output column: Eq. 1 with z = 0 over the whole column (one scale per channel), codes packed like
// the grouped format (nibble = q + 8).
__global__ void w4a8_quantize_weights_kernel(const double* Wt, uint8_t* wpacked, float* wscale, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= g.N) return;
    const double* col = Wt + static_cast<size_t>(g.r) * g.N + n;
    double a = 0.0;
    for (int j = 0; j < g.K_l; ++j) a = fmax(a, fabs(col[static_cast<size_t>(j) * g.N]));
    const uint16_t sb = (a == 0.0) ? 0 : f64_to_bf16(a / 7.0);
    const double s = bf16_to_f64(sb);
    wscale[n] = static_cast<float>(s);
    uint8_t* row = wpacked + static_cast<size_t>(n) * (g.K_lp / 2);
    for (int jb = 0; jb < g.K_lp; jb += 8) {
        uint32_t word = 0;
        for (int t = 0; t < 8; ++t) {
            const int j = jb + t;
            int q = 0;
            if (j < g.K_l && s != 0.0) {
                double qq = rint(col[static_cast<size_t>(j) * g.N] / s);
                qq = fmin(7.0, fmax(-7.0, qq));
                q = static_cast<int>(qq);
            }
            word |= (static_cast<uint32_t>(q + 8) & 0xFu) << (8 * (t & 3) + 4 * (t >> 2));
        }
        *reinterpret_cast<uint32_t*>(row + packed_byte_index(jb)) = word;
    }
}

// Second pass of the W4A8 activation side, one warp per token: s = bf16(max|x~| / 127), q = clip(rint(x~ / s), -127, 127).
__global__ void a8_quantize_kernel(const float* xtilde, const unsigned int* rowmax, int8_t* codes, float* xscale, int M,
                                   Geometry g) {
    const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= M) return;
    const float amax = __uint_as_float(rowmax[m]);
    const float s = amax > 0.f ? __bfloat162float(__float2bfloat16_rn(__fdiv_rn(amax, 127.0f))) : 0.f;
    const bool slow = !(s >= 1e-30f);
    const float inv = slow ? 0.f : __frcp_rn(s);
    if (lane == 0) xscale[m] = s;
    const float* xr = xtilde + static_cast<size_t>(m) * g.K_lp;
    int8_t* cr = codes + static_cast<size_t>(m) * g.K_lp;
    // four independent 16-byte loads in flight per thread (a warp covers 2 KB of its row per step): with one load per
    // step the pass ran at the latency of a load, not at the rate of the memory
    constexpr int UNROLL = 4;
    for (int j0 = lane * 4; j0 < g.K_lp; j0 += 128 * UNROLL) {
        float4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int j = j0 + 128 * u;
            v[u] = j < g.K_l ? __ldcs(reinterpret_cast<const float4*>(xr + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int j = j0 + 128 * u;
            if (j >= g.K_lp) break;
            uint32_t word = 0;
            if (j < g.K_l) {  // K_l is a multiple of 16: the four values are all real or all padding
                const float vv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    float q = slow ? (s != 0.f ? vv[t] / s : 0.f) : vv[t] * inv;
                    q = fminf(fmaxf(q, -127.0f), 127.0f);
                    word |= (static_cast<uint32_t>(__float2int_rn(q)) & 0xFFu) << (8 * t);
                }
            }
            *reinterpret_cast<uint32_t*>(cr + j) = word;
        }
    }
}

__global__ void export_workspace_w4a8_kernel(const int8_t* codes, const float* xscale, const uint16_t* xh_pad, int M, Geometry g,
                                             uint16_t* xh, int8_t* codes_out, uint16_t* scales) {
    const int m = blockIdx.y;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < g.K_l; c += gridDim.x * blockDim.x)
        if (codes_out) codes_out[static_cast<size_t>(m) * g.K_l + c] = codes[static_cast<size_t>(m) * g.K_lp + c];
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < g.r; i += blockDim.x)
            if (xh) xh[static_cast<size_t>(m) * g.r + i] = xh_pad[static_cast<size_t>(m) * g.r_pad + i];
        if (threadIdx.x == 0 && scales) scales[m] = static_cast<uint16_t>(__float_as_uint(xscale[m]) >> 16);
    }
}

// ================================================================ NVFP4 variant (paper Sec. 5.1)
// E2M1 elements, blocks of 16 along K with an E4M3 scale, one power-of-two scale per tensor.
// Everything offline is done in fp64 so that codes and scales equal the CPU checker's.

// Non-negative fp64 -> E4M3 byte: nearest, ties to even, saturating at 448, subnormals kept.
__device__ __forceinline__ uint8_t f64_to_e4m3(double v) {
    if (!(v > 0.0)) return 0;
    if (v >= 448.0) return 0x7E;
    int e = ilogb(v);
    if (e < -6) e = -6;
    const double quantum = ldexp(1.0, e - 3);
    const double r = rint(v / quantum) * quantum;
    if (r >= 448.0) return 0x7E;
    if (r == 0.0) return 0;
    const int er = ilogb(r);
    if (er < -6) return static_cast<uint8_t>(static_cast<int>(r * 512.0));
    const int mant = static_cast<int>((r / ldexp(1.0, er) - 1.0) * 8.0);
    return static_cast<uint8_t>(((er + 7) << 3) | mant);
}

__device__ __forceinline__ double e4m3_to_f64(uint8_t b) {
    const int e = (b >> 3) & 0xF, m = b & 7;
    return e == 0 ? ldexp(static_cast<double>(m), -9) : ldexp(1.0 + m / 8.0, e - 7);
}

// fp64 -> E2M1 code (bit 3 = sign): nearest of {0, .5, 1, 1.5, 2, 3, 4, 6}, ties to the even code, saturating.
__device__ __forceinline__ uint8_t f64_to_e2m1(double t) {
    const double vals[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};
    const double a = fabs(t);
    int best = 0;
    double bd = a;
    for (int c = 1; c < 8; ++c) {
        const double d = fabs(a - vals[c]);
        if (d < bd || (d == bd && (c & 1) == 0)) { bd = d; best = c; }
    }
    return static_cast<uint8_t>((t < 0.0 ? 8 : 0) | best);
}

struct Nvfp4Meta {
    float out_scale;  // 2^(ex + ew): what the accumulator is multiplied by in the epilogue
    int ew;           // exponent of the weights' per-tensor scale
    int ex;           // exponent of the activations' per-tensor scale (argument of prepare)
    int pad;
    unsigned long long amax_bits;  // fp64 bit pattern of max |W~_l|
};

__global__ void nvfp4_amax_kernel(const double* Wt, Geometry g, Nvfp4Meta* meta) {
    double a = 0.0;
    const size_t lo = static_cast<size_t>(g.r) * g.N, hi = static_cast<size_t>(g.r + g.K_l) * g.N;  // the low rows of the scratch
    for (size_t i = lo + blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < hi;
         i += static_cast<size_t>(gridDim.x) * blockDim.x)
        a = fmax(a, fabs(Wt[i]));
    for (int o = 16; o > 0; o >>= 1) a = fmax(a, __shfl_xor_sync(0xffffffffu, a, o));
    if ((threadIdx.x & 31) == 0) atomicMax(&meta->amax_bits, static_cast<unsigned long long>(__double_as_longlong(a)));
}

__global__ void nvfp4_meta_kernel(Nvfp4Meta* meta, int ex) {
    const double amax = __longlong_as_double(static_cast<long long>(meta->amax_bits));
    int ew = 0;
    if (amax > 0.0) {
        // ceil(log2(amax / 1536)) without a logarithm: x = m 2^e, m in [0.5, 1)
        int e;
        const double m = frexp(amax / (6.0 * 256.0), &e);
        ew = (m == 0.5) ? e - 1 : e;
    }
    meta->ew = ew;
    meta->ex = ex;
    meta->out_scale = static_cast<float>(ldexp(1.0, ex + ew));
}

// One thread per (output column n, 64-element slab kb): four blocks of 16.
__global__ void nvfp4_quantize_weights_kernel(const double* Wt, uint8_t* wcodes, uint8_t* wsf, const Nvfp4Meta* meta,
                                              Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int kb = blockIdx.y;
    if (n >= g.N) return;
    const int ew = meta->ew;
    uint32_t sfword = 0;
    uint8_t* crow = wcodes + static_cast<size_t>(n) * (g.K4 / 2) + kb * 32;
    for (int b = 0; b < 4; ++b) {
        const int j0 = kb * 64 + b * 16;
        const int len = min(16, g.K_l - j0);
        uint8_t codes[16];
        uint8_t sb = 0;
        if (len > 0) {
            const double* col = Wt + static_cast<size_t>(g.r + j0) * g.N + n;
            double a = 0.0;
            for (int j = 0; j < len; ++j) a = fmax(a, fabs(col[static_cast<size_t>(j) * g.N]));
            sb = f64_to_e4m3(ldexp(a / 6.0, -ew));
            const double s = ldexp(e4m3_to_f64(sb), ew);
            for (int j = 0; j < 16; ++j)
                codes[j] = (j < len && s != 0.0) ? f64_to_e2m1(col[static_cast<size_t>(j) * g.N] / s) : 0;
        } else {
            for (int j = 0; j < 16; ++j) codes[j] = 0;
        }
        sfword |= static_cast<uint32_t>(sb) << (8 * b);
        for (int j = 0; j < 16; j += 2) crow[b * 8 + j / 2] = static_cast<uint8_t>(codes[j] | (codes[j + 1] << 4));
    }
    const int nr = n & 127;
    *reinterpret_cast<uint32_t*>(wsf + wsf_atom_offset(n >> 7, kb, g.nkb64p) + (nr & 31) * 16 + (nr >> 5) * 4) = sfword;
}

// wh[n][i] = bf16(Wt[i][n]) * 2^-(ex+ew)  (exact: a power of two), zero padded to r_pad.
__global__ void nvfp4_high_rows_kernel(const double* Wt, uint16_t* wh, const Nvfp4Meta* meta, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= g.N) return;
    const int sh = meta->ex + meta->ew;
    for (int i = 0; i < g.r_pad; ++i) {
        uint16_t out = 0;
        if (i < g.r) out = f64_to_bf16(ldexp(bf16_to_f64(f64_to_bf16(Wt[static_cast<size_t>(i) * g.N + n])), -sh));
        wh[static_cast<size_t>(n) * g.r_pad + i] = out;
    }
}

__global__ void nvfp4_export_weights_kernel(const uint8_t* wcodes, const uint8_t* wsf, const uint16_t* wh, const Nvfp4Meta* meta,
                                            Geometry g, uint8_t* codes_out, uint8_t* sf_out, uint16_t* wh_out, int* ew_out) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = blockIdx.y;  // low-precision row
    if (n == 0 && j == 0 && ew_out) *ew_out = meta->ew;
    if (n >= g.N) return;
    if (j < g.K_l && codes_out) {
        const uint8_t byte = wcodes[static_cast<size_t>(n) * (g.K4 / 2) + j / 2];
        codes_out[static_cast<size_t>(j) * g.N + n] = (j & 1) ? (byte >> 4) : (byte & 0xF);
    }
    const int nb = (g.K_l + 15) / 16;
    if (j < nb && sf_out) {
        const int nr = n & 127;
        sf_out[static_cast<size_t>(j) * g.N + n] =
            wsf[wsf_atom_offset(n >> 7, j >> 2, g.nkb64p) + (nr & 31) * 16 + (nr >> 5) * 4 + (j & 3)];
    }
    if (j < g.r && wh_out)
        wh_out[static_cast<size_t>(j) * g.N + n] =
            f64_to_bf16(ldexp(bf16_to_f64(wh[static_cast<size_t>(n) * g.r_pad + j]), meta->ex + meta->ew));
}

__global__ void nvfp4_export_workspace_kernel(const uint8_t* codes, const uint8_t* xsf, const uint16_t* xh_pad, int M, Geometry g,
                                              uint16_t* xh, uint8_t* codes_out, uint8_t* sf_out) {
    const int m = blockIdx.y;
    const int nb = (g.K_l + 15) / 16;
    for (int c = blockIdx.x * blockDim.x + threadIdx.x; c < g.K_l; c += gridDim.x * blockDim.x) {
        if (codes_out) {
            const uint8_t byte = codes[static_cast<size_t>(m) * (g.K4 / 2) + c / 2];
            codes_out[static_cast<size_t>(m) * g.K_l + c] = (c & 1) ? (byte >> 4) : (byte & 0xF);
        }
    }
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < g.r; i += blockDim.x)
            if (xh) xh[static_cast<size_t>(m) * g.r + i] = xh_pad[static_cast<size_t>(m) * g.r_pad + i];
        const int mr = m & 127;
        for (int b = threadIdx.x; b < nb; b += blockDim.x)
            if (sf_out)
                sf_out[static_cast<size_t>(m) * nb + b] =
                    xsf[(static_cast<size_t>(m >> 7) * g.nkb64p + (b >> 2)) * 512 + (mr & 31) * 16 + (mr >> 5) * 4 + (b & 3)];
    }
}

inline bool launch_ok() { return cudaGetLastError() == cudaSuccess; }

}  // namespace

dirotq_status_t launch_prepare(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                               int q_dtype, const void* bias, const int8_t* wcodes, const void* wscales, double* scratch,
                               cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    fold_kernel<<<dim3((g.N + 63) / 64, (g.K + 63) / 64), 256, 0, stream>>>(Q, q_dtype, W, w_dtype, w_layout, scratch,
                                                                          g.K, g.N);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    // zero the packed codes first: slots of a ragged last group stay zero
    if (cudaMemsetAsync(blob + L->lay.off_wpacked, 0, static_cast<size_t>(g.N) * (g.K_lp / 2), stream) != cudaSuccess)
        return DIROTQ_ERR_CUDA;
    // the rank-r rows first (zero padded to r_pad), then the quantizer, which for fmt 2 fills its extra columns
    high_rows_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(scratch, reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    if (wcodes)
        pack_codes_kernel<<<dim3((g.N + 127) / 128, g.n_g), 128, 0, stream>>>(
            wcodes, static_cast<const uint16_t*>(wscales), reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked),
            reinterpret_cast<float*>(blob + L->lay.off_wscale), reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    else
        quantize_weights_kernel<<<dim3((g.N + 127) / 128, g.n_g), 128, 0, stream>>>(
            scratch, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked),
            reinterpret_cast<float*>(blob + L->lay.off_wscale), reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    if (!g.no_rot) {
        rotation_kernel<<<dim3((g.K + 31) / 32, (g.K + 31) / 32), dim3(32, 8), 0, stream>>>(
            Q, q_dtype, reinterpret_cast<uint16_t*>(blob + L->lay.off_qt), g);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    bias_kernel<<<(g.N + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t*>(bias),
                                                       reinterpret_cast<float*>(blob + L->lay.off_bias), g.N);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

// Replaces the residual codes and scales of a prepared grouped-INT4 layer (codes int8 [K_l][N], bf16 scales [n_g][N], device).
dirotq_status_t launch_pack_codes(const dirotq_layer* L, const int8_t* wcodes, const uint16_t* wscales, cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    if (cudaMemsetAsync(blob + L->lay.off_wpacked, 0, static_cast<size_t>(g.N) * (g.K_lp / 2), stream) != cudaSuccess)
        return DIROTQ_ERR_CUDA;
    pack_codes_kernel<<<dim3((g.N + 127) / 128, g.n_g), 128, 0, stream>>>(
        wcodes, wscales, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<float*>(blob + L->lay.off_wscale),
        reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

// ------------------------------------------------------------------ projection form (fmt 4)

namespace {

__device__ __forceinline__ double load_uh(const void* Uh, int dtype, int r, int k, int i) {
    const size_t e = static_cast<size_t>(k) * r + i;
    return dtype == DIROTQ_DTYPE_F64 ? static_cast<const double*>(Uh)[e] : static_cast<double>(static_cast<const float*>(Uh)[e]);
}

// uht[i][k] = bf16(Uh[k][i]) = U_hb^T, zero for i >= r
__global__ void ph_round_uh_kernel(const void* Uh, int dtype, uint16_t* uht, Geometry g) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= g.K) return;
    for (int i = 0; i < g.r_pad; ++i)
        uht[static_cast<size_t>(i) * g.K + k] = i < g.r ? f64_to_bf16(load_uh(Uh, dtype, g.r, k, i)) : 0;
}

// V = bf16(U_hb^T H+-): V[i][b hg + c] = bf16(sum_j (-1)^popc(j & c) U_hb[b hg + j][i]) (an exact fp64 sum of bf16 values,
// rounded once).  Stored negated and transposed, negvt[k][i] = -V[i][k], the B operand of the online residual's
// projection term; zero for i >= r.  hg: order of the Hadamard blocks.
__global__ void ph_v_kernel(const uint16_t* uht, uint16_t* negvt, int hg, Geometry g) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= g.K) return;
    const int b = k / hg, c = k % hg;
    for (int i = 0; i < g.r_pad; ++i) {
        uint16_t out = 0;
        if (i < g.r) {
            double acc = 0.0;
            for (int j = 0; j < hg; ++j) {
                const double u = bf16_to_f64(uht[static_cast<size_t>(i) * g.K + b * hg + j]);
                acc += (__popc(j & c) & 1) ? -u : u;
            }
            out = f64_to_bf16(-acc);
        }
        negvt[static_cast<size_t>(k) * g.r_pad + i] = out;
    }
}

// had[c][j] = (-1)^popc(c & j) as bf16
__global__ void ph_hadamard_kernel(uint16_t* had, int hg) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= hg * hg) return;
    had[idx] = (__popc((idx / hg) & (idx % hg)) & 1) ? 0xBF80 : 0x3F80;
}

// Wt[i][n] = sum_k back[k][i] W[k][n] for i < r, with back = H+- V^T / hg, i.e. back[b hg + j][i] =
// (1 / hg) sum_c (-1)^popc(j & c) V[i][b hg + c] (exact in fp64): the weight the 16-bit coefficients multiply.
// One CTA per (128 output columns, i); a block's hg values of `back` are shared through shared memory.
__global__ void __launch_bounds__(128) ph_fold_high_kernel(const uint16_t* negvt, const void* W, int w_dtype, int w_layout,
                                                           double* Wt, int hg, Geometry g) {
    __shared__ double back[128];
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    double acc = 0.0;
    for (int b = 0; b < g.K / hg; ++b) {
        __syncthreads();
        for (int j = threadIdx.x; j < hg; j += blockDim.x) {
            double t = 0.0;
            for (int c = 0; c < hg; ++c) {
                const double v = -bf16_to_f64(negvt[static_cast<size_t>(b * hg + c) * g.r_pad + i]);
                t += (__popc(j & c) & 1) ? -v : v;
            }
            back[j] = t / static_cast<double>(hg);
        }
        __syncthreads();
        if (n < g.N)
            for (int j = 0; j < hg; ++j) acc = fma(back[j], load_w(W, w_dtype, w_layout, g.K, g.N, b * hg + j, n), acc);
    }
    if (n < g.N) Wt[static_cast<size_t>(i) * g.N + n] = acc;
}

// Wt[r + b G + i][n] = (1 / sqrt(G)) sum_j (-1)^popc(i & j) W[b G + j][n]: the block Hadamard applied to the rows of W
__global__ void ph_fold_low_kernel(const void* W, int w_dtype, int w_layout, double* Wt, Geometry g) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    const int row = blockIdx.y;  // 0 .. K-1
    if (n >= g.N) return;
    const int b = row / g.G, i = row % g.G;
    double acc = 0.0;
    for (int j = 0; j < g.G; ++j) {
        const double w = load_w(W, w_dtype, w_layout, g.K, g.N, b * g.G + j, n);
        acc += (__popc(i & j) & 1) ? -w : w;
    }
    Wt[static_cast<size_t>(g.r + row) * g.N + n] = acc / sqrt(static_cast<double>(g.G));
}

// out_uh[k][i] = U_hb[k][i] (K x r) and/or out_v[i][k] = V[i][k] (r x K)
__global__ void ph_export_uh_kernel(const uint16_t* uht, const uint16_t* negvt, uint16_t* out_uh, uint16_t* out_v, Geometry g) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= g.K) return;
    for (int i = 0; i < g.r; ++i) {
        if (out_uh) out_uh[static_cast<size_t>(k) * g.r + i] = uht[static_cast<size_t>(i) * g.K + k];
        if (out_v) {
            const uint16_t nv = negvt[static_cast<size_t>(k) * g.r_pad + i];
            out_v[static_cast<size_t>(i) * g.K + k] = (nv & 0x7FFF) ? (nv ^ 0x8000) : 0;
        }
    }
}

}  // namespace

dirotq_status_t launch_prepare_ph(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                  const void* bias, double* scratch, cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    uint16_t* uht = reinterpret_cast<uint16_t*>(blob + L->lay.off_qt);
    uint16_t* negvt = reinterpret_cast<uint16_t*>(blob + L->lay.off_uh);
    const int hg = g.fmt == 1 ? 64 : g.G;  // order of the Hadamard blocks
    ph_round_uh_kernel<<<(g.K + 127) / 128, 128, 0, stream>>>(Uh, uh_dtype, uht, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_v_kernel<<<(g.K + 127) / 128, 128, 0, stream>>>(uht, negvt, hg, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_hadamard_kernel<<<(hg * hg + 255) / 256, 256, 0, stream>>>(reinterpret_cast<uint16_t*>(blob + L->lay.off_had), hg);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_fold_high_kernel<<<dim3((g.N + 127) / 128, g.r), 128, 0, stream>>>(negvt, W, w_dtype, w_layout, scratch, hg, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_fold_low_kernel<<<dim3((g.N + 127) / 128, g.K), 128, 0, stream>>>(W, w_dtype, w_layout, scratch, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    if (cudaMemsetAsync(blob + L->lay.off_wpacked, 0, static_cast<size_t>(g.N) * (g.K_lp / 2), stream) != cudaSuccess)
        return DIROTQ_ERR_CUDA;
    // scratch now holds [r + K][N]: the same shape the INT4 pipeline quantizes (rows < r in 16 bits, the rest in groups)
    high_rows_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(scratch, reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    quantize_weights_kernel<<<dim3((g.N + 127) / 128, g.n_g), 128, 0, stream>>>(
        scratch, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<float*>(blob + L->lay.off_wscale),
        reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    bias_kernel<<<(g.N + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t*>(bias),
                                                       reinterpret_cast<float*>(blob + L->lay.off_bias), g.N);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_uh_export(const dirotq_layer* L, uint16_t* uh, uint16_t* v, cudaStream_t stream) {
    const Geometry& g = L->geo;
    ph_export_uh_kernel<<<(g.K + 127) / 128, 128, 0, stream>>>(reinterpret_cast<const uint16_t*>(L->blob + L->lay.off_qt),
                                                              reinterpret_cast<const uint16_t*>(L->blob + L->lay.off_uh), uh, v, g);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_layer_export(const dirotq_layer* L, int8_t* wcodes, uint16_t* wscales, uint16_t* wh,
                                    uint16_t* qb, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const char* blob = L->blob;
    if (wcodes) {
        export_wcodes_kernel<<<dim3((g.N + 127) / 128, g.K_l), 128, 0, stream>>>(
            reinterpret_cast<const uint8_t*>(blob + L->lay.off_wpacked), wcodes, g);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    if (wscales) {
        const int rows = g.fmt == 3 ? 1 : g.n_g;  // W4A8: one scale per output column
        export_wscales_kernel<<<dim3((g.N + 255) / 256, rows), 256, 0, stream>>>(
            reinterpret_cast<const float*>(blob + L->lay.off_wscale), wscales, rows, g.N, g.fmt != 3);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    if (wh) {
        export_wh_kernel<<<dim3((g.N + 127) / 128, g.r), 128, 0, stream>>>(
            reinterpret_cast<const uint16_t*>(blob + L->lay.off_wh), wh, g);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    if (qb) {
        export_q_kernel<<<dim3((g.K + 31) / 32, (g.K + 31) / 32), dim3(32, 8), 0, stream>>>(
            reinterpret_cast<const uint16_t*>(blob + L->lay.off_qt), qb, g);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    return DIROTQ_OK;
}

dirotq_status_t launch_prepare_w4a8(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                                    int q_dtype, const void* bias, double* scratch, cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    fold_kernel<<<dim3((g.N + 63) / 64, (g.K + 63) / 64), 256, 0, stream>>>(Q, q_dtype, W, w_dtype, w_layout, scratch,
                                                                          g.K, g.N);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    high_rows_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(scratch, reinterpret_cast<uint16_t*>(blob + L->lay.off_wh), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    w4a8_quantize_weights_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(
        scratch, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<float*>(blob + L->lay.off_wscale), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    rotation_kernel<<<dim3((g.K + 31) / 32, (g.K + 31) / 32), dim3(32, 8), 0, stream>>>(
        Q, q_dtype, reinterpret_cast<uint16_t*>(blob + L->lay.off_qt), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    bias_kernel<<<(g.N + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t*>(bias),
                                                       reinterpret_cast<float*>(blob + L->lay.off_bias), g.N);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_a8_quantize(const dirotq_layer* L, int M, const float* xtilde, const unsigned int* rowmax, int8_t* codes,
                                   float* xscale, cudaStream_t stream) {
    a8_quantize_kernel<<<(M + 7) / 8, 256, 0, stream>>>(xtilde, rowmax, codes, xscale, M, L->geo);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_workspace_export_w4a8(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh, int8_t* codes,
                                             uint16_t* scales, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const WorkspaceLayoutA8 w = make_workspace_layout_w4a8(g, M);
    export_workspace_w4a8_kernel<<<dim3(8, M), 256, 0, stream>>>(
        reinterpret_cast<const int8_t*>(workspace + w.off_codes), reinterpret_cast<const float*>(workspace + w.off_xscale),
        reinterpret_cast<const uint16_t*>(workspace + w.off_xh), M, g, xh, codes, scales);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_workspace_export_asym(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                             uint8_t* codes, uint16_t* scales, uint16_t* zeros, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const WorkspaceLayout w = make_workspace_layout(g, M);
    export_workspace_asym_kernel<<<dim3(8, M), 256, 0, stream>>>(
        reinterpret_cast<const uint8_t*>(workspace + w.off_codes), reinterpret_cast<const float*>(workspace + w.off_xscale),
        reinterpret_cast<const uint16_t*>(workspace + w.off_xh), M, w.ldm, g, xh, codes, scales, zeros);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_zero_term_export(const dirotq_layer* L, float* d, cudaStream_t stream) {
    const Geometry& g = L->geo;
    export_zero_term_kernel<<<dim3((g.N + 127) / 128, g.n_g), 128, 0, stream>>>(
        reinterpret_cast<const uint16_t*>(L->blob + L->lay.off_wh), d, g);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_debug_codes(const dirotq_layer* L, int M, const int8_t* act_codes, char* workspace,
                                   cudaStream_t stream) {
    const Geometry& g = L->geo;
    const WorkspaceLayout w = make_workspace_layout(g, M);
    debug_codes_kernel<<<dim3((M + 127) / 128, g.n_g), 128, 0, stream>>>(
        act_codes, reinterpret_cast<uint8_t*>(workspace + w.off_codes), reinterpret_cast<float*>(workspace + w.off_xscale), M,
        w.ldm, g);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_workspace_export(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                        int8_t* codes, uint16_t* scales, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const WorkspaceLayout w = make_workspace_layout(g, M);
    export_workspace_kernel<<<dim3(8, M), 256, 0, stream>>>(
        reinterpret_cast<const int8_t*>(workspace + w.off_codes), reinterpret_cast<const float*>(workspace + w.off_xscale),
        reinterpret_cast<const uint16_t*>(workspace + w.off_xh), M, w.ldm, g, xh, codes, scales);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

}  // namespace dirotq

namespace dirotq {

dirotq_status_t launch_prepare_nvfp4(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                                     int q_dtype, const void* bias, double* scratch, cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    Nvfp4Meta* meta = reinterpret_cast<Nvfp4Meta*>(blob + L->lay.off_meta);
    fold_kernel<<<dim3((g.N + 63) / 64, (g.K + 63) / 64), 256, 0, stream>>>(Q, q_dtype, W, w_dtype, w_layout, scratch,
                                                                          g.K, g.N);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    if (cudaMemsetAsync(meta, 0, 64, stream) != cudaSuccess) return DIROTQ_ERR_CUDA;
    if (cudaMemsetAsync(blob + L->lay.off_wscale, 0, wsf_bytes(g.N, g.nkb64p), stream) !=
        cudaSuccess)
        return DIROTQ_ERR_CUDA;
    nvfp4_amax_kernel<<<592, 256, 0, stream>>>(scratch, g, meta);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_meta_kernel<<<1, 1, 0, stream>>>(meta, L->act_scale_log2);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_quantize_weights_kernel<<<dim3((g.N + 127) / 128, g.nkb64), 128, 0, stream>>>(
        scratch, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<uint8_t*>(blob + L->lay.off_wscale),
        meta, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_high_rows_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(scratch, reinterpret_cast<uint16_t*>(blob + L->lay.off_wh),
                                                                  meta, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    rotation_kernel<<<dim3((g.K + 31) / 32, (g.K + 31) / 32), dim3(32, 8), 0, stream>>>(
        Q, q_dtype, reinterpret_cast<uint16_t*>(blob + L->lay.off_qt), g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    bias_kernel<<<(g.N + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t*>(bias),
                                                       reinterpret_cast<float*>(blob + L->lay.off_bias), g.N);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_prepare_nvfp4_ph(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                        const void* bias, double* scratch, cudaStream_t stream) {
    const Geometry& g = L->geo;
    char* blob = L->blob;
    Nvfp4Meta* meta = reinterpret_cast<Nvfp4Meta*>(blob + L->lay.off_meta);
    uint16_t* uht = reinterpret_cast<uint16_t*>(blob + L->lay.off_qt);
    uint16_t* negvt = reinterpret_cast<uint16_t*>(blob + L->lay.off_uh);
    const int hg = g.fmt == 1 ? 64 : g.G;  // order of the Hadamard blocks
    ph_round_uh_kernel<<<(g.K + 127) / 128, 128, 0, stream>>>(Uh, uh_dtype, uht, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_v_kernel<<<(g.K + 127) / 128, 128, 0, stream>>>(uht, negvt, hg, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_hadamard_kernel<<<(hg * hg + 255) / 256, 256, 0, stream>>>(reinterpret_cast<uint16_t*>(blob + L->lay.off_had), hg);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_fold_high_kernel<<<dim3((g.N + 127) / 128, g.r), 128, 0, stream>>>(negvt, W, w_dtype, w_layout, scratch, hg, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    ph_fold_low_kernel<<<dim3((g.N + 127) / 128, g.K), 128, 0, stream>>>(W, w_dtype, w_layout, scratch, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    // the scratch now holds [r + K][N]: quantized exactly like the dense form's folded weight
    if (cudaMemsetAsync(meta, 0, 64, stream) != cudaSuccess) return DIROTQ_ERR_CUDA;
    if (cudaMemsetAsync(blob + L->lay.off_wscale, 0, wsf_bytes(g.N, g.nkb64p), stream) !=
        cudaSuccess)
        return DIROTQ_ERR_CUDA;
    nvfp4_amax_kernel<<<592, 256, 0, stream>>>(scratch, g, meta);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_meta_kernel<<<1, 1, 0, stream>>>(meta, L->act_scale_log2);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_quantize_weights_kernel<<<dim3((g.N + 127) / 128, g.nkb64), 128, 0, stream>>>(
        scratch, reinterpret_cast<uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<uint8_t*>(blob + L->lay.off_wscale),
        meta, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    nvfp4_high_rows_kernel<<<(g.N + 127) / 128, 128, 0, stream>>>(scratch, reinterpret_cast<uint16_t*>(blob + L->lay.off_wh),
                                                                  meta, g);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    bias_kernel<<<(g.N + 255) / 256, 256, 0, stream>>>(static_cast<const uint16_t*>(bias),
                                                       reinterpret_cast<float*>(blob + L->lay.off_bias), g.N);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

dirotq_status_t launch_layer_export_nvfp4(const dirotq_layer* L, uint8_t* wcodes, uint8_t* wsf, uint16_t* wh, uint16_t* qb,
                                          int* ew, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const char* blob = L->blob;
    const int rows = g.K_l > g.r ? g.K_l : g.r;
    nvfp4_export_weights_kernel<<<dim3((g.N + 127) / 128, rows), 128, 0, stream>>>(
        reinterpret_cast<const uint8_t*>(blob + L->lay.off_wpacked), reinterpret_cast<const uint8_t*>(blob + L->lay.off_wscale),
        reinterpret_cast<const uint16_t*>(blob + L->lay.off_wh), reinterpret_cast<const Nvfp4Meta*>(blob + L->lay.off_meta), g,
        wcodes, wsf, wh, ew);
    if (!launch_ok()) return DIROTQ_ERR_CUDA;
    if (qb) {
        export_q_kernel<<<dim3((g.K + 31) / 32, (g.K + 31) / 32), dim3(32, 8), 0, stream>>>(
            reinterpret_cast<const uint16_t*>(blob + L->lay.off_qt), qb, g);
        if (!launch_ok()) return DIROTQ_ERR_CUDA;
    }
    return DIROTQ_OK;
}

dirotq_status_t launch_workspace_export_nvfp4(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                              uint8_t* codes, uint8_t* sf, cudaStream_t stream) {
    const Geometry& g = L->geo;
    const WorkspaceLayout w = make_workspace_layout_nvfp4(g, M);
    nvfp4_export_workspace_kernel<<<dim3(8, M), 256, 0, stream>>>(
        reinterpret_cast<const uint8_t*>(workspace + w.off_codes), reinterpret_cast<const uint8_t*>(workspace + w.off_xscale),
        reinterpret_cast<const uint16_t*>(workspace + w.off_xh), M, g, xh, codes, sf);
    return launch_ok() ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

}  // namespace dirotq
