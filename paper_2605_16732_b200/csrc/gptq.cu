// GPTQ rounding of the residual weight W~_l (paper Sec. 4.1: the rounding minimises ||X W - X W^||^2 on calibration
// tokens; App. "Quantization details": damping 0.01, block size 128), offline, fp64, on CUDA cores.
//
// The steps are those of the published GPTQ algorithm, on the rows of W~_l = (Q^T W)[r:] :
//   X~_l = (x_calib Q_b)[:, low]                          rotated calibration tokens (bf16 inputs, fp64 sums)
//   H    = X~_l^T X~_l ;  dead columns (H_jj = 0) get H_jj = 1 and a zero weight row ;  H += damp * mean(diag H) * I
//   U    = upper-triangular factor of H^-1 = U^T U        (here: H = R R^T with R upper triangular, U = R^-1)
//   for the rows j of W~_l in order, in blocks of `block` rows:
//       at the first row of a group: s = bf16(max |w| / 7) over the group's rows AS THEY STAND (after all feedback so far)
//       q_j = clip(rint(w_j / s), -7, 7) ;  e_j = (w_j - s q_j) / U_jj ;  w_k -= U_jk e_j  for the later rows k of the block
//       after the block: w_k -= sum_{j in block} U_jk e_j  for every row k behind the block
// Every output column evolves on its own, so the row loop runs with one thread per column.  Products and differences
// are rounded separately where the row-by-row definition does so (no fused multiply-add in the feedback of a block), so
// that codes and scales come out equal to a plain fp64 evaluation of the same steps unless a quotient falls within
// rounding error of a tie.
#include "common.h"

namespace dirotq {
namespace {

__device__ __forceinline__ double bf16_bits_to_f64(uint16_t h) {
    return static_cast<double>(__uint_as_float(static_cast<uint32_t>(h) << 16));
}

// fp64 -> bf16 bits, nearest even, single rounding (round to odd into fp32 first)
__device__ __forceinline__ uint16_t f64_to_bf16_bits(double v) {
    float f = __double2float_rz(v);
    uint32_t u = __float_as_uint(f);
    if (static_cast<double>(f) != v && (u & 0x7F800000u) != 0x7F800000u) u |= 1u;
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0;
    u += 0x7FFFu + ((u >> 16) & 1u);
    return static_cast<uint16_t>(u >> 16);
}

// C[i][j] = sum_k A[i][k] B[j][k], A bf16 [I][K], B bf16 [J][K] (both K-contiguous), C fp64 [I][ldc]: the rotation of the
// calibration tokens by the layer's own bf16 rotation (rows of B = rotated columns).  64 x 64 tiles, 4 x 4 per thread.
__global__ void __launch_bounds__(256) gemm_nt_bf16_kernel(const uint16_t* A, const uint16_t* B, double* C, int I, int J, int K,
                                                           int ldc) {
    __shared__ double sa[16][64 + 1];
    __shared__ double sb[16][64 + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    double acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int e = threadIdx.x; e < 16 * 64; e += 256) {
            const int kk = e & 15, c = e >> 4;  // consecutive threads read consecutive k
            sa[kk][c] = (i0 + c < I && k0 + kk < K) ? bf16_bits_to_f64(A[static_cast<size_t>(i0 + c) * K + k0 + kk]) : 0.0;
            sb[kk][c] = (j0 + c < J && k0 + kk < K) ? bf16_bits_to_f64(B[static_cast<size_t>(j0 + c) * K + k0 + kk]) : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = sa[kk][ty * 4 + u]; b[u] = sb[kk][tx * 4 + u]; }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
    for (int u = 0; u < 4; ++u)
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * 4 + u, j = j0 + tx * 4 + v;
            if (i < I && j < J) C[static_cast<size_t>(i) * ldc + j] = acc[u][v];
        }
}

// C[i][j] (= or -=) sum_t A[t][i] B[t][j]   (A fp64 [T][lda], B fp64 [T][ldb], C fp64 [I][ldc]); `subtract` selects -=.
__global__ void __launch_bounds__(256) gemm_tn_f64_kernel(const double* A, int lda, const double* B, int ldb, double* C, int ldc,
                                                          int I, int J, int T, int subtract) {
    __shared__ double sa[16][64 + 1];
    __shared__ double sb[16][64 + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    double acc[4][4] = {};
    for (int t0 = 0; t0 < T; t0 += 16) {
        for (int e = threadIdx.x; e < 16 * 64; e += 256) {
            const int tt = e >> 6, c = e & 63;
            sa[tt][c] = (t0 + tt < T && i0 + c < I) ? A[static_cast<size_t>(t0 + tt) * lda + i0 + c] : 0.0;
            sb[tt][c] = (t0 + tt < T && j0 + c < J) ? B[static_cast<size_t>(t0 + tt) * ldb + j0 + c] : 0.0;
        }
        __syncthreads();
#pragma unroll
        for (int tt = 0; tt < 16; ++tt) {
            double a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { a[u] = sa[tt][ty * 4 + u]; b[u] = sb[tt][tx * 4 + u]; }
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
        }
        __syncthreads();
    }
    for (int u = 0; u < 4; ++u)
        for (int v = 0; v < 4; ++v) {
            const int i = i0 + ty * 4 + u, j = j0 + tx * 4 + v;
            if (i < I && j < J) {
                double* c = C + static_cast<size_t>(i) * ldc + j;
                *c = subtract ? *c - acc[u][v] : acc[u][v];
            }
        }
}

// Dead columns and damping (one CTA): a column no calibration token excites gets H_jj = 1 and a zero weight row; then
// damp * mean(diag H) is added to the diagonal.  dead[j] is kept for the weight rows.
__global__ void __launch_bounds__(1024) damp_kernel(double* H, int n, double damp, unsigned char* dead) {
    __shared__ double part[1024];
    double s = 0.0;
    for (int j = threadIdx.x; j < n; j += blockDim.x) {
        double d = H[static_cast<size_t>(j) * n + j];
        const bool is_dead = d == 0.0;
        dead[j] = is_dead ? 1 : 0;
        if (is_dead) { d = 1.0; H[static_cast<size_t>(j) * n + j] = 1.0; }
        s += d;
    }
    part[threadIdx.x] = s;
    __syncthreads();
    for (int w = blockDim.x / 2; w > 0; w >>= 1) {
        if (threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
        __syncthreads();
    }
    const double add = damp * (part[0] / static_cast<double>(n));
    for (int j = threadIdx.x; j < n; j += blockDim.x) H[static_cast<size_t>(j) * n + j] += add;
}

__global__ void zero_dead_rows_kernel(double* Wlow, int n, int N, const unsigned char* dead) {
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = blockIdx.y;
    if (col < N && j < n && dead[j]) Wlow[static_cast<size_t>(j) * N + col] = 0.0;
}

// H = R R^T with R upper triangular, columns taken from the last to the first (a Cholesky factorisation in reversed
// order), in place in the upper triangle of A (A symmetric; only entries [i][k], i <= k, are read or written).
//   column j:  R_jj = sqrt(A_jj);  R_ij = A_ij / R_jj (i < j);  then  A_ik -= R_ij R_kj  for i <= k < j.
__global__ void ul_column_kernel(double* A, int n, int j) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const double d = sqrt(A[static_cast<size_t>(j) * n + j]);
    if (i < j) A[static_cast<size_t>(i) * n + j] /= d;
    // the diagonal entry is written by the update kernel's first thread, after every reader of A_jj is done
}
__global__ void ul_update_kernel(double* A, int n, int j) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;  // column of the trailing (leading, here) block
    const int i = blockIdx.y;
    if (i == 0 && k == 0) A[static_cast<size_t>(j) * n + j] = sqrt(A[static_cast<size_t>(j) * n + j]);
    if (k < j && i <= k)
        A[static_cast<size_t>(i) * n + k] -= A[static_cast<size_t>(i) * n + j] * A[static_cast<size_t>(k) * n + j];
}

// U = R^-1 (both upper triangular), rows from the last to the first:
//   U_ii = 1 / R_ii ;  U_ij = -(sum_{k = i+1..j} R_ik U_kj) / R_ii  for j > i.
__global__ void upper_inverse_row_kernel(const double* R, double* U, int n, int i) {
    const int j = i + blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const double rii = R[static_cast<size_t>(i) * n + i];
    if (j == i) { U[static_cast<size_t>(i) * n + i] = 1.0 / rii; return; }
    double s = 0.0;
    for (int k = i + 1; k <= j; ++k) s = fma(R[static_cast<size_t>(i) * n + k], U[static_cast<size_t>(k) * n + j], s);
    U[static_cast<size_t>(i) * n + j] = -s / rii;
}

// One block of rows [b0, b1) of the residual weight, one thread per output column.  E[j - b0][col] receives the
// scaled rounding errors the rows behind the block are corrected with.
__global__ void __launch_bounds__(128) gptq_block_kernel(double* W, const double* U, double* E, int8_t* codes, uint16_t* scales,
                                                         int n, int N, int G, int b0, int b1) {
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= N) return;
    double s = 0.0;
    if (b0 % G != 0) s = bf16_bits_to_f64(scales[static_cast<size_t>(b0 / G) * N + col]);  // a group that began in an earlier block
    for (int j = b0; j < b1; ++j) {
        if (j % G == 0) {
            const int g1 = min(j + G, n);
            double a = 0.0;
            for (int k = j; k < g1; ++k) a = fmax(a, fabs(W[static_cast<size_t>(k) * N + col]));
            const uint16_t sb = a == 0.0 ? 0 : f64_to_bf16_bits(a / 7.0);
            scales[static_cast<size_t>(j / G) * N + col] = sb;
            s = bf16_bits_to_f64(sb);
        }
        const double w = W[static_cast<size_t>(j) * N + col];
        double q = 0.0;
        if (s > 0.0) q = fmin(7.0, fmax(-7.0, rint(w / s)));
        codes[static_cast<size_t>(j) * N + col] = static_cast<int8_t>(q);
        const double err = __ddiv_rn(__dsub_rn(w, __dmul_rn(s, q)), U[static_cast<size_t>(j) * n + j]);
        for (int k = j + 1; k < b1; ++k) {
            double* wk = W + static_cast<size_t>(k) * N + col;
            *wk = __dsub_rn(*wk, __dmul_rn(U[static_cast<size_t>(j) * n + k], err));  // product and difference rounded separately
        }
        E[static_cast<size_t>(j - b0) * N + col] = err;
    }
}

inline bool ok_launch() { return cudaGetLastError() == cudaSuccess; }

}  // namespace

size_t gptq_scratch_bytes(int K, int N, int r, int T) {
    const size_t n = static_cast<size_t>(K - r);
    size_t o = 0;
    o += align_up(static_cast<size_t>(K) * N * sizeof(double));  // folded weight
    o += align_up(static_cast<size_t>(T) * n * sizeof(double));  // rotated calibration tokens (low columns)
    o += align_up(n * n * sizeof(double));                       // H, then R
    o += align_up(n * n * sizeof(double));                       // U
    o += align_up(static_cast<size_t>(128) * N * sizeof(double));  // E of one block (block <= 128 rows)
    o += align_up(n * N);                                        // codes
    o += align_up(static_cast<size_t>((n + 63) / 64) * N * 2);   // scales
    o += align_up(n);                                            // dead flags
    return o;
}

// Runs the steps above.  On entry `scratch` holds the folded weight W~ = Q^T W [K][N] (fp64) in its first K*N doubles and
// the layer's blob holds the bf16 rotation; on return *codes_out / *scales_out point at int8 codes [K_l][N] and bf16
// scales [n_g][N] inside `scratch` (device memory; valid in stream order).
dirotq_status_t launch_gptq_round(const dirotq_layer* L, const void* calib_bf16, int T, double damp, int block, char* scratch,
                                  cudaStream_t stream, const int8_t** codes_out, const uint16_t** scales_out) {
    const Geometry& g = L->geo;
    const int n = g.K_l, N = g.N;
    size_t o = 0;
    double* Wt = reinterpret_cast<double*>(scratch + o);      o += align_up(static_cast<size_t>(g.K) * N * sizeof(double));
    double* Xt = reinterpret_cast<double*>(scratch + o);      o += align_up(static_cast<size_t>(T) * n * sizeof(double));
    double* H = reinterpret_cast<double*>(scratch + o);       o += align_up(static_cast<size_t>(n) * n * sizeof(double));
    double* U = reinterpret_cast<double*>(scratch + o);       o += align_up(static_cast<size_t>(n) * n * sizeof(double));
    double* E = reinterpret_cast<double*>(scratch + o);       o += align_up(static_cast<size_t>(128) * N * sizeof(double));
    int8_t* codes = reinterpret_cast<int8_t*>(scratch + o);   o += align_up(static_cast<size_t>(n) * N);
    uint16_t* scales = reinterpret_cast<uint16_t*>(scratch + o); o += align_up(static_cast<size_t>((n + 63) / 64) * N * 2);
    unsigned char* dead = reinterpret_cast<unsigned char*>(scratch + o);
    double* Wlow = Wt + static_cast<size_t>(g.r) * N;
    const uint16_t* qt = reinterpret_cast<const uint16_t*>(L->blob + L->lay.off_qt);  // row c' = rotated column, low ones first

    gemm_nt_bf16_kernel<<<dim3((n + 63) / 64, (T + 63) / 64), 256, 0, stream>>>(static_cast<const uint16_t*>(calib_bf16), qt, Xt,
                                                                                T, n, g.K, n);
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    gemm_tn_f64_kernel<<<dim3((n + 63) / 64, (n + 63) / 64), 256, 0, stream>>>(Xt, n, Xt, n, H, n, n, n, T, 0);
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    damp_kernel<<<1, 1024, 0, stream>>>(H, n, damp, dead);
    zero_dead_rows_kernel<<<dim3((N + 127) / 128, n), 128, 0, stream>>>(Wlow, n, N, dead);
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    for (int j = n - 1; j >= 0; --j) {
        ul_column_kernel<<<(j + 255) / 256 + 1, 256, 0, stream>>>(H, n, j);
        if (j > 0) ul_update_kernel<<<dim3((j + 127) / 128, j), 128, 0, stream>>>(H, n, j);
        else ul_update_kernel<<<dim3(1, 1), 128, 0, stream>>>(H, n, 0);  // only the diagonal entry is left to finish
    }
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    for (int i = n - 1; i >= 0; --i)
        upper_inverse_row_kernel<<<(n - i + 127) / 128, 128, 0, stream>>>(H, U, n, i);
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    for (int b0 = 0; b0 < n; b0 += block) {
        const int b1 = b0 + block < n ? b0 + block : n;
        gptq_block_kernel<<<(N + 127) / 128, 128, 0, stream>>>(Wlow, U, E, codes, scales, n, N, g.G, b0, b1);
        if (b1 < n)
            gemm_tn_f64_kernel<<<dim3((N + 63) / 64, (n - b1 + 63) / 64), 256, 0, stream>>>(
                U + static_cast<size_t>(b0) * n + b1, n, E, N, Wlow + static_cast<size_t>(b1) * N, N, n - b1, N, b1 - b0, 1);
    }
    if (!ok_launch()) return DIROTQ_ERR_CUDA;
    *codes_out = codes;
    *scales_out = scales;
    return DIROTQ_OK;
}

}  // namespace dirotq
