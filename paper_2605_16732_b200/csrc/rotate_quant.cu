// Kernel (a): online rotation, split and activation quantization in one pass.
//
//   x~ = x Q_b                      bf16 x bf16 -> fp32 on tcgen05 (kind::f16), operands by TMA
//   x~_h = bf16(x~[:, high])        the r high-precision coefficients          (paper Sec. 4.2)
//   per token, per group of G low-precision coefficients:                      (paper Eq. 1, z = 0)
//       s = bf16(max|x~| / 7),  q = clip(rint(x~ / s), -7, 7)   stored as a sign-magnitude byte
//
// The rotated activations never reach HBM: the fp32 accumulators are read from tensor memory by
// the epilogue warps, where each thread owns one token row, so the group maximum is a
// thread-local reduction over the row's G values.
//
// Roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer (+ TMEM owner),
// warps 2..9 = epilogue (lane quadrant = warp_id % 4; the two warps of a quadrant take half of the
// tile's column groups each).  Persistent CTAs walk the tile list; two 128x256 fp32 accumulators in
// TMEM let the epilogue of tile i overlap the MMAs of tile i+1.
//
// What bounds it (timing runs with one kind of work switched off, 4608 x 3072 x 3072): the operand stream
// alone takes 0.050 ms (1.0 GB from L2 at 20 TB/s with 4 x 48 KB in flight per SM; 0.056 ms with three
// stages, so the ring depth, i.e. the latency of a loaded L2, sets the rate), with the MMAs 0.064 ms (a
// stage is only refilled once its MMAs have completed, which adds their time to each slot's cycle), with
// the epilogue 0.069 ms (0.074 ms with four epilogue warps).  All 227 KB of shared memory are in use.
#include "common.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>

namespace dirotq {
namespace {

constexpr int BM_MMA = 128;   // token rows of one MMA; a tile has BM = 128 or 256 rows (template parameter)
constexpr int BN_MAX = 256;   // rotated columns per tile: 256, or 128 when there are few tiles (template parameter BN)
constexpr int BK = 64;        // bf16 elements per k-block (128-byte rows)
constexpr int STAGES_WIDE = 4;  // 256-column tiles: 4 x 48 KB; 128-column tiles: 6 x 32 KB (same bytes in flight)
constexpr int A_BYTES_128 = BM_MMA * BK * 2;  // 16 KB per 128 token rows
constexpr int B_BYTES = BN_MAX * BK * 2;  // 32 KB (a 128-column tile uses half of it)
constexpr int STAGE_BYTES_WIDE = A_BYTES_128 + B_BYTES;
constexpr int NUM_THREADS = 320;  // TMA warp, MMA warp, eight epilogue warps
// Behind the ring: 1 KB for the barriers, then one 4 KB staging tile per epilogue warp (32 rows x up to 128 bytes, swizzled),
// from which the activation codes (or the W4A8 path's fp32 coefficients) leave as TMA stores.
constexpr int STORE_OFFSET = STAGES_WIDE * STAGE_BYTES_WIDE + 1024;
constexpr int SMEM_BYTES = STORE_OFFSET + 8 * 4096 + 1024 /*alignment slack*/;
static_assert(SMEM_BYTES <= 232448, "shared memory plan");

struct RotKernelParams {
    int M, K, K_l, K_lp, r, r_pad, r_pad0, ldm, n_g;
    int n_out, k_red;      // output columns and reduction length of the GEMM (both K for the rotation x Q)
    int8_t* codes;
    float* xscale;
    uint16_t* xh;
    float* xrot;
    int* status;
    // NVFP4 variant
    uint8_t* xsf;     // scale-factor atoms [ceil(M/128)][nkb64p][512]
    int K4, nkb64p;   // packed row width in elements; atoms per row block
    int ex;           // exponent of the activations' per-tensor power-of-two scale
    // W4A8 variant: first pass only (the token's scale needs its whole row)
    float* xtilde;          // fp32 [M][K_lp]
    unsigned int* rowmax;   // per-token max |x~_l| as a bit pattern, atomic max (zeroed by the host before the launch)
    // Split reduction (first step of the projection form with few row tiles): the k-blocks are cut into `ksplit` ranges,
    // one tile each, and every range's fp32 accumulators go to partial[range][M][n_out]; nothing else is written.
    int ksplit = 1;
    float* partial = nullptr;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    // byte permute; a selector nibble with bit 3 set replicates the sign bit of the selected byte
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// Quantizes 16 consecutive values, q = clip(rint(pre * v / s), -7, 7), and packs them one code per byte in
// sign-magnitude form (bit 7 = sign, bits 2..0 = |q|): read as E4M3 that byte is q * 2^-9 exactly, which
// is how the second kernel's tensor-core instruction consumes it.
// Common path (SLOW = false): t = v * inv with inv = pre / s.  The scale is bf16(max|pre v| / 7) >= max|pre v| / 7 *
// (1 - 2^-9), so |t| <= 7.02 for finite inputs and rounds to at most 7: no clamp is needed.  |t| + 1.5 * 2^23 leaves
// |q| (nearest, ties to even) in the low byte of the sum's bit pattern; the signs come from the top bytes of t.
// SLOW: the scale is zero or too small for its reciprocal: divide (rare, kept out of the common path's code).
template <bool SLOW>
__device__ __forceinline__ uint4 quantize16(const float* v, float inv, float s, float pre) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if constexpr (SLOW || kI8Path) {
            uint32_t f[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float t = SLOW ? (s != 0.f ? (v[4 * i + j] * pre) / s : 0.f) : v[4 * i + j] * inv;
                t = fminf(fmaxf(t, -7.0f), 7.0f);
                // adding 1.5 * 2^23 rounds to the nearest integer, ties to even, and leaves the two's-complement code
                // in the low byte of the bit pattern
                f[j] = __float_as_uint(t + 12582912.0f);
            }
            const uint32_t tw = __byte_perm(__byte_perm(f[0], f[1], 0x0040), __byte_perm(f[2], f[3], 0x0040), 0x5410);
            const uint32_t sg = (tw >> 7) & 0x01010101u;           // 1 where the code is negative
            const uint32_t mag = (tw ^ (sg * 0xFFu)) + sg;         // |q| per byte (at most 7: no carry between bytes)
            w[i] = kI8Path ? tw : (mag | (tw & 0x80808080u));  // the integer-path build keeps two's complement
        } else {
            uint32_t t[4], m[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float tj = v[4 * i + j] * inv;
                t[j] = __float_as_uint(tj);
                m[j] = __float_as_uint(fabsf(tj) + 12582912.0f);
            }
            const uint32_t mag = prmt(prmt(m[0], m[1], 0x0040u), prmt(m[2], m[3], 0x0040u), 0x5410u);
            const uint32_t sgn = prmt(prmt(t[0], t[1], 0x00FBu), prmt(t[2], t[3], 0x00FBu), 0x5410u);  // 0xFF where t < 0
            w[i] = (sgn & 0x80808080u) | mag;
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Asymmetric variant (Eq. 1 with z = min X): 16 values -> 16 bytes u = clip(rint((v - z) / s), 0, 15); as E4M3 the byte
// 0000uuuu is u * 2^-9 exactly.
template <bool SLOW>
__device__ __forceinline__ uint4 quantize16_asym(const float* v, float z, float inv, float s) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t f[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float d = v[4 * i + j] - z;
            float t = SLOW ? (s != 0.f ? d / s : 0.f) : d * inv;
            t = fminf(fmaxf(t, 0.0f), 15.0f);
            f[j] = __float_as_uint(t + 12582912.0f);  // nearest integer, ties to even, in the low byte
        }
        const uint32_t tw = __byte_perm(__byte_perm(f[0], f[1], 0x0040), __byte_perm(f[2], f[3], 0x0040), 0x5410);
        w[i] = tw;
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// ---- NVFP4 (paper Sec. 5.1): E2M1 elements, blocks of 16, E4M3 block scale relative to 2^ex ----------

// Non-negative float -> E4M3 byte, nearest-even, saturating at 448 (hardware conversion).
__device__ __forceinline__ uint32_t f32_to_e4m3(float v) {
    uint16_t pair;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(0.0f), "f"(v));  // second operand -> low byte
    return pair & 0xFFu;
}

__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
    const uint32_t e = (b >> 3) & 0xFu, m = b & 7u;
    return e == 0 ? static_cast<float>(m) * 0.001953125f : __uint_as_float(((e + 120u) << 23) | (m << 20));
}

// Two floats -> one byte of two E2M1 codes, nearest-even, saturating at 6: `lo` in bits 0..3, `hi` in bits 4..7.
__device__ __forceinline__ uint32_t f32x2_to_e2m1x2(float lo, float hi) {
    uint32_t out;
    asm("{\n\t"
        ".reg .b8 t;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\t"
        "cvt.u32.u8 %0, t;\n\t"
        "}\n"
        : "=r"(out)
        : "f"(hi), "f"(lo));
    return out;
}

// One block of 16 values: returns the E4M3 scale byte and writes the 8 code bytes (two 32-bit words).
// The values quantized are pre * v[j], pre a power of two (so that scaling the maximum and the reciprocal instead of
// every value gives the same bits).
__device__ __forceinline__ uint32_t nvfp4_block16(const float* v, float pre, float ex_inv, float ex_scale, uint32_t& w0, uint32_t& w1) {
    float am[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < 16; ++j) am[j & 3] = fmaxf(am[j & 3], fabsf(v[j]));
    const float amax = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])) * pre;
    const uint32_t sb = f32_to_e4m3(__fdiv_rn(amax, 6.0f) * ex_inv);
    const float s = e4m3_to_f32(sb) * ex_scale;
    const float inv = s > 0.f ? __frcp_rn(s) * pre : 0.f;
    w0 = 0;
    w1 = 0;
#pragma unroll
    for (int j = 0; j < 8; j += 2) {
        w0 |= f32x2_to_e2m1x2(v[j] * inv, v[j + 1] * inv) << (4 * j);
        w1 |= f32x2_to_e2m1x2(v[8 + j] * inv, v[9 + j] * inv) << (4 * j);
    }
    return sb;
}

// PH: second step of the projection form (FMT 4 is PH with the INT4 quantizer of FMT 0).  The accumulator of a tile is
//     x H+- - x~_h V  =  [x~_h | x] [-V ; H+-]
// built from k_red / 64 k-blocks of x~_h (tmap_x) against -V^T (tmap_qt) over all BN columns, followed, for every group of
// G columns under the tile, by G / 64 k-blocks of that group's columns of x (tmap_x2) against the +-1 Hadamard block
// (tmap_had) into the group's own column slice of the accumulator (MMAs with N = G).  The epilogue scales by
// 1 / sqrt(G) and quantizes.  Without PH the last two tensor maps are not used.  (Cutting the projection term into
// per-group k-blocks too, for a ring of eight 24 KB stages that holds a whole tile ahead of the MMAs, measured slower:
// 87 against 79 us for the whole first stage at M = 4608, K = 12288.)
// EPI_WARPS: 8, or 16 for the PH mode with groups of 64 (four warps per lane quadrant, one 64-column chunk each): that
// mode has no long main loop to hide the epilogue under, and its epilogue is a chain of dependent instructions per
// thread that only more warps per scheduler speed up.
// PAIR: launched as clusters of two CTAs that share every MMA (tcgen05.mma.cta_group::2, M = 256): a pair owns 256
// token rows x BN columns, each CTA loads its own 128 rows of x and HALF of the rotation tile (BN / 2 rows of Q^T), so a
// third fewer operand bytes travel from L2 per flop than with 128 x 256 tiles, and both accumulator buffers stay free
// for overlapping the epilogue (which the single-CTA 256 x 256 plan gives up).  The even CTA (rank 0) issues the MMAs
// and owns the "stage full" and "accumulator drained" barriers both CTAs' loads and epilogue warps report to; completion
// of the MMAs is signalled to both CTAs' "stage empty" / "accumulator full" barriers.
template <int G, int FMT, int BN, int BM, bool PH = (FMT == 4), int EPI_WARPS = 8, bool PAIR = false>
__global__ void __launch_bounds__(64 + 32 * EPI_WARPS, 1)
rotate_quant_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_qt,
                    const __grid_constant__ CUtensorMap tmap_x2, const __grid_constant__ CUtensorMap tmap_had,
                    const __grid_constant__ CUtensorMap tmap_out, const RotKernelParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // The ring holds 192 KB either way; with narrow tiles it is cut into more, smaller stages: the operand stream is
    // paced by (L2 latency + MMA time of a stage) / number of stages.
    // A 256 x 256 tile (two MMAs of 128 rows on one Qt tile: a third fewer operand bytes per flop) takes three 64 KB
    // stages and all 512 tensor-memory columns, so its epilogue does not overlap the next tile's MMAs; it is used
    // where a tile's main loop is long and there are many tiles per SM.
    static_assert(BM == 128 || (BM == 256 && BN == 256), "256-row tiles are 256 columns wide");
    constexpr int A_BYTES = BM * BK * 2;
    static_assert(!PAIR || (BM == 128 && BN == 256 && !PH), "pairs: 128 rows per CTA, 256 columns per pair");
    constexpr int B_ROWS = PAIR ? BN / 2 : BN;  // rows of the rotation tile this CTA holds
    static_assert(BN >= G, "a tile holds whole groups");
    // 64-column tiles (few token rows) put TWO k-blocks into a stage: there the kernel is paced by the producer's and the MMA
    // issuer's chains of single-thread instructions per stage (wait, expect, loads; wait, fence, MMAs, commit), so fewer, larger
    // stages shorten it (the split reduction of the projection form's first step never runs with this plan)
    constexpr int KSUB = BN == 64 ? 2 : 1;
    constexpr int SUB_BYTES = A_BYTES + B_ROWS * BK * 2;  // one k-block's operands: [x tile | rotation tile]
    constexpr int STAGES = BM == 256 ? 3 : (B_ROWS == 256 ? STAGES_WIDE : B_ROWS == 128 ? 6 : 4);
    constexpr int STAGE_BYTES = KSUB * SUB_BYTES;
    constexpr int ACC_BUFS = BM == 256 ? 1 : 2;
    static_assert(STAGES * STAGE_BYTES == STAGES_WIDE * STAGE_BYTES_WIDE && STAGE_BYTES % 1024 == 0, "ring layout");
    const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
    // barrier map (8 bytes each): full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2] (at most 20 of them); the
    // tensor-memory slot, the abort flag and the spare barrier follow at +192, +196 and +200
    static_assert(8 * (2 * STAGES + 4) <= 192, "barriers end below the words at +192");
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + STAGES * STAGE_BYTES + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + STAGES * STAGE_BYTES + 196);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Trace build (TRACE_CLK): slot 9 entry, 10 set-up done, 11 previous grid ended, 12 producer has filled the ring once, 13 producer has
    // issued everything, 14 / 15 MMA warp sees the first / ninth stage, 16 MMA warp has committed its last tile, 17 first epilogue
    // warp sees its first accumulator, 18 that warp has finished its last tile.
    if (threadIdx.x == 0) TRACE_CLK(p.status, 9);

    const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
    constexpr int TILE_ROWS = PAIR ? 2 * BM : BM;  // token rows of a tile (of the pair's tile)
    const int tile_first = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int tile_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    const int num_m_blocks = (p.M + TILE_ROWS - 1) / TILE_ROWS;
    const int num_n_blocks = (p.n_out + BN - 1) / BN;
    const int num_mn = num_m_blocks * num_n_blocks;
    const int num_tiles = num_mn * p.ksplit;
    const int num_kb = p.k_red / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), EPI_WARPS * 32 * (PAIR ? 2 : 1));  // every thread of the epilogue warps (of both CTAs) arrives
        }
        mbar_init(bar_base + 200u, 1);  // spare: see umma_drain
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_qt);
        tma_prefetch_desc(&tmap_out);
        if constexpr (PH) {
            tma_prefetch_desc(&tmap_x2);
            tma_prefetch_desc(&tmap_had);
        }
    }
    if (warp == 1) {
        if constexpr (PAIR) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
            tmem_relinquish();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();  // the other CTA's barriers are initialised before anything arrives on them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) TRACE_CLK(p.status, 10);
    grid_dependency_wait();
    if (threadIdx.x == 0) TRACE_CLK(p.status, 11);
    // the second kernel of the layer may be scheduled onto SMs as this grid's CTAs leave them (it waits for the whole
    // grid before it reads anything)
    grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // The whole warp walks the loops and waits; one elected lane issues.  Loop counters, addresses and coordinates
        // then stay warp-uniform, which shortens the chain of instructions per stage (337 against 475 cycles per stage
        // measured with 18 SMs busy, where that chain paces the kernel).
        {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step) {
                const int mn = PH ? num_mn - 1 - tile : tile % num_mn, sp = tile / num_mn;
                const int m0 = (mn % num_m_blocks) * TILE_ROWS + static_cast<int>(cta_rank) * BM * (PAIR ? 1 : 0);
                const int n0 = (mn / num_m_blocks) * BN;
                if constexpr (PH) {
                    const int nv = num_kb;                            // k-blocks of the projection term
                    const int nx = min(BN, p.n_out - n0) / BK;        // 64-column pieces of x under this tile
                    for (int i = 0; i < nv + nx; ++i, ++it) {
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1;
                        if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                        const uint32_t sa = smem_base + s * STAGE_BYTES;
                        if (!elect_one()) continue;
                        if (i < nv) {
                            mbar_arrive_expect_tx(full_bar(s), A_BYTES + BN * BK * 2);
                            tma_load_2d(sa, &tmap_x, full_bar(s), i * BK, m0);
                            tma_load_2d(sa + A_BYTES, &tmap_qt, full_bar(s), i * BK, n0);
                        } else {
                            const int j = i - nv;
                            mbar_arrive_expect_tx(full_bar(s), A_BYTES + G * BK * 2);
                            tma_load_2d(sa, &tmap_x2, full_bar(s), n0 + j * BK, m0);
                            tma_load_2d(sa + A_BYTES, &tmap_had, full_bar(s), (j % (G / BK)) * BK, 0);
                        }
                    }
                    continue;
                }
                // a split reduction is dealt out k-block by k-block: range sp takes k-blocks sp, sp + ksplit, ... (measured the
                // same as contiguous ranges)
                for (int kb = sp; kb < num_kb; kb += p.ksplit * KSUB, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * STAGE_BYTES;
                    if (!elect_one()) continue;
                    if constexpr (KSUB > 1) {
                        const int nsub = min(KSUB, num_kb - kb);  // k-blocks in this stage
                        mbar_arrive_expect_tx(full_bar(s), nsub * SUB_BYTES);
                        for (int j = 0; j < nsub; ++j) {
                            tma_load_2d(sa + j * SUB_BYTES, &tmap_x, full_bar(s), (kb + j) * BK, m0);
                            tma_load_2d(sa + j * SUB_BYTES + A_BYTES, &tmap_qt, full_bar(s), (kb + j) * BK, n0);
                        }
                        if (it == STAGES - 1) TRACE_CLK(p.status, 12);
                        continue;
                    }
                    if constexpr (PAIR) {
                        // both CTAs' bytes are counted on the leader's barrier, which expects the sum
                        const uint32_t full_leader = map_to_cta(full_bar(s), 0);
                        if (cta_rank == 0) mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);
                        tma_load_2d_pair(sa, &tmap_x, full_leader, kb * BK, m0);
                        tma_load_2d_pair(sa + A_BYTES, &tmap_qt, full_leader, kb * BK, n0 + static_cast<int>(cta_rank) * B_ROWS);
                    } else {
                        mbar_arrive_expect_tx(full_bar(s), A_BYTES + BN * BK * 2);
                        tma_load_2d(sa, &tmap_x, full_bar(s), kb * BK, m0);
                        tma_load_2d(sa + A_BYTES, &tmap_qt, full_bar(s), kb * BK, n0);
                    }
                    if (it == STAGES - 1) TRACE_CLK(p.status, 12);
                }
            }
            if (lane == 0) TRACE_CLK(p.status, 13);
            if (lane != 0) {
                // one lane looks after the loads in flight
            } else if (!ok && PAIR && cta_rank != 0) {
                // this CTA's loads report to the leader's barriers: give them a fixed time instead
                const unsigned long long t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 1000000ull) {}
            } else if (!ok) {
                // leave no bulk copy in flight: wait (bounded) for the loads already issued
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1) &&
                           globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp in the loops, one lane issues)
        if (cta_rank == 0) {
            constexpr uint32_t idesc = umma_idesc(1 /*f32*/, 1 /*bf16*/, PAIR ? 2 * BM_MMA : BM_MMA, BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step, ++tcount) {
                const uint32_t acc = tcount % ACC_BUFS;
                const uint32_t acc_ph = (tcount / ACC_BUFS) & 1;
                if (!mbar_wait(tempty_bar(acc), acc_ph ^ 1, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem_base + acc * BN;
                if constexpr (PH) {
                    constexpr uint32_t idesc_g = umma_idesc(1 /*f32*/, 1 /*bf16*/, BM_MMA, G);
                    const int n0 = ((num_mn - 1 - tile) / num_m_blocks) * BN;
                    const int nv = num_kb, nx = min(BN, p.n_out - n0) / BK;
                    for (int i = 0; i < nv + nx; ++i, ++it) {
                        const int s = it % STAGES;
                        const uint32_t ph = (it / STAGES) & 1;
                        if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t sa = smem_base + s * STAGE_BYTES;
                        const uint64_t adesc = umma_desc_sw128(sa);
                        const uint64_t bdesc = umma_desc_sw128(sa + A_BYTES);
                        if (!elect_one()) continue;
                        if (i < nv) {
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k) umma_bf16(d, adesc + 2 * k, bdesc + 2 * k, idesc, (i | k) != 0);
                        } else {
                            const uint32_t dg = d + ((i - nv) / (G / BK)) * G;  // the group's columns of the accumulator
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k) umma_bf16(dg, adesc + 2 * k, bdesc + 2 * k, idesc_g, 1);
                        }
                        umma_commit(empty_bar(s));
                    }
                    if (ok && elect_one()) umma_commit(tfull_bar(acc));
                    continue;
                }
                const int sp = tile / num_mn;
                const int kb_begin = sp;
                for (int kb = kb_begin; kb < num_kb; kb += p.ksplit * KSUB, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + s * STAGE_BYTES;
                    const uint64_t adesc = umma_desc_sw128(sa);
                    const uint64_t bdesc = umma_desc_sw128(sa + A_BYTES);
                    if (!elect_one()) continue;
                    if (it == 0) TRACE_CLK(p.status, 14);
                    if (it == 8) TRACE_CLK(p.status, 15);
                    if constexpr (KSUB > 1) {
                        const int nsub = min(KSUB, num_kb - kb);
                        for (int j = 0; j < nsub; ++j) {
#pragma unroll
                            for (int k = 0; k < BK / 16; ++k)
                                umma_bf16(d, adesc + j * (SUB_BYTES >> 4) + 2 * k, bdesc + j * (SUB_BYTES >> 4) + 2 * k, idesc,
                                          kb != kb_begin || j != 0 || k != 0);
                        }
                        umma_commit(empty_bar(s));
                        continue;
                    }
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        if constexpr (PAIR) {
                            umma_bf16_pair(d, adesc + 2 * k, bdesc + 2 * k, idesc, kb != kb_begin || k != 0);
                        } else {
                            umma_bf16(d, adesc + 2 * k, bdesc + 2 * k, idesc, kb != kb_begin || k != 0);
                            if constexpr (BM == 256)  // token rows 128..255: next 16 KB of the x tile, columns 256..511 of TMEM
                                umma_bf16(d + 256, adesc + (A_BYTES_128 >> 4) + 2 * k, bdesc + 2 * k, idesc, kb != kb_begin || k != 0);
                        }
                    }
                    if constexpr (PAIR) umma_commit_pair(empty_bar(s), 3);  // both CTAs' producers may refill the stage
                    else umma_commit(empty_bar(s));
                }
                if (ok && elect_one()) {
                    if constexpr (PAIR) umma_commit_pair(tfull_bar(acc), 3);  // both CTAs' epilogue warps
                    else umma_commit(tfull_bar(acc));
                    TRACE_CLK(p.status, 16);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        // two warps per quadrant: with 128-row tiles they share the tile's column chunks, with 256-row tiles each
        // takes all chunks of one 128-row block
        const int half = (warp - 2) >> 2;
        constexpr int EPI_Q = EPI_WARPS / 4;  // warps per lane quadrant
        static_assert(EPI_WARPS == 8 || (EPI_WARPS == 16 && BM == 128 && BN / G >= 4), "epilogue warp plan");
        constexpr int CHUNKS = BN / G, CPH = BM == 256 ? CHUNKS : (CHUNKS >= EPI_Q ? CHUNKS / EPI_Q : 1);
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step, ++tcount) {
            // PH: the tiles are walked from the last columns to the first, i.e. starting with the part of x that the step
            // before this one read last and that is most likely still in L2
            const int mn = PH ? num_mn - 1 - tile : tile % num_mn;
            const int m0 = (mn % num_m_blocks) * TILE_ROWS + static_cast<int>(cta_rank) * BM * (PAIR ? 1 : 0);
            const int n_blk = mn / num_m_blocks;
            const int n0 = n_blk * BN;
            const uint32_t acc = tcount % ACC_BUFS;
            const uint32_t acc_ph = (tcount / ACC_BUFS) & 1;
            const int row = m0 + (BM == 256 ? half * 128 : 0) + q * 32 + lane;
            const bool row_ok = row < p.M;
            // A thread holds one token row, so direct stores of its codes would be 16-byte pieces of 32 different rows per
            // instruction (in the NVFP4 second kernel a clock trace showed such stores taking thousands of cycles per tile
            // and halving the rate of the operand loads).  The INT4 codes (one byte each: G bytes per row and chunk) and the
            // W4A8 path's fp32 coefficients (128 bytes per row at a time) go into the warp's staging tile instead, swizzled
            // so that a quarter-warp's pieces fall into different banks, and one lane hands the tile to a TMA store
            // (tmap_out), which writes whole sectors and clips at M and at the row's width.
            constexpr bool STAGED = EPI_WARPS == 8;
            const uint32_t sbuf = smem_base + STORE_OFFSET + static_cast<uint32_t>(warp - 2) * 4096u;
            const int row0w = row - lane;  // the warp's first row
            auto stage_piece128 = [&](int piece, uint4 val) {  // rows of 128 bytes, 128-byte swizzle
                const uint32_t dst = sbuf + static_cast<uint32_t>(lane) * 128u + (static_cast<uint32_t>(piece ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
            };
            auto stage_code_piece = [&](int piece, uint4 val) {  // G one-byte codes per row: 64-byte rows (64-byte swizzle) or 128
                if constexpr (G == 64) {
                    const uint32_t dst = sbuf + static_cast<uint32_t>(lane) * 64u + (static_cast<uint32_t>(piece ^ ((lane >> 1) & 3)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
                } else {
                    stage_piece128(piece, val);
                }
            };
            if (!mbar_wait(tfull_bar(acc), acc_ph, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE)) { ok = false; break; }
            if (warp == 2 && lane == 0 && tcount == 0) TRACE_CLK(p.status, 17);
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + (BM == 256 ? half * 256 : acc * BN);

            float tile_amax = 0.f;  // W4A8: this thread's row, this tile's columns
#pragma unroll 1
            for (int chunk = (BM == 256 ? 0 : half * CPH); chunk < min(CHUNKS, (BM == 256 ? 1 : half + 1) * CPH); ++chunk) {
                const int col0 = n0 + chunk * G;  // permuted column of v[0]
                if (col0 >= p.n_out) break;
                float v[G];
#pragma unroll
                for (int c = 0; c < G / 32; ++c) {
                    uint32_t raw[32];
                    tmem_ld_32x32b_x32(taddr + chunk * G + c * 32, raw);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[c * 32 + j] = __uint_as_float(raw[j]);
                }
                if (p.partial != nullptr) {
                    // split reduction: this range's accumulators, as they are
                    if (row_ok) {
                        float4* dst = reinterpret_cast<float4*>(
                            p.partial + (static_cast<size_t>(tile / num_mn) * p.M + row) * p.n_out + col0);
#pragma unroll
                        for (int j = 0; j < G / 4; ++j)
                            if (col0 + 4 * j < p.n_out) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    }
                    continue;
                }
                if (p.xrot != nullptr && row_ok) {
#pragma unroll
                    for (int b = 0; b < G / 16; ++b) {
                        const int pc = col0 + 16 * b;
                        const int oc = pc < p.K_l ? pc + p.r : pc - p.K_l;  // caller's column order
                        float4* dst = reinterpret_cast<float4*>(p.xrot + static_cast<size_t>(row) * p.K + oc);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dst[j] = make_float4(v[16 * b + 4 * j], v[16 * b + 4 * j + 1], v[16 * b + 4 * j + 2],
                                                 v[16 * b + 4 * j + 3]);
                    }
                }
                if constexpr (PH) {
                    // projection form: the accumulator holds x H+- - x~_h V = sqrt(G) x~_l
                    // (G = 64: the factor 1/8 goes into the quantizers' scale arithmetic instead, see kPre)
                    if constexpr (G != 64) {
#pragma unroll
                        for (int j = 0; j < G; ++j) v[j] *= 0.08838834764831845f;  // 1 / sqrt(128)
                    }
                }
                constexpr float kPre = (PH && G == 64) ? 0.125f : 1.0f;
                // number of low-precision values among v[] (a multiple of 16)
                const int nlow = min(G, max(0, p.K_l - col0));
                if constexpr (FMT == 1) {
                    // NVFP4: four blocks of 16 per 64-column chunk; one 32-bit word of scale bytes per chunk
                    static_assert(FMT == 0 || G == 64, "the NVFP4 epilogue works on 64-column chunks");
                    if (col0 < p.K4) {
                        const float ex_scale = __uint_as_float(static_cast<uint32_t>(127 + p.ex) << 23);
                        const float ex_inv = __uint_as_float(static_cast<uint32_t>(127 - p.ex) << 23);
                        uint32_t sfword = 0;
                        uint8_t* crow = reinterpret_cast<uint8_t*>(p.codes) + static_cast<size_t>(row) * (p.K4 / 2) + col0 / 2;
                        if constexpr (STAGED) {
                            if (lane == 0) bulk_wait_group_read_all();  // the staging tile's previous contents have been read
                            __syncwarp();
                        }
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            uint32_t w0 = 0, w1 = 0;
                            if (16 * b < nlow) sfword |= nvfp4_block16(v + 16 * b, kPre, ex_inv, ex_scale, w0, w1) << (8 * b);
                            if constexpr (STAGED) {
                                // 32 bytes of codes per row: rows of 32 bytes, 32-byte swizzle (16-byte piece b / 2)
                                const uint32_t dst = sbuf + static_cast<uint32_t>(lane) * 32u +
                                                     (static_cast<uint32_t>((b >> 1) ^ ((lane >> 2) & 1)) << 4) + (b & 1) * 8u;
                                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst), "r"(w0), "r"(w1) : "memory");
                            } else if (row_ok) {
                                *reinterpret_cast<uint2*>(crow + 8 * b) = make_uint2(w0, w1);  // zero in the padding slots
                            }
                        }
                        if constexpr (STAGED) {
                            fence_proxy_async_smem();  // these writes -> visible to the copy engine
                            __syncwarp();
                            if (lane == 0 && row0w < p.M) {
                                tma_store_2d(&tmap_out, sbuf, col0 / 2, row0w);
                                bulk_commit_group();
                            }
                        }
                      if (row_ok) {
                        const int mr = row & 127;
                        *reinterpret_cast<uint32_t*>(p.xsf + (static_cast<size_t>(row >> 7) * p.nkb64p + (col0 >> 6)) * 512 +
                                                     (mr & 31) * 16 + (mr >> 5) * 4) = sfword;
                        // atoms that only pad the last 256-element k-block: scale 0 (never NaN bytes)
                        if (col0 + 64 >= p.K4)
                            for (int a = (col0 >> 6) + 1; a < p.nkb64p; ++a)
                                *reinterpret_cast<uint32_t*>(p.xsf + (static_cast<size_t>(row >> 7) * p.nkb64p + a) * 512 +
                                                             (mr & 31) * 16 + (mr >> 5) * 4) = 0u;
                      }
                    }
                } else if constexpr (FMT == 3) {
                    // W4A8, first pass: the rotated low-precision coefficients go out as fp32 and the token's maximum is
                    // gathered with an atomic max (non-negative floats order like their bit patterns).  Columns of the chunk
                    // past K_l are written too where the chunk is staged (the quantizer pass reads none of them).
                    if (nlow > 0) {
#pragma unroll
                        for (int b = 0; b < G / 16; ++b) {
                            if (16 * b < nlow) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) tile_amax = fmaxf(tile_amax, fabsf(v[16 * b + j]));
                            }
                        }
                        if constexpr (STAGED) {
#pragma unroll
                            for (int h = 0; h < G / 32; ++h) {  // 32 floats = 128 bytes per row at a time
                                if (lane == 0) bulk_wait_group_read_all();  // the staging tile's previous contents have been read
                                __syncwarp();
#pragma unroll
                                for (int f = 0; f < 8; ++f)
                                    stage_piece128(f, make_uint4(__float_as_uint(v[32 * h + 4 * f]), __float_as_uint(v[32 * h + 4 * f + 1]),
                                                                 __float_as_uint(v[32 * h + 4 * f + 2]), __float_as_uint(v[32 * h + 4 * f + 3])));
                                fence_proxy_async_smem();  // these writes -> visible to the copy engine
                                __syncwarp();
                                if (lane == 0 && row0w < p.M && col0 + 32 * h < p.K_lp) {
                                    tma_store_2d(&tmap_out, sbuf, col0 + 32 * h, row0w);
                                    bulk_commit_group();
                                }
                            }
                        } else if (row_ok) {
                            float4* dst = reinterpret_cast<float4*>(p.xtilde + static_cast<size_t>(row) * p.K_lp + col0);
#pragma unroll
                            for (int b = 0; b < G / 16; ++b) {
                                if (16 * b < nlow) {
#pragma unroll
                                    for (int j = 0; j < 4; ++j)
                                        dst[4 * b + j] = make_float4(v[16 * b + 4 * j], v[16 * b + 4 * j + 1], v[16 * b + 4 * j + 2],
                                                                     v[16 * b + 4 * j + 3]);
                                }
                            }
                        }
                    }
                } else if constexpr (FMT == 2) {
                    if (nlow > 0) {
                        // asymmetric: z = bf16(min), s = bf16((max - min) / 15) over the group's real elements
                        float lo = v[0], hi = v[0];
#pragma unroll
                        for (int b = 0; b < G / 16; ++b) {
                            if (16 * b < nlow) {
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    lo = fminf(lo, v[16 * b + j]);
                                    hi = fmaxf(hi, v[16 * b + j]);
                                }
                            }
                        }
                        const __nv_bfloat16 zb = __float2bfloat16_rn(lo);
                        const float z = __bfloat162float(zb);
                        const float s = hi > lo ? __bfloat162float(__float2bfloat16_rn(__fdiv_rn(hi - lo, 15.0f))) : 0.f;
                        const bool slow = !(s >= 1e-30f);
                        const float inv = slow ? 0.f : __frcp_rn(s);
                        int8_t* crow = p.codes + static_cast<size_t>(row) * p.K_lp + col0;
                        if constexpr (STAGED) {
                            if (lane == 0) bulk_wait_group_read_all();
                            __syncwarp();
                        }
                        if (!slow) {
#pragma unroll
                            for (int b = 0; b < G / 16; ++b) {
                                uint4 packed = make_uint4(0, 0, 0, 0);  // padding slots of a ragged group
                                if (16 * b < nlow) packed = quantize16_asym<false>(v + 16 * b, z, inv, s);
                                if constexpr (STAGED) stage_code_piece(b, packed);
                                else if (row_ok) *reinterpret_cast<uint4*>(crow + 16 * b) = packed;
                            }
                        } else {
#pragma unroll
                            for (int b = 0; b < G / 16; ++b) {
                                uint4 packed = make_uint4(0, 0, 0, 0);
                                if (16 * b < nlow) packed = quantize16_asym<true>(v + 16 * b, z, inv, s);
                                if constexpr (STAGED) stage_code_piece(b, packed);
                                else if (row_ok) *reinterpret_cast<uint4*>(crow + 16 * b) = packed;
                            }
                        }
                        if constexpr (STAGED) {
                            fence_proxy_async_smem();
                            __syncwarp();
                            if (lane == 0 && row0w < p.M) {
                                tma_store_2d(&tmap_out, sbuf, col0, row0w);
                                bulk_commit_group();
                            }
                        }
                        if (row_ok) {
                            const int grp = col0 / G;
                            p.xscale[static_cast<size_t>(grp) * p.ldm + row] = s;
                            // the zero-point, three times, in the extra columns of the bf16 rank-r operand
                            uint16_t* zrow = p.xh + static_cast<size_t>(row) * p.r_pad + p.r_pad0 + grp;
                            const uint16_t zbits = *reinterpret_cast<const uint16_t*>(&zb);
                            zrow[0] = zbits;
                            zrow[p.n_g] = zbits;
                            zrow[2 * p.n_g] = zbits;
                        }
                    }
                } else if (nlow > 0) {
                    // four running maxima instead of one chain of G dependent instructions
                    float am[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int b = 0; b < G / 16; ++b) {
                        if (16 * b < nlow) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) am[j & 3] = fmaxf(am[j & 3], fabsf(v[16 * b + j]));
                        }
                    }
                    const float amax = fmaxf(fmaxf(am[0], am[1]), fmaxf(am[2], am[3])) * kPre;
                    const float s = __bfloat162float(__float2bfloat16_rn(__fdiv_rn(amax, 7.0f)));
                    const bool slow = !(s >= 1e-30f);  // zero or tiny scale: divide instead of multiplying
                    const float inv = slow ? 0.f : __frcp_rn(s) * kPre;
                    int8_t* crow = p.codes + static_cast<size_t>(row) * p.K_lp + col0;
                    if constexpr (STAGED) {
                        if (lane == 0) bulk_wait_group_read_all();  // the staging tile's previous contents have been read
                        __syncwarp();
                    }
                    if (!slow) {
#pragma unroll
                        for (int b = 0; b < G / 16; ++b) {
                            uint4 packed = make_uint4(0, 0, 0, 0);  // padding slots of a ragged group
                            if (16 * b < nlow) packed = quantize16<false>(v + 16 * b, inv, s, kPre);
                            if constexpr (STAGED) stage_code_piece(b, packed);
                            else if (row_ok) *reinterpret_cast<uint4*>(crow + 16 * b) = packed;
                        }
                    } else {
#pragma unroll
                        for (int b = 0; b < G / 16; ++b) {
                            uint4 packed = make_uint4(0, 0, 0, 0);
                            if (16 * b < nlow) packed = quantize16<true>(v + 16 * b, inv, s, kPre);
                            if constexpr (STAGED) stage_code_piece(b, packed);
                            else if (row_ok) *reinterpret_cast<uint4*>(crow + 16 * b) = packed;
                        }
                    }
                    if constexpr (STAGED) {
                        fence_proxy_async_smem();  // these writes -> visible to the copy engine
                        __syncwarp();
                        if (lane == 0 && row0w < p.M) {
                            tma_store_2d(&tmap_out, sbuf, col0, row0w);
                            bulk_commit_group();
                        }
                    }
                    if (row_ok) p.xscale[static_cast<size_t>(col0 / G) * p.ldm + row] = s;
                }
                if (nlow < G && row_ok) {
                    // high-precision coefficients: permuted columns >= K_l
#pragma unroll
                    for (int b = 0; b < G / 16; ++b) {
                        const int pc = col0 + 16 * b;
                        if (16 * b >= nlow && pc < p.n_out) {
                            uint4 lo = make_uint4(pack_bf16x2(v[16 * b + 0], v[16 * b + 1]), pack_bf16x2(v[16 * b + 2], v[16 * b + 3]),
                                                  pack_bf16x2(v[16 * b + 4], v[16 * b + 5]), pack_bf16x2(v[16 * b + 6], v[16 * b + 7]));
                            uint4 hi = make_uint4(pack_bf16x2(v[16 * b + 8], v[16 * b + 9]), pack_bf16x2(v[16 * b + 10], v[16 * b + 11]),
                                                  pack_bf16x2(v[16 * b + 12], v[16 * b + 13]), pack_bf16x2(v[16 * b + 14], v[16 * b + 15]));
                            uint4* dst = reinterpret_cast<uint4*>(p.xh + static_cast<size_t>(row) * p.r_pad + (pc - p.K_l));
                            dst[0] = lo;
                            dst[1] = hi;
                        }
                    }
                }
            }
            if constexpr (FMT == 3) {
                if (row_ok && tile_amax > 0.f) atomicMax(p.rowmax + row, __float_as_uint(tile_amax));
            }
            // release the accumulator: every tcgen05.ld of this warp has completed
            tc_fence_before_sync();
            // every lane arrives for itself: a warp barrier followed by one elected lane's arrival costs about a hundred cycles more
            if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));  // the leader's barrier
            else mbar_arrive(tempty_bar(acc));
            // zero padding of the bf16 rank-r operand (written once, by the tile that holds column K-1)
            if (!PH && n_blk == num_n_blocks - 1 && row_ok && (BM == 256 || half == 0)) {
                for (int c = p.r; c < p.r_pad0; c += 8)
                    *reinterpret_cast<uint4*>(p.xh + static_cast<size_t>(row) * p.r_pad + c) = make_uint4(0, 0, 0, 0);
                if constexpr (FMT == 2) {  // behind the 3 n_g zero-point columns
                    for (int c = p.r_pad0 + 3 * p.n_g; c < p.r_pad; ++c) p.xh[static_cast<size_t>(row) * p.r_pad + c] = 0;
                }
            }
        }
    }

    if (warp >= 2 && lane == 0) bulk_wait_group_all();  // an epilogue warp's TMA stores are performed before the CTA leaves
    if (warp == 2 && lane == 0) TRACE_CLK(p.status, 18);
    // ---------------------------------------------------------------- teardown
    if constexpr (PAIR) {
        if (warp == 1 && lane == 0 && cta_rank == 0 && *abort_flag != 0) {  // a wait gave up: let issued MMAs finish first
            umma_commit_pair(bar_base + 200u, 1);
            const unsigned long long t0 = globaltimer_ns();
            while (!mbar_try_wait(bar_base + 200u, 0) && globaltimer_ns() - t0 < 100000000ull) {}
        }
        tc_fence_before_sync();
        cluster_sync_all();  // neither CTA leaves while the other may still read its operands or signal its barriers
        if (warp == 1) {
            tc_fence_after_sync();
            tmem_dealloc_pair(tmem_base, 512);
        }
    } else {
        if (warp == 1 && lane == 0 && *abort_flag != 0) umma_drain(bar_base + 200u);  // a wait gave up: let issued MMAs finish first
        tc_fence_before_sync();
        __syncthreads();
        if (warp == 1) {
            tc_fence_after_sync();
            tmem_dealloc(tmem_base, 512);
        }
    }
}

// Sums the ranges of a split reduction in range order and rounds to bf16: xh[row][c] = bf16(sum_s partial[s][row][c]).
// One thread per 8 consecutive columns.
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float* __restrict__ partial, int ksplit, int M, int n_out,
                                                              uint16_t* __restrict__ xh) {
    grid_dependency_wait();
    grid_launch_dependents();
    const long idx = static_cast<long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long total = static_cast<long>(M) * n_out / 8;
    if (idx >= total) return;
    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < ksplit; ++s) {
        const float4* src = reinterpret_cast<const float4*>(partial + static_cast<size_t>(s) * M * n_out) + 2 * idx;
        const float4 u = src[0], w = src[1];
        a[0] += u.x; a[1] += u.y; a[2] += u.z; a[3] += u.w;
        a[4] += w.x; a[5] += w.y; a[6] += w.z; a[7] += w.w;
    }
    reinterpret_cast<uint4*>(xh)[idx] = make_uint4(pack_bf16x2(a[0], a[1]), pack_bf16x2(a[2], a[3]), pack_bf16x2(a[4], a[5]),
                                                   pack_bf16x2(a[6], a[7]));
}

static std::atomic<int> g_first_step_split{1};  // projection form: 0 keeps the first step's reduction in one piece
static std::atomic<int> g_rotation_plan{0};  // 0: chosen per call; 1: 128 x 128, 2: 128 x 256, 3: 256 x 256 tiles, 4: CTA pairs, 5: 128 x 64

}  // namespace

void set_first_step_split(bool on) { g_first_step_split.store(on ? 1 : 0); }

dirotq_status_t set_rotation_plan(int plan) {
    if (plan < 0 || plan > 5) return DIROTQ_ERR_INVALID_ARG;
    g_rotation_plan.store(plan);
    return DIROTQ_OK;
}

// The tensor map the epilogue's TMA stores go through: the INT4 activation codes (one byte each, [M][K_lp], boxes of 32 rows x
// one group), the NVFP4 codes (two per byte, [M][K4/2], boxes of 32 rows x 32 bytes) or, on the W4A8 path, the fp32 coefficients
// ([M][K_lp], boxes of 32 rows x 32 values).
static dirotq_status_t encode_out_map(CUtensorMap* out, const Geometry& g, const RotateArgs& a, const CUtensorMap& unused) {
    if (g.fmt == 3)
        return encode_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.xtilde, (uint64_t)g.K_lp, (uint64_t)a.M, (uint64_t)g.K_lp * 4,
                              32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    (void)unused;
    if (g.fmt == 1)  // NVFP4: two codes per byte, 32 bytes per row and 64-column chunk
        return encode_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.codes, (uint64_t)g.K4 / 2, (uint64_t)a.M, (uint64_t)g.K4 / 2, 32, 32,
                              CU_TENSOR_MAP_SWIZZLE_32B);
    return encode_tmap_2d(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.codes, (uint64_t)g.K_lp, (uint64_t)a.M, (uint64_t)g.K_lp, g.G, 32,
                          g.G == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B);
}

dirotq_status_t launch_rotate_quantize(const dirotq_layer* L, const RotateArgs& a, cudaStream_t stream) {
    const Geometry& g = L->geo;
    RotKernelParams p;
    p.n_out = g.K; p.k_red = g.K;
    p.M = a.M; p.K = g.K; p.K_l = g.K_l; p.K_lp = g.K_lp; p.r = g.r; p.r_pad = g.r_pad; p.r_pad0 = g.r_pad0; p.ldm = a.ldm; p.n_g = g.n_g;
    p.codes = a.codes; p.xscale = a.xscale; p.xh = a.xh; p.xrot = a.xrot; p.status = a.status;
    p.xsf = a.xsf; p.K4 = g.K4; p.nkb64p = g.nkb64p; p.ex = L->act_scale_log2;
    p.xtilde = a.xtilde; p.rowmax = a.rowmax;
    // Tile plan.  128 x 256 is the default.  128 x 128 when the wide tiles would not give every SM about two of them
    // (few, large tiles leave a nearly empty last wave: 160 tiles on 148 SMs take as long as 296).  256 x 256 (a third
    // fewer operand bytes per flop, but the epilogue, about 11 k-blocks' worth, is not overlapped) for long main
    // loops only: measured 0.99 -> 0.92 ms at M = 4608, K = 12288 and 1.54 -> 1.48 ms at K = 15360, but 0.125 ->
    // 0.141 ms at M = 9216, K = 3072.
    const int sms = sm_count(L->device);
    const long mb128 = (a.M + 127) / 128, mb256 = (a.M + 255) / 256, nb256 = (g.K + 255) / 256;
    int plan = g_rotation_plan.load();
    if (plan == 0) {
        const long nb128 = (g.K + 127) / 128;
        const long waves128 = (mb128 * nb256 + sms - 1) / sms, waves256 = (mb256 * nb256 + sms - 1) / sms;
        const long waves_narrow = (mb128 * nb128 + sms - 1) / sms;
        const double kb = static_cast<double>(g.K / BK);
        // a 256-row tile in units of a 128-row tile; once x no longer fits the L2 beside the rotation the 128-row plan
        // re-reads it from HBM and the ratio falls to 1.9 (measured at M = 18432, K = 3072: 0.304 -> 0.288 ms)
        const bool x_exceeds_l2 = static_cast<double>(a.M) * g.K * 2.0 > 96e6;
        const double cost256 = x_exceeds_l2 ? 1.9 : 1.86 + 11.0 / kb;
        // a 128-column tile costs about 0.62 of a 256-column one: narrow tiles when that shortens the schedule (few
        // tiles: M = 256, K = 1152 runs on 18 instead of 10 SMs; M = 4096, K = 1152: 288 tiles in two waves instead of
        // 160 in two), not otherwise (M = 1024, K = 3072: 96 wide tiles in one wave, 30 us, against 192 narrow ones in
        // two, 45 us)
        // few token rows: when even the 128-column tiles would keep fewer than half of the SMs busy, 64-column tiles (eight
        // 24 KB stages) on twice as many: every CTA streams all of x's row block and its own columns of the rotation through
        // one SM's port to L2, so the time of a call this small falls with the bytes per CTA
        if (2 * mb128 * nb128 <= sms && g.G == 64) plan = 5;
        else if (0.62 * static_cast<double>(waves_narrow) < static_cast<double>(waves128)) plan = 1;
        else if ((g.K >= 8192 || x_exceeds_l2) && cost256 * static_cast<double>(waves256) < 0.98 * static_cast<double>(waves128)) plan = 3;
        // CTA pairs where there are a few waves of tiles and the main loop is not long enough for the operand traffic
        // to hide behind the MMAs anyway (measured against 128 x 256 tiles: M = 4608, K = 3072 68.4 -> 67.3 us; M = 9216,
        // K = 3072 122 -> 114; M = 4096, K = 4608 124 -> 111; at K = 12288 and 15360 the 256-row plan stays ahead)
        else if (mb128 * nb256 >= 5 * sms / 2 && g.K < 8192) plan = 4;
        else plan = 2;
    }
    if (plan == 4) {
        // CTA pairs: 256 rows x 256 columns per pair, 128 rows of x and half of the rotation tile per CTA
        CUtensorMap tmap_xp;
        dirotq_status_t stp = encode_tmap_2d(&tmap_xp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.x, (uint64_t)g.K, (uint64_t)a.M,
                                             (uint64_t)g.K * 2, BK, 128, CU_TENSOR_MAP_SWIZZLE_128B);
        if (stp != DIROTQ_OK) return stp;
        const long pair_tiles = ((a.M + 255) / 256) * nb256;
        const int pairs = static_cast<int>(pair_tiles < sms / 2 ? pair_tiles : sms / 2);
        const int vi = g.fmt == 1 ? 2 : g.fmt == 3 ? 5 : (g.fmt == 2 ? (g.G == 64 ? 3 : 4) : (g.G == 64 ? 0 : 1));
        using PairFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const RotKernelParams);
        static const PairFn pair_table[6] = {
            rotate_quant_kernel<64, 0, 256, 128, false, 8, true>, rotate_quant_kernel<128, 0, 256, 128, false, 8, true>,
            rotate_quant_kernel<64, 1, 256, 128, false, 8, true>, rotate_quant_kernel<64, 2, 256, 128, false, 8, true>,
            rotate_quant_kernel<128, 2, 256, 128, false, 8, true>, rotate_quant_kernel<64, 3, 256, 128, false, 8, true>};
        static SmemOptIn<6> opt_in_pair;
        if (!opt_in_pair.ensure(pair_table[vi], vi, L->device, SMEM_BYTES)) return DIROTQ_ERR_CUDA;
        CUtensorMap tmap_out;
        stp = encode_out_map(&tmap_out, g, a, tmap_xp);
        if (stp != DIROTQ_OK) return stp;
        return launch_kernel_pairs(pair_table[vi], 2 * pairs, NUM_THREADS, SMEM_BYTES, stream, g.fmt != 3, tmap_xp, L->tmap_qt128,
                                   tmap_xp, L->tmap_qt128, tmap_out, p) == cudaSuccess
                   ? DIROTQ_OK
                   : DIROTQ_ERR_CUDA;
    }
    if (plan == 5 && g.G != 64) plan = 1;  // a tile holds whole groups
    if (plan == 5) {
        CUtensorMap tmap_x5;
        dirotq_status_t st5 = encode_tmap_2d(&tmap_x5, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.x, (uint64_t)g.K, (uint64_t)a.M,
                                             (uint64_t)g.K * 2, BK, 128, CU_TENSOR_MAP_SWIZZLE_128B);
        if (st5 != DIROTQ_OK) return st5;
        const long tiles5 = mb128 * ((g.K + 63) / 64);
        const int vi5 = g.fmt == 1 ? 1 : g.fmt == 2 ? 2 : g.fmt == 3 ? 3 : 0;
        using Fn5 = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const RotKernelParams);
        static const Fn5 table5[4] = {rotate_quant_kernel<64, 0, 64, 128>, rotate_quant_kernel<64, 1, 64, 128>,
                                      rotate_quant_kernel<64, 2, 64, 128>, rotate_quant_kernel<64, 3, 64, 128>};
        static SmemOptIn<4> opt_in5;
        if (!opt_in5.ensure(table5[vi5], vi5, L->device, SMEM_BYTES)) return DIROTQ_ERR_CUDA;
        CUtensorMap tmap_out5;
        st5 = encode_out_map(&tmap_out5, g, a, tmap_x5);
        if (st5 != DIROTQ_OK) return st5;
        return launch_kernel(table5[vi5], static_cast<int>(tiles5 < sms ? tiles5 : sms), NUM_THREADS, SMEM_BYTES, stream, g.fmt != 3,
                             tmap_x5, L->tmap_qt64, tmap_x5, L->tmap_qt64, tmap_out5, p) == cudaSuccess
                   ? DIROTQ_OK
                   : DIROTQ_ERR_CUDA;
    }
    const int bm = plan == 3 ? 256 : 128, bn = plan == 1 ? 128 : 256;
    CUtensorMap tmap_x;
    dirotq_status_t st = encode_tmap_2d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.x, (uint64_t)g.K, (uint64_t)a.M,
                                        (uint64_t)g.K * 2, BK, bm, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    const long num_tiles = ((a.M + bm - 1) / bm) * ((g.K + bn - 1) / bn);
    const int grid = num_tiles < sms ? static_cast<int>(num_tiles) : sms;
    const int vi = g.fmt == 1 ? 2 : g.fmt == 3 ? 5 : (g.fmt == 2 ? (g.G == 64 ? 3 : 4) : (g.G == 64 ? 0 : 1));
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const RotKernelParams);
    static const KernelFn table[3][6] = {
        {rotate_quant_kernel<64, 0, 128, 128>, rotate_quant_kernel<128, 0, 128, 128>, rotate_quant_kernel<64, 1, 128, 128>,
         rotate_quant_kernel<64, 2, 128, 128>, rotate_quant_kernel<128, 2, 128, 128>, rotate_quant_kernel<64, 3, 128, 128>},
        {rotate_quant_kernel<64, 0, 256, 128>, rotate_quant_kernel<128, 0, 256, 128>, rotate_quant_kernel<64, 1, 256, 128>,
         rotate_quant_kernel<64, 2, 256, 128>, rotate_quant_kernel<128, 2, 256, 128>, rotate_quant_kernel<64, 3, 256, 128>},
        {rotate_quant_kernel<64, 0, 256, 256>, rotate_quant_kernel<128, 0, 256, 256>, rotate_quant_kernel<64, 1, 256, 256>,
         rotate_quant_kernel<64, 2, 256, 256>, rotate_quant_kernel<128, 2, 256, 256>, rotate_quant_kernel<64, 3, 256, 256>}};
    const KernelFn kern = table[plan - 1][vi];
    // the W4A8 path puts a memset in front of this kernel; programmatic serialization only relaxes the wait for a
    // preceding KERNEL, so nothing would be gained there and the launch is a plain one
    const bool dependent = g.fmt != 3;
    static SmemOptIn<18> opt_in;
    if (!opt_in.ensure(kern, (plan - 1) * 6 + vi, L->device, SMEM_BYTES)) return DIROTQ_ERR_CUDA;
    const CUtensorMap& tmap_q = plan == 1 ? L->tmap_qt128 : L->tmap_qt;
    CUtensorMap tmap_out;
    st = encode_out_map(&tmap_out, g, a, tmap_x);
    if (st != DIROTQ_OK) return st;
    return launch_kernel(kern, grid, NUM_THREADS, SMEM_BYTES, stream, dependent, tmap_x, tmap_q, tmap_x, tmap_q, tmap_out, p) == cudaSuccess
               ? DIROTQ_OK
               : DIROTQ_ERR_CUDA;
}

// Projection form (fmt 4): x~_h = bf16(x U_hb) with the rotation kernel on r_pad output columns, then
// x~_l = (x H+- - x~_h V) / sqrt(G) and the group quantizer with the same kernel in its PH mode.
dirotq_status_t launch_project_quantize(const dirotq_layer* L, const RotateArgs& a, cudaStream_t stream) {
    const Geometry& g = L->geo;
    if (a.xrot != nullptr) return DIROTQ_ERR_INVALID_ARG;  // there is no K-wide rotated activation in this form
    const int sms = sm_count(L->device);
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, const RotKernelParams);
    RotKernelParams p;
    p.M = a.M; p.K = g.K; p.K_lp = g.K_lp; p.r_pad = g.r_pad; p.r_pad0 = g.r_pad0; p.ldm = a.ldm; p.n_g = g.n_g;
    p.codes = a.codes; p.xscale = a.xscale; p.xh = a.xh; p.xrot = nullptr; p.status = a.status;
    p.xsf = nullptr; p.K4 = 0; p.nkb64p = 0; p.ex = 0; p.xtilde = nullptr; p.rowmax = nullptr;
    dirotq_status_t st;
    CUtensorMap tmap_x;
    st = encode_tmap_2d(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.x, (uint64_t)g.K, (uint64_t)a.M, (uint64_t)g.K * 2, BK,
                        128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    {
        // step 1: all r_pad output columns are "high" (K_l = 0): the epilogue only rounds them to bf16 into xh
        RotKernelParams p1 = p;
        p1.n_out = g.r_pad; p1.k_red = g.K; p1.K_l = 0; p1.r = g.r_pad;
        const KernelFn k1 = rotate_quant_kernel<64, 0, 128, 128>;
        static SmemOptIn<1> opt_in1;
        if (!opt_in1.ensure(k1, 0, L->device, SMEM_BYTES)) return DIROTQ_ERR_CUDA;
        long tiles = static_cast<long>((a.M + 127) / 128) * ((g.r_pad + 127) / 128);
        // Few row tiles leave most SMs idle while x streams through: cut the reduction into ranges, one tile each.  The
        // ranges' fp32 sums are parked in the (still unused) code region of the workspace and added up in range order.
        int ksplit = static_cast<int>(sms / tiles);
        ksplit = std::min(ksplit, std::min(8, (g.K / BK) / 8));
        if (g.K / BK < 32) ksplit = 1;  // short reductions gain nothing (K = 1152 measured the same either way): one launch fewer
        const size_t code_bytes = static_cast<size_t>(a.M) * (g.fmt == 1 ? g.K4 / 2 : g.K_lp);
        while (ksplit > 1 && static_cast<size_t>(ksplit) * a.M * g.r_pad * 4 > code_bytes) --ksplit;
        if (ksplit > 1 && g_first_step_split.load() != 0) {
            p1.ksplit = ksplit;
            p1.partial = reinterpret_cast<float*>(a.codes);
            tiles *= ksplit;
        }
        if (launch_kernel(k1, static_cast<int>(tiles < sms ? tiles : sms), NUM_THREADS, SMEM_BYTES, stream, true, tmap_x,
                          L->tmap_qt128, tmap_x, L->tmap_qt128, tmap_x /* no codes in this step */, p1) != cudaSuccess)
            return DIROTQ_ERR_CUDA;
        if (p1.partial != nullptr) {
            const long threads = static_cast<long>(a.M) * g.r_pad / 8;
            if (launch_kernel(reduce_partials_kernel, static_cast<int>((threads + 255) / 256), 256, 0, stream, true,
                              static_cast<const float*>(p1.partial), p1.ksplit, a.M, g.r_pad, a.xh) != cudaSuccess)
                return DIROTQ_ERR_CUDA;
        }
    }
    {
        // step 2: x~_h [M][r_pad] against -V^T [K][r_pad], then x against the Hadamard block, group by group (see the
        // kernel's PH note); every output column is low-precision (K_l = K)
        CUtensorMap tmap_xh;
        st = encode_tmap_2d(&tmap_xh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.xh, (uint64_t)g.r_pad, (uint64_t)a.M,
                            (uint64_t)g.r_pad * 2, BK, 128, CU_TENSOR_MAP_SWIZZLE_128B);
        if (st != DIROTQ_OK) return st;
        RotKernelParams p2 = p;
        p2.n_out = g.K; p2.k_red = g.r_pad; p2.K_l = g.K; p2.r = g.r;
        const int vi = g.fmt == 1 ? 2 : (g.G == 64 ? 0 : 1);
        static const KernelFn k2s[3] = {rotate_quant_kernel<64, 4, 256, 128, true, 8>, rotate_quant_kernel<128, 4, 256, 128>,
                                        rotate_quant_kernel<64, 1, 256, 128, true, 8>};
        const int threads2 = NUM_THREADS;
        const KernelFn k2 = k2s[vi];
        if (g.fmt == 1) { p2.xsf = a.xsf; p2.K4 = g.K4; p2.nkb64p = g.nkb64p; p2.ex = L->act_scale_log2; }
        static SmemOptIn<3> opt_in2;
        if (!opt_in2.ensure(k2, vi, L->device, SMEM_BYTES)) return DIROTQ_ERR_CUDA;
        const long tiles = static_cast<long>((a.M + 127) / 128) * ((g.K + 255) / 256);
        CUtensorMap tmap_out;
        st = encode_out_map(&tmap_out, g, a, tmap_x);
        if (st != DIROTQ_OK) return st;
        if (launch_kernel(k2, static_cast<int>(tiles < sms ? tiles : sms), threads2, SMEM_BYTES, stream, true, tmap_xh, L->tmap_qt,
                          tmap_x, L->tmap_had, tmap_out, p2) != cudaSuccess)
            return DIROTQ_ERR_CUDA;
    }
    return DIROTQ_OK;
}

}  // namespace dirotq
