// NVFP4 variant of the second kernel (paper Sec. 5.1: 4-bit float elements, blocks of 16, FP8 scales).
//
//   y[m,n] = bf16( 2^(ex+ew) * D[m,n] + bias[n] ),
//   D = sum over blocks of 16:  sf_x[m,blk] * sf_w[n,blk] * sum_{k in blk} v_x[m,k] v_w[n,k]   (E2M1 x E2M1)
//       + sum_{i<r} x~_h[m,i] * (W~_h[i,n] * 2^-(ex+ew))                                        (bf16 x bf16)
//
// The block scales are applied INSIDE the tensor core (tcgen05.mma kind::mxf4nvf4, block16): there is
// no per-group pass over the accumulator on the CUDA cores, which is what limits the INT4 kernel.
// The two per-tensor scales are powers of two, so the bf16 rank-r weights can be pre-divided
// exactly and the rank-r branch accumulates into the same fp32 tile (kind::f16 on the same TMEM
// columns); the epilogue is one multiply-add per element.
//
// Data movement: packed E2M1 operands by TMA (128-byte rows = 256 elements, 128-byte swizzle); the
// E4M3 scale factors travel as 512-byte atoms (128 rows x 4 scales, row r at (r%32)*16 + (r/32)*4),
// fetched with cp.async.bulk and copied into tensor memory with tcgen05.cp.32x128b.warpx4 by two copier
// threads, which hand the stage to the MMA thread through an mbarrier (tcgen05.commit).
//
// Roles (384 threads): warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2..3 copy the scale factors of
// each stage from shared to tensor memory (activation side / weight side), warps 4..11 epilogue.
// TMEM: one 256-column fp32 accumulator (or two of 128 columns, see Plan) and, per pipeline stage, 16 columns of
// scale factors for the tokens and 16 per 128 output columns.
#include "common.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

#include <atomic>

namespace dirotq {
namespace {

constexpr int BM = 128;
constexpr int BKE = 256;      // E2M1 elements per k-block (128-byte rows)
constexpr int A_BYTES = BM * 128;      // 16 KB
constexpr int SF_BYTES = 4 * 512;      // four atoms per 128 rows (tokens or output columns) and k-block
constexpr int NUM_THREADS = 384;
constexpr int NUM_EPI_WARPS = 8;

// Tile plans.  Both kernels are bound by the stream of operands from L2 into shared memory, so the wider tile (a
// quarter less traffic per flop) is the default; the 128-column plan double-buffers the accumulator and serves
// layers with few tiles.  With 256 columns one accumulator (256 of the 512 tensor-memory columns) is all that fits
// beside the scale factors: the epilogue of a tile then does not overlap the MMAs of the next, but the producer keeps
// filling the stages meanwhile, and the MMAs catch up on a full pipeline.
// PAIR (BN = 256): clusters of two CTAs share every MMA (cta_group::2, M = 256): a pair owns 256 token rows x 256 columns;
// each CTA loads its own 128 rows of activation codes with their scale atoms, ONE of the tile's two 128-column blocks of
// weight codes, and the scale atoms of both blocks (every CTA's tensor core scales all 256 columns of its rows): 38
// instead of 54 KB per k-block and CTA.  All loads complete on the CTA's own "stage full" barrier; the second CTA's first
// copier thread then tells the leader (one arrival per stage on the leader's "peer landed" barrier), whose copier threads
// issue the pair-wide scale copies and whose MMA thread issues the pair-wide MMAs.
template <int BN, bool PAIR = false>
struct Plan {
    static constexpr int NB = BN / 128;               // 128-column blocks per tile
    static constexpr int NB_DATA = PAIR ? 1 : NB;     // ... whose weight codes this CTA holds
    // outputs through per-warp staging tiles and TMA stores where the shared memory allows it: the pair plan, and the
    // 128-column plan with five stages instead of six
    static constexpr bool STAGED_OUT = PAIR || BN == 128;
    static constexpr int STAGES = PAIR ? 5 : (BN == 128 ? 5 : 4);
    static constexpr int ACC_BUFS = BN == 128 ? 2 : 1;
    static constexpr int B_BYTES = NB_DATA * 128 * 128;  // 16 / 32 KB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + (1 + NB) * SF_BYTES;  // 36 / 54 KB (pairs: 38 KB)
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int BIAS_OFFSET = BAR_OFFSET + 256;  // two buffers of a tile's bias values
    // pairs: one 32-row x 128-byte staging tile per epilogue warp (1024-byte aligned: 128-byte swizzle), from which the outputs
    // leave as TMA stores
    static constexpr int STORE_OFFSET = (BIAS_OFFSET + 2 * BN * 4 + 1023) / 1024 * 1024;
    static constexpr int SMEM_BYTES = STAGED_OUT ? STORE_OFFSET + NUM_EPI_WARPS * 4096 + 1024 : BIAS_OFFSET + 2 * BN * 4 + 1024;
    static constexpr int TMEM_SF_BASE = ACC_BUFS * BN;    // columns 256.. hold the scale factors
    static constexpr int SF_COLS = 16 * (1 + NB);         // per stage: 16 columns for the tokens, 16 per 128 output columns
    static_assert(TMEM_SF_BASE + STAGES * SF_COLS <= 512, "tensor memory plan");
    static_assert(8 * ((PAIR ? 4 : 3) * STAGES + 4) <= 192, "barriers end below the words at +192");
    static_assert(SMEM_BYTES <= 232448, "shared memory plan");
    static_assert(STAGE_BYTES % 1024 == 0, "operand tiles must stay 1024-byte aligned");
};

struct NvKernelParams {
    int M, N, num_kb, nkb64p, lr_chunks;
    const uint8_t* xsf;   // activation scale atoms [ceil(M/128)][nkb64p][512]
    const uint8_t* wsf;   // weight scale atoms, see wsf_atom_offset
    const float* bias;
    const float* out_scale;  // 2^(ex+ew)
    uint16_t* y;
    int* status;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// 1-D bulk copy global -> shared, completion counted in bytes on `bar` (16-byte aligned, size % 16 == 0).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
                 : "memory");
}

// Shared-memory descriptor of one scale-factor atom for tcgen05.cp: 32 rows of 16 bytes, no swizzle,
// 8-row core matrices 128 bytes apart.
__device__ __forceinline__ uint64_t sf_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>(128 >> 4) << 16;  // leading byte offset (one 16-byte column only: not stepped over)
    d |= static_cast<uint64_t>(128 >> 4) << 32;  // stride byte offset: next group of 8 rows
    d |= static_cast<uint64_t>(1) << 46;         // descriptor version
    return d;                                    // layout type 0: no swizzle
}

// 32 lanes x 128 bits from shared memory into 4 TMEM columns, replicated to the four lane quadrants.
__device__ __forceinline__ void tmem_cp_32x128b_warpx4(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
// The same over a CTA pair: each CTA's shared memory (same offset) into its own tensor memory (same address).
__device__ __forceinline__ void tmem_cp_32x128b_warpx4_pair(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}

// Block-scaled instruction descriptor: E2M1 x E2M1 -> fp32, UE4M3 scales, both operands K-major.
__host__ __device__ constexpr uint32_t nvfp4_idesc(uint32_t M, uint32_t N) {
    return (1u << 7) /*A: E2M1*/ | (1u << 10) /*B: E2M1*/ | ((N >> 3) << 17) | (0u << 23) /*scale format UE4M3*/ |
           ((M >> 4) << 24);
}

__device__ __forceinline__ void umma_nvfp4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t tsfa,
                                           uint32_t tsfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
        : "memory");
}

__device__ __forceinline__ void umma_nvfp4_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t tsfa,
                                                uint32_t tsfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t"
        "}\n" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
        : "memory");
}

template <int BN, bool PAIR = false>
__global__ void __launch_bounds__(NUM_THREADS, 1)
nvfp4_gemm_kernel(const __grid_constant__ CUtensorMap tmap_codes, const __grid_constant__ CUtensorMap tmap_wcodes,
                  const __grid_constant__ CUtensorMap tmap_xh, const __grid_constant__ CUtensorMap tmap_wh,
                  const __grid_constant__ CUtensorMap tmap_y, const NvKernelParams p) {
    using P = Plan<BN, PAIR>;
    static_assert(!PAIR || BN == 256, "pairs: 256 columns per pair");
    constexpr int NB = P::NB, NB_DATA = P::NB_DATA, STAGES = P::STAGES, ACC_BUFS = P::ACC_BUFS, B_BYTES = P::B_BYTES;
    constexpr int STAGE_BYTES = P::STAGE_BYTES, BAR_OFFSET = P::BAR_OFFSET, BIAS_OFFSET = P::BIAS_OFFSET;
    constexpr int TMEM_SF_BASE = P::TMEM_SF_BASE, SF_COLS = P::SF_COLS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
    auto sfready_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + 4 + s); };
    auto peer_bar = [&](int s) { return bar_base + 8u * (3 * STAGES + 4 + s); };  // pairs, leader: the other CTA's stage has landed
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + BAR_OFFSET + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + BAR_OFFSET + 196);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Trace build (TRACE_CLK), stages 6..8 of the block's first tile: slots 9..11 producer has issued the stage, 12..14 first copier warp
    // sees it landed, 15..17 / 18..20 first / second copier warp has committed its scale copies, 21..23 MMA warp sees the scales
    // ready, 24..26 it has committed the stage's MMAs; tiles 0, 1, 2 of the first epilogue warp: accumulator seen / released / outputs
    // handed over in slots 27..29, 1..3, 4..6; slot 30 entry.
    if (threadIdx.x == 0) TRACE_CLK(p.status, 30);
    const uint32_t cta_rank = PAIR ? cluster_ctarank() : 0u;
    constexpr int TILE_ROWS = PAIR ? 2 * BM : BM;  // token rows of a tile (of the pair's tile)
    const int tile_first = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
    const int tile_step = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
    const int num_m_blocks = (p.M + TILE_ROWS - 1) / TILE_ROWS;
    const int num_n_blocks = (p.N + BN - 1) / BN;
    const int num_tiles = num_m_blocks * num_n_blocks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(sfready_bar(s), 2);  // one arrival per copier warp
            if constexpr (PAIR) mbar_init(peer_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), NUM_EPI_WARPS * 32 * (PAIR ? 2 : 1));
        }
        mbar_init(bar_base + 200u, 1);  // spare: see umma_drain
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap_codes);
        tma_prefetch_desc(&tmap_wcodes);
        tma_prefetch_desc(&tmap_xh);
        tma_prefetch_desc(&tmap_wh);
        if constexpr (P::STAGED_OUT) tma_prefetch_desc(&tmap_y);
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
    // everything above touched only this CTA's own shared and tensor memory; what follows reads the first kernel's output
    grid_dependency_wait();
    // the next layer's first kernel may be scheduled as this grid's CTAs leave their SMs (it waits for this whole grid)
    grid_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // (the whole warp walks the loops and waits, one elected lane issues: counters, addresses and coordinates stay
        // warp-uniform, which shortens the chain of instructions per stage; the same in the MMA and copier warps)
        {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step) {
                // m_blk: this CTA's block of 128 token rows
                const int m_blk = (tile % num_m_blocks) * (PAIR ? 2 : 1) + static_cast<int>(cta_rank), n_blk = tile / num_m_blocks;
                const int m0 = m_blk * BM, n0 = n_blk * BN;
                // 128-column blocks of this tile that exist (the scale atoms of a missing one are not fetched; its
                // outputs are never stored)
                const int nb_here = min(NB, (p.N + 127) / 128 - n_blk * NB);
                // pairs: the second CTA's block of rows may lie past M (odd number of row blocks): it has no scale atoms
                // (its codes are read as zeros, its outputs never stored)
                const int sfa_here = m0 < p.M ? 1 : 0;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    if (!elect_one()) continue;
                    mbar_arrive_expect_tx(full_bar(s), A_BYTES + B_BYTES + (sfa_here + nb_here) * SF_BYTES);
                    tma_load_2d(st, &tmap_codes, full_bar(s), kb * 128, m0);             // byte coordinates
#pragma unroll
                    for (int b = 0; b < NB_DATA; ++b)  // rows past N are filled with zeros (and still counted)
                        tma_load_2d(st + A_BYTES + b * 16384, &tmap_wcodes, full_bar(s), kb * 128,
                                    n0 + (PAIR ? static_cast<int>(cta_rank) : b) * 128);
                    if (sfa_here)
                        bulk_load(st + A_BYTES + B_BYTES, p.xsf + (static_cast<size_t>(m_blk) * p.nkb64p + kb * 4) * 512, SF_BYTES,
                                  full_bar(s));
                    // the atoms of the tile's 128-column blocks for this k-block are contiguous: one copy
                    bulk_load(st + A_BYTES + B_BYTES + SF_BYTES, p.wsf + wsf_atom_offset(n_blk * NB, kb * 4, p.nkb64p),
                              nb_here * SF_BYTES, full_bar(s));
                    if (it >= 6 && it <= 8) TRACE_CLK(p.status, 3 + it);
                }
                if (!ok) break;
                for (int lr = 0; lr < p.lr_chunks; ++lr, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    if (!elect_one()) continue;
                    mbar_arrive_expect_tx(full_bar(s), A_BYTES + B_BYTES);
                    tma_load_2d(st, &tmap_xh, full_bar(s), lr * 64, m0);
#pragma unroll
                    for (int b = 0; b < NB_DATA; ++b)
                        tma_load_2d(st + A_BYTES + b * 16384, &tmap_wh, full_bar(s), lr * 64,
                                    n0 + (PAIR ? static_cast<int>(cta_rank) : b) * 128);
                }
            }
            if (!ok && lane == 0) {
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1) && globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (cta_rank == 0) {
            constexpr uint32_t idesc_nv = nvfp4_idesc(TILE_ROWS, BN);
            constexpr uint32_t idesc_bf = umma_idesc(1 /*f32*/, 1 /*bf16*/, TILE_ROWS, BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step, ++tcount) {
                const uint32_t acc = tcount % ACC_BUFS;
                if (!mbar_wait(tempty_bar(acc), ((tcount / ACC_BUFS) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem_base + acc * BN;
                for (int kb = 0; kb < p.num_kb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    const uint32_t tsf = tmem_base + TMEM_SF_BASE + s * SF_COLS;
                    // the scale factors of this stage are copied into tensor memory by the copier warps, which have seen the
                    // stage's loads land first (in both CTAs of a pair): their barrier covers the operands as well
                    if (!mbar_wait(sfready_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t adesc = umma_desc_sw128(st);
                    const uint64_t bdesc = umma_desc_sw128(st + A_BYTES);
                    if (!elect_one()) continue;
                    if (it >= 6 && it <= 8) TRACE_CLK(p.status, 15 + it);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {  // K = 64 elements = 32 bytes per instruction
                        if constexpr (PAIR)
                            umma_nvfp4_pair(d, adesc + 2 * k, bdesc + 2 * k, idesc_nv, tsf + 4 * k, tsf + 16 + 4 * NB * k, (kb | k) != 0);
                        else
                            umma_nvfp4(d, adesc + 2 * k, bdesc + 2 * k, idesc_nv, tsf + 4 * k, tsf + 16 + 4 * NB * k, (kb | k) != 0);
                    }
                    if constexpr (PAIR) umma_commit_pair(empty_bar(s), 3);  // both CTAs' producers may refill the stage
                    else umma_commit(empty_bar(s));
                    if (it >= 6 && it <= 8) TRACE_CLK(p.status, 18 + it);
                }
                if (!ok) break;
                for (int lr = 0; lr < p.lr_chunks; ++lr, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(sfready_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    const uint64_t adesc = umma_desc_sw128(st);
                    const uint64_t bdesc = umma_desc_sw128(st + A_BYTES);
                    if (!elect_one()) continue;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if constexpr (PAIR) umma_bf16_pair(d, adesc + 2 * k, bdesc + 2 * k, idesc_bf, 1u);
                        else umma_bf16(d, adesc + 2 * k, bdesc + 2 * k, idesc_bf, 1u);
                    }
                    if constexpr (PAIR) umma_commit_pair(empty_bar(s), 3);
                    else umma_commit(empty_bar(s));
                }
                if (ok && elect_one()) {
                    if constexpr (PAIR) umma_commit_pair(tfull_bar(acc), 3);  // both CTAs' epilogue warps
                    else umma_commit(tfull_bar(acc));
                }
            }
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ scale-factor copier
        // A tcgen05.cp occupies the issuing thread for roughly a hundred cycles.  With the eight copies of a k-block on
        // the MMA thread, that thread bounded the kernel (0.137 ms on the 4608 x 3072 -> 9216 layer; 0.112 ms with one
        // copier thread, itself the bound; 0.093 ms with two).  Each copier hands its half of a stage over through an
        // mbarrier that tcgen05.commit arrives on once the copies have landed in tensor memory.
        {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step) {
                const int items = p.num_kb + p.lr_chunks;
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_UNPACK)) { ok = false; break; }
                    if constexpr (PAIR) {
                        if (cta_rank != 0) {
                            // this CTA's stage has landed: one word to the leader, whose copiers and MMA thread act for both
                            if (warp == 2 && elect_one()) mbar_arrive_cluster(map_to_cta(peer_bar(s), 0));
                            continue;
                        }
                        if (!mbar_wait(peer_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_UNPACK)) { ok = false; break; }
                    }
                    if (i < p.num_kb) {
                        tc_fence_after_sync();
                        const uint32_t sf = smem_base + s * STAGE_BYTES + A_BYTES + B_BYTES;
                        const uint32_t tsf = tmem_base + TMEM_SF_BASE + s * SF_COLS;
                        if (!elect_one()) continue;
                        if (warp == 2 && it >= 6 && it <= 8) TRACE_CLK(p.status, 6 + it);
                        if (warp == 2) {
                            // activation scales: the four K = 64 steps of the k-block, 4 columns each
#pragma unroll
                            for (int a = 0; a < 4; ++a) {
                                if constexpr (PAIR) tmem_cp_32x128b_warpx4_pair(tsf + 4 * a, sf_desc(sf + a * 512));
                                else tmem_cp_32x128b_warpx4(tsf + 4 * a, sf_desc(sf + a * 512));
                            }
                        } else {
                            // weight scales: per K step, the tile's 128-column blocks side by side (4 columns each)
#pragma unroll
                            for (int a = 0; a < 4; ++a)
#pragma unroll
                                for (int b = 0; b < NB; ++b) {
                                    if constexpr (PAIR)
                                        tmem_cp_32x128b_warpx4_pair(tsf + 16 + 4 * NB * a + 4 * b, sf_desc(sf + (1 + b) * SF_BYTES + a * 512));
                                    else
                                        tmem_cp_32x128b_warpx4(tsf + 16 + 4 * NB * a + 4 * b, sf_desc(sf + (1 + b) * SF_BYTES + a * 512));
                                }
                        }
                        if constexpr (PAIR) umma_commit_pair(sfready_bar(s), 1);  // the leader's barrier only
                        else umma_commit(sfready_bar(s));
                        if (it >= 6 && it <= 8) TRACE_CLK(p.status, (warp == 2 ? 9 : 12) + it);
                    } else if (elect_one()) {
                        mbar_arrive(sfready_bar(s));  // a rank-r chunk: nothing to copy
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 4..11)
        // warp % 4 selects the TMEM lane quadrant (32 token rows), the warpgroup the half of the tile's columns.  The
        // whole slice of the accumulator is read into registers first and the accumulator handed back at once, so that
        // the conversion and the stores overlap the next tile's MMAs even where there is a single accumulator.
        constexpr int HB = BN / 2;
        const int q = warp & 3;
        const int half = (warp - 4) >> 2;
        uint32_t tcount = 0;
        bool ok = true;
        const float out_scale = __ldg(p.out_scale);
        for (int tile = tile_first; ok && tile < num_tiles; tile += tile_step, ++tcount) {
            const int m0 = (tile % num_m_blocks) * TILE_ROWS + (PAIR ? static_cast<int>(cta_rank) * BM : 0);
            const int n0 = (tile / num_m_blocks) * BN;
            const uint32_t acc = tcount % ACC_BUFS;
            // The tile's bias goes to shared memory while its MMAs are still running (two buffers: a warp can be one tile
            // ahead of the others).  The reducing barrier orders the stores before the reads below and makes the eight
            // warps agree on whether to go on: a plain barrier behind a bounded wait could strand a warp.
            float* s_b = reinterpret_cast<float*>(smem_gen + BIAS_OFFSET) + (tcount & 1) * BN;
            {
                const int e = threadIdx.x - 128;  // 0..255
                if (e < BN) s_b[e] = n0 + e < p.N ? __ldg(p.bias + n0 + e) : 0.f;
            }
            const bool mine = mbar_wait(tfull_bar(acc), (tcount / ACC_BUFS) & 1, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
            uint32_t any_failed;
            asm volatile(
                "{\n\t"
                ".reg .pred pin, pout;\n\t"
                "setp.eq.u32 pin, %1, 0;\n\t"
                "bar.red.or.pred pout, 1, 256, pin;\n\t"
                "selp.u32 %0, 1, 0, pout;\n\t"
                "}\n"
                : "=r"(any_failed)
                : "r"(static_cast<uint32_t>(mine))
                : "memory");
            ok = any_failed == 0;
            if (!ok) break;
            tc_fence_after_sync();
            const int row = m0 + q * 32 + lane;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * BN + half * HB;
            uint32_t raw[HB / 32][32];
            if (warp == 4 && lane == 0 && tcount == 0) TRACE_CLK(p.status, 27);
            if (warp == 4 && lane == 0 && tcount >= 1 && tcount <= 2) TRACE_CLK(p.status, 3 * tcount - 2);
#pragma unroll
            for (int c = 0; c < HB / 32; ++c) tmem_ld_32x32b_x32(taddr + c * 32, raw[c]);
            tmem_ld_wait();
            tc_fence_before_sync();
            if (warp == 4 && lane == 0 && tcount == 0) TRACE_CLK(p.status, 28);
            if (warp == 4 && lane == 0 && tcount >= 1 && tcount <= 2) TRACE_CLK(p.status, 3 * tcount - 1);
            // every lane arrives for itself: a warp barrier followed by one elected lane's arrival costs about a hundred cycles more
            if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));  // the leader's barrier
            else mbar_arrive(tempty_bar(acc));
            if constexpr (P::STAGED_OUT) {
                // Outputs leave through shared memory: a thread holds one token row, so direct stores would be 32 scattered
                // 16-byte pieces per instruction, and a clock trace showed 7600-9500 cycles of them per tile, during which
                // the next tile's operand loads ran at half their rate.  Each warp converts 64 columns of its 32 rows into
                // its own staging tile (128-byte swizzle: a quarter-warp's pieces fall into different banks) and one lane
                // hands the tile to a TMA store, which writes whole lines and clips at M and N.
                const float* bq = s_b + half * HB;
                const uint32_t sbuf = smem_base + P::STORE_OFFSET + static_cast<uint32_t>(warp - 4) * 4096u;
                const int row0 = m0 + q * 32;
#pragma unroll
                for (int cc = 0; cc < HB / 64; ++cc) {
                    if (lane == 0) bulk_wait_group_read_all();  // the tile's previous contents have been read
                    __syncwarp();
#pragma unroll
                    for (int p8 = 0; p8 < 8; ++p8) {
                        const int c = cc * 2 + (p8 >> 2), j = (p8 & 3) * 8;
                        const float4 b0 = *reinterpret_cast<const float4*>(bq + c * 32 + j);
                        const float4 b1 = *reinterpret_cast<const float4*>(bq + c * 32 + j + 4);
                        uint4 o;
                        o.x = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 0]), out_scale, b0.x), fmaf(__uint_as_float(raw[c][j + 1]), out_scale, b0.y));
                        o.y = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 2]), out_scale, b0.z), fmaf(__uint_as_float(raw[c][j + 3]), out_scale, b0.w));
                        o.z = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 4]), out_scale, b1.x), fmaf(__uint_as_float(raw[c][j + 5]), out_scale, b1.y));
                        o.w = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 6]), out_scale, b1.z), fmaf(__uint_as_float(raw[c][j + 7]), out_scale, b1.w));
                        const uint32_t dst = sbuf + static_cast<uint32_t>(lane) * 128u + (static_cast<uint32_t>(p8 ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w) : "memory");
                    }
                    fence_proxy_async_smem();  // these writes -> visible to the copy engine
                    __syncwarp();
                    const int col0 = n0 + half * HB + cc * 64;
                    if (lane == 0 && row0 < p.M && col0 < p.N) {
                        tma_store_2d(&tmap_y, sbuf, col0, row0);
                        bulk_commit_group();
                    }
                }
            } else if (row < p.M) {
                const float* bq = s_b + half * HB;
                uint16_t* yrow = p.y + static_cast<size_t>(row) * p.N + n0 + half * HB;
#pragma unroll
                for (int c = 0; c < HB / 32; ++c) {
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        if (n0 + half * HB + c * 32 + j < p.N) {
                            const float4 b0 = *reinterpret_cast<const float4*>(bq + c * 32 + j);
                            const float4 b1 = *reinterpret_cast<const float4*>(bq + c * 32 + j + 4);
                            uint4 o;
                            o.x = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 0]), out_scale, b0.x), fmaf(__uint_as_float(raw[c][j + 1]), out_scale, b0.y));
                            o.y = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 2]), out_scale, b0.z), fmaf(__uint_as_float(raw[c][j + 3]), out_scale, b0.w));
                            o.z = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 4]), out_scale, b1.x), fmaf(__uint_as_float(raw[c][j + 5]), out_scale, b1.y));
                            o.w = pack_bf16x2(fmaf(__uint_as_float(raw[c][j + 6]), out_scale, b1.z), fmaf(__uint_as_float(raw[c][j + 7]), out_scale, b1.w));
                            *reinterpret_cast<uint4*>(yrow + c * 32 + j) = o;
                        }
                    }
                }
            }
            if (warp == 4 && lane == 0 && tcount == 0) TRACE_CLK(p.status, 29);
            if (warp == 4 && lane == 0 && tcount >= 1 && tcount <= 2) TRACE_CLK(p.status, 3 * tcount);
        }
        if constexpr (P::STAGED_OUT) {
            if (lane == 0) bulk_wait_group_all();  // this warp's stores are performed before the CTA leaves
        }
    }

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

template <int BN, bool PAIR = false>
static dirotq_status_t launch_nvfp4_gemm_bn(const dirotq_layer* L, const Nvfp4GemmArgs& a, cudaStream_t stream) {
    const Geometry& g = L->geo;
    CUtensorMap tmap_codes, tmap_xh;
    dirotq_status_t st;
    st = encode_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.codes, (uint64_t)g.K4 / 2, (uint64_t)a.M,
                        (uint64_t)g.K4 / 2, 128, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    st = encode_tmap_2d(&tmap_xh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.xh, (uint64_t)g.r_pad, (uint64_t)a.M,
                        (uint64_t)g.r_pad * 2, 64, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    NvKernelParams p;
    p.M = a.M; p.N = g.N;
    p.num_kb = (g.K4 + BKE - 1) / BKE;
    p.nkb64p = g.nkb64p;
    p.lr_chunks = g.r_pad / 64;
    p.xsf = a.xsf;
    p.wsf = reinterpret_cast<const uint8_t*>(L->blob + L->lay.off_wscale);
    p.bias = reinterpret_cast<const float*>(L->blob + L->lay.off_bias);
    p.out_scale = reinterpret_cast<const float*>(L->blob + L->lay.off_meta);
    p.y = a.y; p.status = a.status;
    const int sms = sm_count(L->device);
    static SmemOptIn<1> opt_in;  // one per instantiation of this launcher
    if (!opt_in.ensure(nvfp4_gemm_kernel<BN, PAIR>, 0, L->device, Plan<BN, PAIR>::SMEM_BYTES)) return DIROTQ_ERR_CUDA;
    // the weight-side tensor maps have 128-row boxes: a 256-column tile fetches two of them per operand (one per CTA of a pair)
    cudaError_t err;
    // where the outputs leave as TMA stores: boxes of 32 rows x 64 columns (128-byte swizzle in shared memory)
    CUtensorMap tmap_y = tmap_xh;  // (unused by the plan that stores directly)
    if constexpr (Plan<BN, PAIR>::STAGED_OUT) {
        st = encode_tmap_2d(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.y, (uint64_t)g.N, (uint64_t)a.M, (uint64_t)g.N * 2, 64, 32,
                            CU_TENSOR_MAP_SWIZZLE_128B);
        if (st != DIROTQ_OK) return st;
    }
    if constexpr (PAIR) {
        const int pair_tiles = ((a.M + 2 * BM - 1) / (2 * BM)) * ((g.N + BN - 1) / BN);
        const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
        err = launch_kernel_pairs(nvfp4_gemm_kernel<BN, PAIR>, 2 * pairs, NUM_THREADS, Plan<BN, PAIR>::SMEM_BYTES, stream, true,
                                  tmap_codes, L->tmap_wpacked, tmap_xh, L->tmap_wh, tmap_y, p);
    } else {
        const int num_tiles = ((a.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
        const int grid = num_tiles < sms ? num_tiles : sms;
        err = launch_kernel(nvfp4_gemm_kernel<BN>, grid, NUM_THREADS, Plan<BN>::SMEM_BYTES, stream, true,
                            tmap_codes, L->tmap_wpacked, tmap_xh, L->tmap_wh, tmap_y, p);
    }
    return err == cudaSuccess ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

static std::atomic<int> g_nv_tile_columns{0};  // 0: chosen per call; 128 / 256: forced

}  // namespace

dirotq_status_t set_nvfp4_tile_columns(int columns) {  // 512: 256 columns per pair of CTAs
    if (columns != 0 && columns != 128 && columns != 256 && columns != 512) return DIROTQ_ERR_INVALID_ARG;
    g_nv_tile_columns.store(columns);
    return DIROTQ_OK;
}

dirotq_status_t launch_nvfp4_gemm(const dirotq_layer* L, const Nvfp4GemmArgs& a, cudaStream_t stream) {
    // A 128-column tile takes about 0.6 of the time of a 256-column one (measured), so the narrow plan is chosen only
    // when it fills the SMs so much better that it wins anyway (few tiles, or a nearly empty last wave).
    const int forced = g_nv_tile_columns.load();
    const int sms = sm_count(L->device);
    const long m_blocks = (a.M + BM - 1) / BM;
    const long t_wide = m_blocks * ((L->geo.N + 255) / 256), t_narrow = m_blocks * ((L->geo.N + 127) / 128);
    const double cost_wide = static_cast<double>((t_wide + sms - 1) / sms);
    const double cost_narrow = 0.6 * static_cast<double>((t_narrow + sms - 1) / sms);
    // CTA pairs (256 token rows x 256 columns per cluster of two) do two wide tiles' work in about 0.9 of a wide tile's
    // time (measured on the FLUX shapes at M = 4608: 0.078 -> 0.071, 0.033 -> 0.031, 0.106 -> 0.094, 0.078 -> 0.070 ms), on
    // half as many schedulable units; same bits as the other plans
    const int pair_units = sms / 2;
    const long t_pair = ((a.M + 2 * BM - 1) / (2 * BM)) * ((L->geo.N + 255) / 256);
    const double cost_pair = a.M > BM ? 0.9 * static_cast<double>((t_pair + pair_units - 1) / pair_units) : 1e30;
    if (forced == 512 || (forced == 0 && cost_pair < 0.98 * cost_wide && cost_pair < 0.98 * cost_narrow))
        return launch_nvfp4_gemm_bn<256, true>(L, a, stream);
    const bool wide = forced ? forced == 256 : !(cost_narrow < 0.98 * cost_wide);
    return wide ? launch_nvfp4_gemm_bn<256>(L, a, stream) : launch_nvfp4_gemm_bn<128>(L, a, stream);
}

}  // namespace dirotq
