// Kernels (b)+(c): W4A4 group GEMM with per-group rescale, bf16 rank-r branch and bias.
//
//   y[m,n] = bf16( sum_g s_x[m,g] s_w[g,n] P_g[m,n]  +  sum_{i<r} x~_h[m,i] W~_h[i,n]  +  bias[n] )
//   P_g[m,n] = sum_{j in group g} q_x[m,j] q_w[j,n]                              (paper Eq. 5)
//
// sm_100a has no INT4 MMA, and an int32 accumulator costs a conversion per element and group before it
// can be scaled.  The integer products are therefore computed EXACTLY on the 8-bit float path
// (tcgen05.mma kind::f8f6f4, E4M3 operands, fp32 accumulation):
//   * an E4M3 byte s0000mmm is (-1)^s m * 2^-9 for m = 0..7 (subnormals; with a fourth magnitude bit, 0..15: the
//     first binade continues the same line), so a code stored as sign + magnitude IS an E4M3 number;
//   * activation codes arrive from kernel (a) one per byte in that form: q_x * 2^-9 (the asymmetric variant
//     stores u = 0..15 as 0000uuuu = u * 2^-9);
//   * weight codes stay packed (two per byte: sign + 3-bit magnitude each) in HBM and in the TMA staging
//     buffer; two "unpack" warps split every 32-bit word of eight codes into two words of four bytes
//     s0000mmm = q_w * 2^-9 (one mask, one rotate and one mask: the nibble order of prepare.cu is chosen for
//     that) in the 128-byte-swizzled layout the MMA reads;
//   * every product is an integer times 2^-18 and a group's sum is below 2^24 in magnitude, so the fp32
//     accumulator holds S_g = 2^-18 P_g without rounding.  The weight scales are stored as 2^18 s_w (exact), so
//         t = s_x * (2^18 s_w)            -- exact: two bf16-valued factors and a power of two --
//         acc = fma(S_g, t, acc)          -- one rounding per element and group --
//     folds a group in with one (packed, two columns at a time) multiply and one fused multiply-add per element and
//     no integer conversion.
// The exactness of the accumulation is a property of the tensor core that the parity tests pin: the
// group sums exported by the debug entry equal the CPU checker's int32 sums bit for bit, on random
// codes and on patterns built to lose low bits (long runs of +-49 followed by +-1).
//
// Every K-group gets its own accumulator tile in tensor memory (two tiles, ping-pong): the MMA warp
// fills tile g%2 while the epilogue warps drain tile (g-1)%2 into per-thread fp32 accumulators.  The
// bf16 rank-r branch is issued as one more "group" (kind::f16 into the same ping-pong tile) and added
// unscaled.
//
// Roles (384 threads = 3 warpgroups):
//   warpgroup 0: warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2-3 nibble -> byte unpack
//   warpgroups 1-2: epilogue; warp%4 selects the TMEM lane quadrant (token rows), the warpgroup
//                   selects the half of the tile's columns.
#include "common.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

#include <atomic>

namespace dirotq {
namespace {

constexpr int BM = 128;
constexpr int BKC = 128;  // one-byte codes per k-block (128-byte rows)
constexpr int A_BYTES = BM * BKC;          // 16 KB  activation codes / bf16 x~_h chunk
constexpr uint32_t kSignMag = 0x87878787u;  // sign and 3-bit magnitude of four one-byte codes
constexpr float kAccUnit = kI8Path ? 1.0f : kWScaleFold;  // integer group sum = accumulator value x this

// Plan for tiles of BN output columns.
//   256: two epilogue warpgroups, 128 columns (128 fp32 accumulators) per thread; an accumulator tile can only be read in
//        pieces between the arithmetic and is held for three quarters of a group.
//   192: three epilogue warpgroups, 64 columns per thread: a thread's share of an accumulator tile fits its two chunk
//        buffers, so the tile goes back to the tensor core after the first quarter of a group, and three warps per scheduler
//        hide each other's waits.  16 warps: 152 registers for the epilogue threads, 56 for the others.
//   128: two warpgroups, 64 columns per thread, four accumulator tiles; for layers whose wider tiles would leave SMs idle.
//    64: one warpgroup, 64 columns per thread, four accumulator tiles, seven stages; for calls with so few token rows that
//        even 128-column tiles occupy a fraction of the SMs: there a tile's K-groups are a chain of hand-overs between the
//        tensor core and the epilogue, whose length does not depend on the tile's width, so more, narrower tiles on more SMs
//        shorten the call.  256 threads, no register re-partitioning (every thread may use 255).
//    64 + SPLITK: clusters of up to four CTAs cut the K-groups of one 128 x 64 tile into contiguous ranges; each CTA rescales its
//        range into its own fp32 accumulators, the others store theirs into the last CTA's shared memory (distributed shared
//        memory, one cluster-scope barrier), and that CTA adds them in rank order, adds the rank-r branch and the bias, and
//        stores.  For calls so small that the chain of K-groups per tile, not the number of tiles, sets the time.
constexpr int SPLIT_MAX = 4;          // CTAs per cluster of the split plan
constexpr int RED_BYTES = 128 * 64 * 4;  // one CTA's partial tile: 128 rows x 64 columns fp32
template <int BN, bool SPLITK = false>
struct Plan {
    static constexpr int EPI_WG = BN == 192 ? 3 : BN == 64 ? 1 : 2;  // epilogue warpgroups
    static constexpr int EPI_WARPS = 4 * EPI_WG;
    static constexpr int THREADS = 128 + 128 * EPI_WG;
    static constexpr bool REPARTITION = EPI_WG > 1;            // setmaxnreg after the role split
    static constexpr int EPI_REGS = EPI_WG == 3 ? 152 : 216;  // setmaxnreg budgets: 128 * AUX + 128 * EPI_WG * EPI <= 65536
    static constexpr int AUX_REGS = EPI_WG == 3 ? 56 : 64;
    static constexpr int SC_SLOTS = BN == 192 ? 6 : 8;
    static constexpr int STAGES = BN == 256 ? 3 : BN == 192 ? 4 : BN == 128 ? 5 : SPLITK ? 3 : 7;
    static constexpr int BU_BYTES = BN * BKC;         // unpacked weight codes / bf16 W~_h chunk (32 KB at BN = 256)
    static constexpr int BP_BYTES = BN * BKC / 2;     // packed weight codes (TMA staging)
    static constexpr int STAGE_BYTES = A_BYTES + BU_BYTES + BP_BYTES;  // 64 KB / 40 KB
    static constexpr int SC_SW_BYTES = 2 * BN * 4;    // up to two groups per k-block
    static constexpr int SC_SX_BYTES = 2 * BM * 4;    // activation scales of up to two groups
    static constexpr int SC_BYTES = SC_SW_BYTES + SC_SX_BYTES;  // 3 KB / 2 KB
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES + SC_SLOTS * SC_BYTES;
    static constexpr int RED_OFFSET = BAR_OFFSET + 512;  // split plan: the other CTAs' partial tiles land here (last CTA)
    static constexpr int SMEM_BYTES = BAR_OFFSET + 512 + 1024 + (SPLITK ? (SPLIT_MAX - 1) * RED_BYTES : 0);
    static_assert(!SPLITK || BN == 64, "the split plan has 64-column tiles");
};
static_assert(Plan<64, true>::SMEM_BYTES <= 232448, "shared memory plan too large");
static_assert(Plan<256>::SMEM_BYTES <= 232448 && Plan<192>::SMEM_BYTES <= 232448 && Plan<128>::SMEM_BYTES <= 232448, "shared memory plan too large");
static_assert(Plan<128>::STAGE_BYTES % 1024 == 0 && Plan<128>::SC_BYTES % 128 == 0, "tile alignment");
static_assert(Plan<192>::STAGE_BYTES % 1024 == 0 && Plan<192>::SC_BYTES % 128 == 0, "tile alignment");
static_assert(Plan<64>::SMEM_BYTES <= 232448 && Plan<64>::STAGE_BYTES % 1024 == 0 && Plan<64>::SC_BYTES % 128 == 0, "tile alignment");
static_assert(8 * (3 * Plan<128>::STAGES + 2 * 8 + 9) <= 400 && 8 * (3 * Plan<192>::STAGES + 2 * 6 + 9) <= 400 &&
              8 * (3 * Plan<64>::STAGES + 2 * 8 + 9) <= 400, "barriers end below the words at +400");

struct GemmKernelParams {
    int M, N, n_g, num_kb, lr_chunks;
    const float* bias;
    uint16_t* y;
    int32_t* partials;
    int* status;
};

// Wait accounting (diagnostics): cycles a role spends blocked on each kind of barrier are summed into
// 64-bit counters that follow the status word in the workspace (8-byte slots 1..8, see WaitSlot).
enum WaitSlot : int { WS_PROD_EMPTY = 1, WS_MMA_OPERANDS = 2, WS_MMA_TEMPTY = 3, WS_UNPACK_FULL = 4, WS_EPI_TFULL = 5,
                      WS_EPI_SCALES = 6, WS_EPI_TOTAL = 7, WS_KERNEL = 8 };

__device__ __forceinline__ bool timed_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int code,
                                           long long& acc) {
    if (mbar_try_wait(bar, parity)) return true;  // the common case costs no clock reads
    const long long t0 = clock64();
    const bool ok = mbar_wait(bar, parity, abort_flag, status, code);
    acc += clock64() - t0;
    return ok;
}

__device__ __forceinline__ void flush_wait(int* status, int slot, long long cycles) {
    atomicAdd(reinterpret_cast<unsigned long long*>(status) + slot, static_cast<unsigned long long>(cycles));
}

// Two fp32 values in one 64-bit register pair (sm_100 has packed fp32 arithmetic on such pairs).
__device__ __forceinline__ uint64_t pack_u32x2(uint32_t lo, uint32_t hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) { return pack_u32x2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {  // round to nearest even, per element
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Four weight codes as the bytes the MMA reads: the sign-magnitude bytes themselves (E4M3 path) or, in the integer-path
// build, their two's complement (per byte: (m ^ s) - s with s = 0xFF where the sign bit is set).
__device__ __forceinline__ uint32_t code_bytes(uint32_t v) {
    if constexpr (!kI8Path) {
        return v;
    } else {
        const uint32_t sg = ((v >> 7) & 0x01010101u) * 0xFFu;
        return __vsub4((v & 0x07070707u) ^ sg, sg);
    }
}

__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {  // round to nearest even, per element
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int G, bool kPartials, int BN, bool SPLITK = false>
__global__ void __launch_bounds__(Plan<BN>::THREADS, 1)
w4a4_gemm_kernel(const __grid_constant__ CUtensorMap tmap_codes, const __grid_constant__ CUtensorMap tmap_wpacked,
                 const __grid_constant__ CUtensorMap tmap_wscale, const __grid_constant__ CUtensorMap tmap_xscale,
                 const __grid_constant__ CUtensorMap tmap_xh, const __grid_constant__ CUtensorMap tmap_wh,
                 const GemmKernelParams p) {
    using P = Plan<BN, SPLITK>;
    static_assert(!SPLITK || !kPartials, "the debug export runs unsplit");
    constexpr int STAGES = P::STAGES, STAGE_BYTES = P::STAGE_BYTES, BU_BYTES = P::BU_BYTES, BP_BYTES = P::BP_BYTES;
    constexpr int SC_SW_BYTES = P::SC_SW_BYTES, SC_BYTES = P::SC_BYTES, BAR_OFFSET = P::BAR_OFFSET;
    constexpr int SC_SLOTS = P::SC_SLOTS, NUM_EPI_WARPS = P::EPI_WARPS;
    constexpr int HB = BN / P::EPI_WG;  // columns per epilogue warp: the warpgroup selects the slice of the tile
    constexpr int CHUNKS = HB / 32;    // 32-column chunks per epilogue warp and accumulator tile
    constexpr int GPK = BKC / G;       // groups per k-block: 2 (G = 64) or 1 (G = 128)
    constexpr int MMA_PER_G = G / 32;  // 8-bit MMA instructions (K = 32) per group
    constexpr int NBUF = BN == 64 ? 4 : 512 / BN;  // accumulator tiles in tensor memory: 2 of 256 columns, 4 of 128 or of 64 (the barrier map has four slots)

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sc_base = smem_base + STAGES * STAGE_BYTES;
    const uint32_t bar_base = smem_base + BAR_OFFSET;
    // barriers: full[S], unpacked[S], empty[S], sc_full[SC], sc_empty[SC], tmem_full[NBUF], tmem_empty[NBUF]
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto unp_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto empty_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
    auto scfull_bar = [&](int s) { return bar_base + 8u * (3 * STAGES + s); };
    auto scempty_bar = [&](int s) { return bar_base + 8u * (3 * STAGES + SC_SLOTS + s); };
    auto tfull_bar = [&](int a) { return bar_base + 8u * (3 * STAGES + 2 * SC_SLOTS + a); };
    auto tempty_bar = [&](int a) { return bar_base + 8u * (3 * STAGES + 2 * SC_SLOTS + 4 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + BAR_OFFSET + 400);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + BAR_OFFSET + 404);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Trace build (TRACE_CLK): slot 9 entry, 10 set-up done, 11 previous grid ended, 12 / 13 producer has issued its first k-block /
    // everything, 14 / 15 first unpack warp sees / has expanded the first stage, 16 / 17 / 18 MMA warp starts the first / fifth / last
    // k-block, 19 it has committed the last tile, 20 first epilogue warp sees its first accumulator, 21 starts its ninth K-group, 22 has
    // folded in the last group, 23 the rank-r tile, 24 has stored its last outputs.
    if (threadIdx.x == 0) TRACE_CLK(p.status, 9);

    const int num_m_blocks = (p.M + BM - 1) / BM;
    const int num_n_blocks = (p.N + BN - 1) / BN;
    const int num_tiles = num_m_blocks * num_n_blocks;
    // Split plan: this CTA's range of k-blocks [kb0, kb1) and of K-groups [g0, g1) of the cluster's tile (the first ranks take
    // one k-block more when the division leaves a rest); the LAST rank gathers the partial tiles and has the rank-r branch.
    // (Without the split every one of these is the constant or the parameter it stands for.)
    const uint32_t csize = SPLITK ? cluster_nctarank() : 1u, crank = SPLITK ? cluster_ctarank() : 0u;
    const bool gathers = !SPLITK || crank == csize - 1;
    const int split_base = SPLITK ? p.num_kb / static_cast<int>(csize) : 0, split_rest = SPLITK ? p.num_kb % static_cast<int>(csize) : 0;
    const int kb0 = SPLITK ? static_cast<int>(crank) * split_base + min(static_cast<int>(crank), split_rest) : 0;
    const int kb1 = SPLITK ? kb0 + split_base + (static_cast<int>(crank) < split_rest ? 1 : 0) : p.num_kb;
    const int g0 = SPLITK ? kb0 * GPK : 0, g1 = SPLITK ? min(kb1 * GPK, p.n_g) : p.n_g;
    const int lr_here = gathers ? p.lr_chunks : 0;
    // (tile loops read these where they are needed, like blockIdx.x and gridDim.x themselves: held in registers across the
    // roles' loops they cost the 256-column plan spills)
    auto first_tile = [&]() { return SPLITK ? static_cast<int>(blockIdx.x / csize) : static_cast<int>(blockIdx.x); };
    auto tile_stride = [&]() { return SPLITK ? static_cast<int>(gridDim.x / csize) : static_cast<int>(gridDim.x); };
    const uint32_t red_bar = bar_base + 8u * (3 * STAGES + 2 * SC_SLOTS + 9);  // split plan: "partial tiles landed" (last CTA)

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(unp_bar(s), 64);  // every thread of the two unpack warps arrives for itself
            mbar_init(empty_bar(s), 1);
        }
        for (int s = 0; s < SC_SLOTS; ++s) {
            mbar_init(scfull_bar(s), 1);
            mbar_init(scempty_bar(s), NUM_EPI_WARPS * 32);
        }
        for (int a = 0; a < NBUF; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), NUM_EPI_WARPS * 32);
        }
        mbar_init(bar_base + 8u * (3 * STAGES + 2 * SC_SLOTS + 8), 1);  // spare: see umma_drain
        if constexpr (SPLITK) {
            mbar_init(red_bar, 1);  // counts the bytes of the other CTAs' partial tiles
            mbar_init(red_bar + 8u, 128);  // this CTA's partial tile is in its shared memory (every epilogue thread arrives)
            if (gathers) mbar_arrive_expect_tx(red_bar, (csize - 1) * RED_BYTES);
        }
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap_codes);
        tma_prefetch_desc(&tmap_wpacked);
        tma_prefetch_desc(&tmap_wscale);
        tma_prefetch_desc(&tmap_xscale);
        tma_prefetch_desc(&tmap_xh);
        tma_prefetch_desc(&tmap_wh);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (SPLITK) cluster_sync_all();  // the gathering CTA's barrier is initialised before anything arrives on it
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's own shared and tensor memory; what follows reads the first kernel's output
    if (threadIdx.x == 0) TRACE_CLK(p.status, 10);
    grid_dependency_wait();
    if (threadIdx.x == 0) TRACE_CLK(p.status, 11);
    // the next layer's first kernel may be scheduled as this grid's CTAs leave their SMs (it waits for this whole grid)
    grid_launch_dependents();

    if (warp < 4) {
        if constexpr (P::REPARTITION) reg_dealloc<P::AUX_REGS>();

        if (warp == 0) {
            // -------------------------------------------------------- TMA producer
            // (the whole warp walks the loops and waits, one elected lane issues: counters, addresses and coordinates stay
            // warp-uniform, which shortens the chain of instructions per stage)
            {
                uint32_t it = 0, sc_it = 0;
                long long w_empty = 0;
                bool ok = true;
                for (int tile = first_tile(); ok && tile < num_tiles; tile += tile_stride()) {
                    const int m0 = (tile % num_m_blocks) * BM;
                    const int n0 = (tile / num_m_blocks) * BN;
                    for (int kb = kb0; kb < kb1; ++kb, ++it, ++sc_it) {
                        const int s = it % STAGES;
                        if (!timed_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER, w_empty)) { ok = false; break; }
                        const uint32_t st = smem_base + s * STAGE_BYTES;
                        if (elect_one()) {
                            mbar_arrive_expect_tx(full_bar(s), A_BYTES + BP_BYTES);
                            tma_load_2d(st, &tmap_codes, full_bar(s), kb * BKC, m0);
                            tma_load_2d(st + A_BYTES + BU_BYTES, &tmap_wpacked, full_bar(s), kb * (BKC / 2), n0);
                        }
                        const int slot = sc_it % SC_SLOTS;
                        if (!mbar_wait(scempty_bar(slot), ((sc_it / SC_SLOTS) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                        const uint32_t sc = sc_base + slot * SC_BYTES;
                        if (elect_one()) {
                            mbar_arrive_expect_tx(scfull_bar(slot), GPK * (BN + BM) * 4);
                            tma_load_2d(sc, &tmap_wscale, scfull_bar(slot), n0, kb * GPK);
                            tma_load_2d(sc + SC_SW_BYTES, &tmap_xscale, scfull_bar(slot), m0, kb * GPK);
                            if (it == 0) TRACE_CLK(p.status, 12);
                        }
                    }
                    if (!ok) break;
                    for (int lr = 0; lr < lr_here; ++lr, ++it) {
                        const int s = it % STAGES;
                        if (!mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                        const uint32_t st = smem_base + s * STAGE_BYTES;
                        if (elect_one()) {
                            mbar_arrive_expect_tx(full_bar(s), A_BYTES + BU_BYTES);
                            tma_load_2d(st, &tmap_xh, full_bar(s), lr * 64, m0);
                            tma_load_2d(st + A_BYTES, &tmap_wh, full_bar(s), lr * 64, n0);
                        }
                    }
                }
                if (lane == 0) TRACE_CLK(p.status, 13);
                if (lane == 0) flush_wait(p.status, WS_PROD_EMPTY, w_empty);
                if (!ok && lane == 0) {
                    const uint32_t first = it > STAGES ? it - STAGES : 0;
                    for (uint32_t j = first; j < it; ++j) {
                        const unsigned long long t0 = globaltimer_ns();
                        while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1) &&
                               globaltimer_ns() - t0 < 100000000ull) {}
                    }
                    const uint32_t sfirst = sc_it > SC_SLOTS ? sc_it - SC_SLOTS : 0;
                    for (uint32_t j = sfirst; j < sc_it; ++j) {
                        const unsigned long long t0 = globaltimer_ns();
                        while (!mbar_try_wait(scfull_bar(j % SC_SLOTS), (j / SC_SLOTS) & 1) &&
                               globaltimer_ns() - t0 < 100000000ull) {}
                    }
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------- MMA issuer
            // One thread, and every instruction it executes waits its turn behind the two epilogue warps of its
            // scheduler, so its loop is kept short: stage index, parities and the operand descriptors are carried
            // along instead of recomputed (a descriptor differs between stages only in the address field of its low
            // word, which cannot overflow: shared-memory addresses have 18 bits, the field holds address / 16).
            // (whole warp in the loops, one elected lane issues, as in the producer)
            {
                constexpr uint32_t idesc_f8 = umma_idesc(1 /*f32*/, 0 /*E4M3*/, BM, BN);
                constexpr uint32_t idesc_i8 = umma_idesc(2 /*s32*/, 1 /*s8*/, BM, BN);  // integer-path build only
                constexpr uint32_t idesc_bf = umma_idesc(1 /*f32*/, 1 /*bf16*/, BM, BN);
                const uint64_t desc0 = umma_desc_sw128(smem_base);
                const uint32_t desc_hi = static_cast<uint32_t>(desc0 >> 32), desc_lo0 = static_cast<uint32_t>(desc0);
                auto desc = [&](uint32_t lo) { return (static_cast<uint64_t>(desc_hi) << 32) | lo; };
                uint32_t s = 0, ph = 0;        // stage of the operand ring and its parity
                uint32_t b = 0, bph = 1;       // accumulator tile and the parity its "empty" barrier is waited with
                long long w_ops = 0, w_tempty = 0;
                const long long t_kernel = clock64();
                bool ok = true;
                for (int tile = first_tile(); ok && tile < num_tiles; tile += tile_stride()) {
                    int groups_left = g1 - g0;
                    for (int kb = kb0; ok && kb < kb1; ++kb) {
                        // the unpack warps arrive after they have seen the stage's loads land (one barrier for both operands), so
                        // their barrier covers the activation codes as well
                        if (!timed_wait(unp_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA, w_ops)) { ok = false; break; }
                        if (lane == 0) { if (kb == kb0) TRACE_CLK(p.status, 16); if (kb == 4) TRACE_CLK(p.status, 17); if (kb == kb1 - 1) TRACE_CLK(p.status, 18); }
                        tc_fence_after_sync();
                        const uint32_t a_lo = desc_lo0 + s * (STAGE_BYTES >> 4), b_lo = a_lo + (A_BYTES >> 4);
#pragma unroll
                        for (int gi = 0; gi < GPK; ++gi) {
                            if (gi < groups_left) {
                                if (!timed_wait(tempty_bar(b), bph, abort_flag, p.status, DEV_TIMEOUT_MMA, w_tempty)) { ok = false; break; }
                                tc_fence_after_sync();
                                if (elect_one()) {
#pragma unroll
                                    for (int k = 0; k < MMA_PER_G; ++k) {
                                        const int kk = gi * MMA_PER_G + k;  // 32-byte step inside the 128-byte row
                                        if constexpr (kI8Path)
                                            umma_i8(tmem_base + b * BN, desc(a_lo + 2 * kk), desc(b_lo + 2 * kk), idesc_i8, k != 0);
                                        else
                                            umma_f8f6f4(tmem_base + b * BN, desc(a_lo + 2 * kk), desc(b_lo + 2 * kk), idesc_f8, k != 0);
                                    }
                                    umma_commit(tfull_bar(b));
                                }
                                if (++b == NBUF) { b = 0; bph ^= 1; }
                            }
                        }
                        if (!ok) break;
                        groups_left -= GPK;
                        if (elect_one()) umma_commit(empty_bar(s));
                        if (++s == STAGES) { s = 0; ph ^= 1; }
                    }
                    if (!ok) break;
                    if (SPLITK && lr_here == 0) continue;  // split plan: only the gathering CTA has the rank-r branch
                    // rank-r bf16 branch: one more accumulator tile, fp32
                    if (!mbar_wait(tempty_bar(b), bph, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                    tc_fence_after_sync();
                    for (int lr = 0; lr < lr_here; ++lr) {
                        if (!mbar_wait(unp_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t a_lo = desc_lo0 + s * (STAGE_BYTES >> 4), b_lo = a_lo + (A_BYTES >> 4);
                        if (elect_one()) {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_bf16(tmem_base + b * BN, desc(a_lo + 2 * k), desc(b_lo + 2 * k), idesc_bf, (lr | k) != 0);
                            umma_commit(empty_bar(s));
                        }
                        if (++s == STAGES) { s = 0; ph ^= 1; }
                    }
                    if (!ok) break;
                    if (elect_one()) umma_commit(tfull_bar(b));
                    if (lane == 0) TRACE_CLK(p.status, 19);
                    if (++b == NBUF) { b = 0; bph ^= 1; }
                }
                if (lane == 0) {
                    flush_wait(p.status, WS_MMA_OPERANDS, w_ops);
                    flush_wait(p.status, WS_MMA_TEMPTY, w_tempty);
                    flush_wait(p.status, WS_KERNEL, clock64() - t_kernel);
                }
            }
        } else {
            // -------------------------------------------------------- nibble -> byte unpack (warps 2, 3)
            const int u = threadIdx.x - 64;  // 0..63
            uint32_t it = 0;
            long long w_full = 0;
            bool ok = true;
            for (int tile = first_tile(); ok && tile < num_tiles; tile += tile_stride()) {
                const int items = (kb1 - kb0) + lr_here;
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % STAGES;
                    ok = timed_wait(full_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_UNPACK, w_full);
                    if (!ok) break;
                    if (it == 0 && u == 0) TRACE_CLK(p.status, 14);
                    if (i < kb1 - kb0) {
                        // 16-byte piece idx = u + 64 j of the packed tile: row = idx/4 = u/4 + 16 j, piece c = u%4.
                        // The swizzle phase row%8 = (u/4)%8 and the piece do not depend on j, so every address is
                        // a per-thread base plus a compile-time offset.
                        uint8_t* st = smem_gen + s * STAGE_BYTES;
                        const uint4* src = reinterpret_cast<const uint4*>(st + A_BYTES + BU_BYTES) + u;
                        const int c = u & 3, sw = (u >> 2) & 7;
                        uint8_t* d0 = st + A_BYTES + (u >> 2) * 128 + (((2 * c) ^ sw) << 4);
                        uint8_t* d1 = st + A_BYTES + (u >> 2) * 128 + (((2 * c + 1) ^ sw) << 4);
                        // The loads of a batch are issued before any of its stores: the compiler cannot prove that the
                        // staging buffer and the operand tile do not overlap, so a load written after a store would wait
                        // for it and the whole unpack would run as one dependent chain.
                        constexpr int PIECES = (BN * 4) / 64, BATCH = PIECES % 8 == 0 ? 8 : 4;
#pragma unroll
                        for (int jb = 0; jb < PIECES; jb += BATCH) {
                            uint4 pk[BATCH];
#pragma unroll
                            for (int j = 0; j < BATCH; ++j) pk[j] = src[64 * (jb + j)];
#pragma unroll
                            for (int j = 0; j < BATCH; ++j) {
                                // a word holds codes k..k+3 in bits 7, 2..0 of its bytes and codes k+4..k+7 four bit
                                // positions further up, wrapping around (see prepare.cu): mask, rotate, mask
                                uint4 o0, o1;
                                o0.x = code_bytes(pk[j].x & kSignMag); o0.y = code_bytes(__funnelshift_r(pk[j].x, pk[j].x, 4) & kSignMag);
                                o0.z = code_bytes(pk[j].y & kSignMag); o0.w = code_bytes(__funnelshift_r(pk[j].y, pk[j].y, 4) & kSignMag);
                                o1.x = code_bytes(pk[j].z & kSignMag); o1.y = code_bytes(__funnelshift_r(pk[j].z, pk[j].z, 4) & kSignMag);
                                o1.z = code_bytes(pk[j].w & kSignMag); o1.w = code_bytes(__funnelshift_r(pk[j].w, pk[j].w, 4) & kSignMag);
                                *reinterpret_cast<uint4*>(d0 + (jb + j) * 2048) = o0;  // 16 rows of 128 bytes further down
                                *reinterpret_cast<uint4*>(d1 + (jb + j) * 2048) = o1;
                            }
                        }
                        fence_proxy_async_smem();  // generic-proxy writes -> visible to the tensor core
                    }
                    // each thread signs off its own writes (a warp-wide barrier followed by one lane's arrival costs about
                    // a hundred cycles more on this part than 32 arrivals)
                    mbar_arrive(unp_bar(s));
                    if (it == 0 && u == 0) TRACE_CLK(p.status, 15);
                }
            }
            if (u == 0) flush_wait(p.status, WS_UNPACK_FULL, w_full);
        }
    } else {
        if constexpr (P::REPARTITION) reg_alloc<P::EPI_REGS>();
        // ------------------------------------------------------------ epilogue (warps 4..11)
        // A warp owns 32 token rows (its TMEM lane quadrant) x BN/2 columns.  The accumulators are read with the
        // 16x256b shape: a thread then holds 4 rows (l/4 + 8 i) x the column pairs 2 (l%4) + {0, 1} of every block
        // of 8 columns, so one load of weight scales serves four rows (with the 32x32b shape, one row per thread,
        // every thread would need all 128 column scales of every group and the shared-memory pipe, not the FMA
        // pipe, would bound the kernel).  A chunk is 32 columns: two .x4 loads (TMEM lanes 0..15 and 16..31 of the
        // quadrant), 32 values per thread, and the 8 weight scales of the thread's columns, which the layer stores
        // side by side (see wscale_index in common.h), in two 16-byte loads.
        //
        // The accumulator tiles of an output tile (one per K-group, then the rank-r one) are one stream: while the
        // last chunk of a tile is folded in, the next tile's barrier is tested (not waited for) and, if it has
        // completed, its first chunk is requested, so that in the steady state neither the hand-over nor the first
        // tensor-memory round trip is paid between groups.
        const int q = warp & 3;
        const int half = (warp - 4) >> 2;
        const int lr4 = lane >> 2;        // row inside a group of 8
        const int lc2 = (lane & 3) * 2;   // first of this thread's two columns inside a block of 8
        uint32_t b = 0, bph = 0;          // accumulator tile read next, parity its "full" barrier is waited with
        uint32_t slot = 0, sph = 0;       // scale slot of the current k-block, parity of its "full" barrier
        long long w_tfull = 0, w_sc = 0;
        const long long t_epi = clock64();
        const uint32_t taddr0 = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + half * HB;
        const float* sc0 = reinterpret_cast<const float*>(smem_gen + STAGES * STAGE_BYTES);
        // No vote after a wait: the warp is converged there, so the barrier test, the abort flag and the clock are read
        // by one instruction for all lanes and every lane gets the same answer.
        bool ok = true;
        uint32_t raw[2][32];  // [0..15]: TMEM lanes 0..15 of the quadrant (rows i = 0, 1), [16..31]: lanes 16..31
        auto request_chunk = [&](uint32_t buf, int c, uint32_t* dst) {
            tmem_ld_16x256b_x4(taddr0 + buf * BN + c * 32, dst);
            tmem_ld_16x256b_x4(taddr0 + buf * BN + (16u << 16) + c * 32, dst + 16);
        };
        auto release_tile = [&](uint32_t buf) {  // every tcgen05.ld of this thread on the tile has completed
            tc_fence_before_sync();
            mbar_arrive(tempty_bar(buf));  // all lanes arrive (see the unpack warps' note on the cost of electing one)
        };
        for (int tile = first_tile(); ok && tile < num_tiles; tile += tile_stride()) {
            const int m0 = (tile % num_m_blocks) * BM;
            const int n0 = (tile / num_m_blocks) * BN;
            const int rbase = m0 + q * 32 + lr4;  // this thread's rows: rbase + 8 i, i = 0..3
            const int colbase = n0 + half * HB;
            uint64_t acc2[HB / 2];  // two adjacent columns per 64-bit register: [(block of 8 columns) * 4 + row i]
#pragma unroll
            for (int j = 0; j < HB / 2; ++j) acc2[j] = 0ull;

            // first scales and first accumulator tile of this output tile (split plan: of this CTA's range, which may be
            // empty, and only the gathering CTA has a rank-r tile)
            if (!SPLITK || g1 > g0) ok = timed_wait(scfull_bar(slot), sph, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE, w_sc);
            if (!SPLITK || g1 > g0 || lr_here > 0) {
                ok = ok && timed_wait(tfull_bar(b), bph, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE, w_tfull);
                if (!ok) break;
                if (warp == 4 && lane == 0) TRACE_CLK(p.status, 20);
                tc_fence_after_sync();
                request_chunk(b, 0, raw[0]);
            }

            for (int g = g0; g < g1; ++g) {
                if (warp == 4 && lane == 0 && g == 8) TRACE_CLK(p.status, 21);
                const int gi = g & (GPK - 1);
                const bool last_of_kb = gi == GPK - 1 || g == p.n_g - 1;
                const float* s_sw = sc0 + slot * (SC_BYTES / 4);
                // the accumulator holds S = 2^-18 P (integer-path build: P as int32, and 2^-18 goes into the token scale)
                float sxv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    sxv[i] = s_sw[2 * BN + gi * BM + q * 32 + lr4 + 8 * i] * (kI8Path ? 1.0f / kWScaleFold : 1.0f);
                uint64_t sx2[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) sx2[i] = pack_f32x2(sxv[i], sxv[i]);
                const ulonglong2* swp = reinterpret_cast<const ulonglong2*>(s_sw + gi * BN + half * HB + 4 * lc2);
                // what comes after this tile: the next group's, or the rank-r tile
                const uint32_t nb = b + 1 == NBUF ? 0 : b + 1, nbph = b + 1 == NBUF ? bph ^ 1 : bph;
                const uint32_t nslot = slot + 1 == SC_SLOTS ? 0 : slot + 1, nsph = slot + 1 == SC_SLOTS ? sph ^ 1 : sph;
                const bool new_scales = last_of_kb && g + 1 < g1;
                const bool more = !SPLITK || g + 1 < g1 || lr_here > 0;  // another accumulator tile follows (always, unless split)
                bool ahead = false;
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint32_t (&cur)[32] = raw[c & 1];
                    // this chunk's weight scales, two adjacent columns per 64-bit register: requested before the wait so
                    // that their latency hides behind it
                    uint64_t w2[4];
                    if constexpr (!kPartials) {
                        const ulonglong2 wa = swp[c * 8], wb = swp[c * 8 + 1];
                        w2[0] = wa.x; w2[1] = wa.y; w2[2] = wb.x; w2[3] = wb.y;
                    }
                    tmem_ld_wait();  // waits for every outstanding load, hence a look-ahead of one chunk
                    tmem_ld_fence(cur);
                    if constexpr (kI8Path) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) cur[i] = __float_as_uint(__int2float_rn(static_cast<int>(cur[i])));  // |P| < 2^24: exact
                    }
                    if (c < CHUNKS - 1) {
                        request_chunk(b, c + 1, raw[(c + 1) & 1]);
                    } else {
                        // the whole tile is in registers: hand it back to the MMA warp, and look at the next one
                        release_tile(b);
                        ahead = more && mbar_test_wait(tfull_bar(nb), nbph) && (!new_scales || mbar_test_wait(scfull_bar(nslot), nsph));
                        if (ahead) {
                            tc_fence_after_sync();
                            request_chunk(nb, 0, raw[0]);  // CHUNKS is even: the last chunk sits in raw[1]
                        }
                    }
                    if constexpr (kPartials) {
                        // unit scales here: 2^18 S = P, an integer
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int cb = 0; cb < 4; ++cb) {
                                const int pidx = 16 * (i >> 1) + 4 * cb + 2 * (i & 1);
                                const int row = rbase + 8 * i;
                                const int col = colbase + c * 32 + cb * 8 + lc2;
                                if (row < p.M && col < p.N)
                                    *reinterpret_cast<int2*>(p.partials + (static_cast<size_t>(g) * p.M + row) * p.N + col) =
                                        make_int2(__float2int_rn(__uint_as_float(cur[pidx]) * kAccUnit),
                                                  __float2int_rn(__uint_as_float(cur[pidx + 1]) * kAccUnit));
                            }
                    } else {
                        // The scale of an element is t = s_x * (2^18 s_w): two bf16-valued factors (and a power of two), so
                        // the fp32 product is EXACT.  It is formed for two adjacent columns at a time with one packed
                        // multiply whose operands are 64-bit registers as they come (the pair of column scales straight
                        // from a shared-memory load, the token's scale duplicated once per group), so no register moves
                        // are spent on packing; then acc = fma(S, t, acc), again packed (the accumulator's two adjacent
                        // columns are consecutive registers of the tensor-memory load): one rounding per element and group,
                        // two instructions per two elements.
#pragma unroll
                        for (int cb = 0; cb < 4; ++cb)
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int pidx = 16 * (i >> 1) + 4 * cb + 2 * (i & 1);
                                const int a = (c * 4 + cb) * 4 + i;
                                acc2[a] = fma_f32x2(pack_u32x2(cur[pidx], cur[pidx + 1]), mul_f32x2(w2[cb], sx2[i]), acc2[a]);
                            }
                    }
                }
                if (last_of_kb) {
                    // this k-block's scales have all been read (the multiply-adds that consumed them were issued above)
                    mbar_arrive(scempty_bar(slot));
                    slot = nslot;
                    sph = nsph;
                }
                b = nb;
                bph = nbph;
                if (!ahead && more) {
                    if (new_scales) ok = timed_wait(scfull_bar(slot), sph, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE, w_sc);
                    ok = ok && timed_wait(tfull_bar(b), bph, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE, w_tfull);
                    if (!ok) break;
                    tc_fence_after_sync();
                    request_chunk(b, 0, raw[0]);
                }
            }
            if (!ok) break;
            if (warp == 4 && lane == 0) TRACE_CLK(p.status, 22);
            // rank-r branch: an fp32 tile whose first chunk is already on its way
            if (!SPLITK || lr_here > 0) {
#pragma unroll
                for (int c = 0; c < CHUNKS; ++c) {
                    uint32_t (&cur)[32] = raw[c & 1];
                    tmem_ld_wait();
                    tmem_ld_fence(cur);
                    if (c < CHUNKS - 1) request_chunk(b, c + 1, raw[(c + 1) & 1]);
                    else release_tile(b);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int cb = 0; cb < 4; ++cb) {
                            const int pidx = 16 * (i >> 1) + 4 * cb + 2 * (i & 1);
                            const int a = (c * 4 + cb) * 4 + i;
                            acc2[a] = add_f32x2(acc2[a], pack_u32x2(cur[pidx], cur[pidx + 1]));
                        }
                }
                if (++b == NBUF) { b = 0; bph ^= 1; }
            }
            if (warp == 4 && lane == 0) TRACE_CLK(p.status, 23);
            if constexpr (SPLITK) {
                // The partial tiles meet in the last CTA of the cluster.  Every other CTA's epilogue threads put their 32
                // register pairs into their own shared memory (the operand ring, idle by now: every MMA of this CTA has
                // completed), word j of thread t at [j][t]; one thread then sends the 32 KB to the gathering CTA with a bulk
                // copy that counts its bytes on that CTA's barrier.  The gathering thread t holds the same rows and columns
                // in every CTA and adds the partial tiles in rank order.
                const uint32_t et = threadIdx.x - 128u;
                const uint32_t red_base = smem_base + P::RED_OFFSET;
                if (!gathers) {
#pragma unroll
                    for (int j = 0; j < HB / 2; ++j) st_shared_u64(smem_base + j * 1024u + et * 8u, acc2[j]);
                    fence_proxy_async_smem();       // these writes -> visible to the copy engine
                    mbar_arrive(red_bar + 8u);
                    if (et == 0 && mbar_wait(red_bar + 8u, 0, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE))  // a bounded wait, like all
                        bulk_copy_to_cluster(map_to_cta(red_base + crank * RED_BYTES, csize - 1), smem_base, RED_BYTES,
                                             map_to_cta(red_bar, csize - 1));
                    continue;  // one tile per cluster: nothing else to do (the cluster meets once more before anyone leaves)
                }
                if (!mbar_wait(red_bar, 0, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE)) { ok = false; break; }
                for (uint32_t r = 0; r + 1 < csize; ++r) {
#pragma unroll
                    for (int j = 0; j < HB / 2; ++j)
                        acc2[j] = add_f32x2(acc2[j], ld_shared_u64(red_base + r * RED_BYTES + j * 1024u + et * 8u));
                }
            }
            if constexpr (!kPartials) {
                // A lane holds 2 of the 8 columns of every block; four blocks are transposed inside the quad of lanes
                // (two exchange steps) so that each lane ends up with all 8 columns = 16 bytes of one block and the
                // warp writes 64 contiguous bytes per row.
                const int j = lane & 3;
#pragma unroll
                for (int m = 0; m < CHUNKS; ++m) {
                    float2 bv[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int col = colbase + (4 * m + t) * 8 + lc2;
                        bv[t] = col < p.N ? __ldg(reinterpret_cast<const float2*>(p.bias + col)) : make_float2(0.f, 0.f);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t v[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            float y_lo, y_hi;
                            unpack_f32x2(acc2[(4 * m + t) * 4 + i], y_lo, y_hi);
                            v[t] = pack_bf16x2(y_lo + bv[t].x, y_hi + bv[t].y);
                        }
                        const bool odd = (j & 1) != 0, upper = (j & 2) != 0;
                        const uint32_t r01 = __shfl_xor_sync(0xffffffffu, odd ? v[0] : v[1], 1);
                        const uint32_t r23 = __shfl_xor_sync(0xffffffffu, odd ? v[2] : v[3], 1);
                        const uint32_t u0 = odd ? r01 : v[0], u1 = odd ? v[1] : r01;  // block (j & 1), lanes 2 (j / 2) + {0, 1}
                        const uint32_t p0 = odd ? r23 : v[2], p1 = odd ? v[3] : r23;  // block 2 + (j & 1)
                        const uint32_t x0 = __shfl_xor_sync(0xffffffffu, upper ? u0 : p0, 2);
                        const uint32_t x1 = __shfl_xor_sync(0xffffffffu, upper ? u1 : p1, 2);
                        const uint4 o = upper ? make_uint4(x0, x1, p0, p1) : make_uint4(u0, u1, x0, x1);  // block j
                        const int row = rbase + 8 * i;
                        const int col = colbase + (4 * m + j) * 8;
                        if (row < p.M && col < p.N)
                            *reinterpret_cast<uint4*>(p.y + static_cast<size_t>(row) * p.N + col) = o;
                    }
                }
            }
        }
        if (warp == 4 && lane == 0) TRACE_CLK(p.status, 24);
        if (warp == 4 && lane == 0) {
            flush_wait(p.status, WS_EPI_TFULL, w_tfull);
            flush_wait(p.status, WS_EPI_SCALES, w_sc);
            flush_wait(p.status, WS_EPI_TOTAL, clock64() - t_epi);
        }
    }

    // ---------------------------------------------------------------- teardown
    if (warp == 1 && lane == 0 && *abort_flag != 0) umma_drain(bar_base + 8u * (3 * STAGES + 2 * SC_SLOTS + 8));  // a wait gave up: let issued MMAs finish first
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (SPLITK) cluster_sync_all();  // no CTA of the cluster leaves while another may still write into it or signal it
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

// A 128-column tile takes 0.70-0.76 of the time of a 256-column one (measured: the activation tile, the rank-r
// branch, the pipeline fill and the per-group hand-over are paid per tile whatever its width), so narrow tiles are
// chosen only when they shorten the schedule by more than that: when the wide tiles' last wave would be nearly
// empty (PixArt-sized layers, N = 1152: 160 wide tiles on 148 SMs) or when there are fewer wide tiles than SMs.
static bool narrow_tiles_pay(int M, int N, int sms) {
    const long m_blocks = (M + BM - 1) / BM;
    const long wide = m_blocks * ((N + 255) / 256), narrow = m_blocks * ((N + 127) / 128);
    const double cost_wide = static_cast<double>((wide + sms - 1) / sms);
    const double cost_narrow = 0.73 * static_cast<double>((narrow + sms - 1) / sms);
    return cost_narrow < 0.98 * cost_wide;
}

// split: 0 = one CTA per tile; 2..SPLIT_MAX = the split plan with clusters of that many CTAs (BN = 64, no debug export)
template <int BN>
static dirotq_status_t launch_w4a4_gemm_bn(const dirotq_layer* L, const GemmArgs& a, cudaStream_t stream, int split = 0) {
    const Geometry& g = L->geo;
    CUtensorMap tmap_codes, tmap_xscale, tmap_xh;
    dirotq_status_t st;
    st = encode_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.codes, (uint64_t)g.K_lp, (uint64_t)a.M,
                        (uint64_t)g.K_lp, BKC, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    st = encode_tmap_2d(&tmap_xscale, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, a.xscale, (uint64_t)a.ldm, (uint64_t)g.n_g,
                        (uint64_t)a.ldm * 4, BM, BKC / g.G, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st != DIROTQ_OK) return st;
    st = encode_tmap_2d(&tmap_xh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.xh, (uint64_t)g.r_pad, (uint64_t)a.M,
                        (uint64_t)g.r_pad * 2, 64, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;

    GemmKernelParams p;
    p.M = a.M; p.N = g.N; p.n_g = g.n_g;
    p.num_kb = (g.K_lp + BKC - 1) / BKC;
    p.lr_chunks = g.r_pad / 64;
    p.bias = reinterpret_cast<const float*>(L->blob + L->lay.off_bias);
    p.y = a.y; p.partials = a.partials; p.status = a.status;

    const int num_tiles = ((a.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
    const int grid = num_tiles < sm_count(L->device) ? num_tiles : sm_count(L->device);
    using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap,
                              const CUtensorMap, const CUtensorMap, const GemmKernelParams);
    KernelFn kern;
    const bool dbg = a.partials != nullptr;
    if (g.G == 64) kern = dbg ? w4a4_gemm_kernel<64, true, BN> : w4a4_gemm_kernel<64, false, BN>;
    else           kern = dbg ? w4a4_gemm_kernel<128, true, BN> : w4a4_gemm_kernel<128, false, BN>;
    static SmemOptIn<4> opt_in;  // one per instantiation of this launcher, i.e. per tile width
    const int vi = (g.G == 64 ? 0 : 2) + (dbg ? 1 : 0);
    if constexpr (BN == 64) {
        if (split >= 2 && !dbg) {
            const KernelFn ks = g.G == 64 ? w4a4_gemm_kernel<64, false, 64, true> : w4a4_gemm_kernel<128, false, 64, true>;
            static SmemOptIn<2> opt_in_split;
            if (!opt_in_split.ensure(ks, g.G == 64 ? 0 : 1, L->device, Plan<64, true>::SMEM_BYTES)) return DIROTQ_ERR_CUDA;
            const cudaError_t es = launch_kernel_clusters(ks, num_tiles * split, split, Plan<64>::THREADS, Plan<64, true>::SMEM_BYTES,
                                                          stream, true, tmap_codes, L->tmap_wpacked64, L->tmap_wscale64, tmap_xscale,
                                                          tmap_xh, L->tmap_wh64, p);
            return es == cudaSuccess ? DIROTQ_OK : DIROTQ_ERR_CUDA;
        }
    }
    if (!opt_in.ensure(kern, vi, L->device, Plan<BN>::SMEM_BYTES)) return DIROTQ_ERR_CUDA;
    const cudaError_t err = launch_kernel(kern, grid, Plan<BN>::THREADS, Plan<BN>::SMEM_BYTES, stream, true, tmap_codes,
                                          BN == 64 ? L->tmap_wpacked64 : BN == 128 ? L->tmap_wpacked128 : BN == 192 ? L->tmap_wpacked192 : L->tmap_wpacked,
                                          BN == 64 ? L->tmap_wscale64 : BN == 128 ? L->tmap_wscale128 : BN == 192 ? L->tmap_wscale192 : L->tmap_wscale,
                                          tmap_xscale, tmap_xh,
                                          BN == 64 ? L->tmap_wh64 : BN == 128 ? L->tmap_wh128 : BN == 192 ? L->tmap_wh192 : L->tmap_wh, p);
    return err == cudaSuccess ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

}  // namespace

static std::atomic<int> g_tile_columns{0};  // 0: chosen per call; 64 / 128 / 192 / 256: forced; 66: 64 columns, split plan where it applies

dirotq_status_t set_w4a4_tile_columns(int columns) {
    if (columns != 0 && columns != 64 && columns != 66 && columns != 128 && columns != 192 && columns != 256) return DIROTQ_ERR_INVALID_ARG;
    g_tile_columns.store(columns);
    return DIROTQ_OK;
}

dirotq_status_t launch_w4a4_gemm(const dirotq_layer* L, const GemmArgs& a, cudaStream_t stream) {
    const int forced = g_tile_columns.load();
    if (forced == 192) return launch_w4a4_gemm_bn<192>(L, a, stream);
    // few token rows: when even 128-column tiles would keep fewer than half of the SMs busy, 64-column tiles on twice as many
    const int sms = sm_count(L->device);
    const long t128 = static_cast<long>((a.M + BM - 1) / BM) * ((L->geo.N + 127) / 128);
    if (forced == 64 || forced == 66 || (forced == 0 && 2 * t128 <= sms)) {
        // The split plan: the largest cluster (4, 3 or 2 CTAs over the k-blocks of a tile) that leaves every CTA at least two
        // k-blocks and whose clusters, one per tile, are all resident at once (asked of the runtime once per device and size).
        // Only on request (knob value 66): the partial tiles are added in another order than one CTA adds the groups, and by
        // default a token's output bits do not depend on how many other tokens the call has.  Measured on the 1152 -> 1152 layer
        // at M = 256: 14.5 against 15.1 us per layer in graph replay.
        int split = 0;
        if (forced == 66 && a.partials == nullptr) {
            const long t64 = static_cast<long>((a.M + BM - 1) / BM) * ((L->geo.N + 63) / 64);
            const int num_kb = (L->geo.K_lp + BKC - 1) / BKC;
            static std::atomic<int> resident[64][SPLIT_MAX + 1];  // 0: not asked yet; else clusters resident at once + 1
            for (int c = SPLIT_MAX; c >= 2 && split == 0; --c) {
                if (num_kb / c < 2) continue;
                const int dev = L->device;
                int have = dev >= 0 && dev < 64 ? resident[dev][c].load() : 0;
                if (have == 0) {
                    // (the question needs the kernel's shared-memory limit raised first; both group sizes have the same footprint)
                    if (cudaFuncSetAttribute(w4a4_gemm_kernel<64, false, 64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Plan<64, true>::SMEM_BYTES) != cudaSuccess) {
                        cudaGetLastError();
                        break;
                    }
                    have = 1 + max_active_clusters(w4a4_gemm_kernel<64, false, 64, true>, c, Plan<64>::THREADS, Plan<64, true>::SMEM_BYTES);
                    if (dev >= 0 && dev < 64) resident[dev][c].store(have);
                }
                if (t64 <= have - 1) split = c;
            }
        }
        return launch_w4a4_gemm_bn<64>(L, a, stream, split);
    }
    const bool narrow = forced ? forced == 128 : narrow_tiles_pay(a.M, L->geo.N, sm_count(L->device));
    return narrow ? launch_w4a4_gemm_bn<128>(L, a, stream) : launch_w4a4_gemm_bn<256>(L, a, stream);
}

}  // namespace dirotq
