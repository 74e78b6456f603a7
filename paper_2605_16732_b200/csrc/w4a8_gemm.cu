// W4A8 variant of the second kernel (paper Sec. 5.1, "INT W4A8": 8-bit activations with one scale per
// token, 4-bit weights with one scale per output column).
//
//   y[m,n] = bf16( s_x[m] s_w[n] P[m,n]  +  sum_{i<r} x~_h[m,i] W~_h[i,n]  +  bias[n] ),
//   P[m,n] = sum_j q_x[m,j] q_w[j,n]                  (int8 x int4, exact in int32)
//
// With one scale per row and per column there is no rescale inside K: the whole contraction runs on
// tcgen05.mma kind::i8 into one int32 accumulator tile and the CUDA cores touch every output once.
// The weight codes stay packed (two per byte, nibble = q + 8) in HBM; TMA lands them in the upper half of
// the operand buffer and four unpack warps expand them in place, turning every nibble into the byte 16 q (shift the nibble into the high half, flip
// bit 7: 16 (q + 8) - 128), so the accumulator holds 16 P and the epilogue shifts it back.
//
// Roles (448 threads): warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2..5 unpack,
// warps 6..13 epilogue (one token row per thread, two warps per lane quadrant).  TMEM: columns 0..255 the int32 tile, 256..511 the
// fp32 tile of the bf16 rank-r branch (kind::f16 cannot accumulate into the integer tile); with 256-column tiles that
// pair fills tensor memory and a tile's epilogue (one pass) is not overlapped with the next tile's MMAs; with 128-column
// tiles two pairs alternate and it is.
#include "common.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

#include <atomic>

namespace dirotq {
namespace {

constexpr int BM = 128;
constexpr int BKC = 128;     // one-byte codes per k-block (128-byte rows)
constexpr int A_BYTES = BM * BKC;       // 16 KB activation codes / bf16 x~_h chunk
constexpr int NUM_THREADS = 448;
constexpr int NUM_UNPACK_WARPS = 4;
constexpr int NUM_EPI_WARPS = 8;  // two per TMEM lane quadrant, half of the tile's columns each

// Shared-memory plan for tiles of BN output columns (256, or 128 where wide tiles would leave SMs idle).
template <int BN>
struct Plan {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int BU_BYTES = BN * BKC;      // unpacked weight codes / bf16 W~_h chunk (32 KB at BN = 256)
    static constexpr int BP_BYTES = BN * BKC / 2;  // packed weight codes: TMA puts them into the UPPER HALF of the
    static constexpr int BP_OFFSET = A_BYTES + BU_BYTES - BP_BYTES;  // operand buffer and the unpack expands them in place
    static constexpr int STAGE_BYTES = A_BYTES + BU_BYTES;           // 48 KB x 4 or 32 KB x 6
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int SCALE_OFFSET = BAR_OFFSET + 256;  // two buffers of {weight scales, bias} for a tile's columns
    static constexpr int SCALE_BYTES = 2 * 2 * BN * 4;
    // one 32-row x 64-byte staging tile per epilogue warp (64-byte swizzle), from which the outputs leave as TMA stores
    static constexpr int STORE_OFFSET = (SCALE_OFFSET + SCALE_BYTES + 1023) / 1024 * 1024;
    static constexpr int SMEM_BYTES = STORE_OFFSET + NUM_EPI_WARPS * 2048 + 1024;
    static constexpr int NACC = 512 / (2 * BN);  // {int32 tile, fp32 tile} pairs in tensor memory: 1 (wide) or 2 (narrow tiles)
    static_assert(8 * (3 * STAGES + 4) <= 192, "barriers must end below the two words at +192");
    static_assert(SMEM_BYTES <= 232448 && STAGE_BYTES % 1024 == 0, "shared memory plan");
};

struct A8KernelParams {
    int M, N, num_kb, lr_chunks;
    const float* xscale;  // [M]
    const float* wscale;  // [N]
    const float* bias;    // [N]
    uint16_t* y;
    int32_t* partials;
    int* status;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ void tmem_ld_fence32(uint32_t (&v)[32]) {
    asm volatile("" : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                      "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                      "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
                      "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
                 :: "memory");
}

template <bool kPartials, int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
w4a8_gemm_kernel(const __grid_constant__ CUtensorMap tmap_codes, const __grid_constant__ CUtensorMap tmap_wpacked,
                 const __grid_constant__ CUtensorMap tmap_xh, const __grid_constant__ CUtensorMap tmap_wh,
                 const __grid_constant__ CUtensorMap tmap_y, const A8KernelParams p) {
    using P = Plan<BN>;
    constexpr int STAGES = P::STAGES, BU_BYTES = P::BU_BYTES, BP_BYTES = P::BP_BYTES, BP_OFFSET = P::BP_OFFSET;
    constexpr int STAGE_BYTES = P::STAGE_BYTES, BAR_OFFSET = P::BAR_OFFSET, SCALE_OFFSET = P::SCALE_OFFSET;
    constexpr int PIECES = BN * 4 / (NUM_UNPACK_WARPS * 32);  // 16-byte pieces of the packed tile per unpack thread
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto unp_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto empty_bar = [&](int s) { return bar_base + 8u * (2 * STAGES + s); };
    constexpr int NACC = P::NACC;
    auto tfull_bar = [&](uint32_t a) { return bar_base + 8u * (3 * STAGES + a); };
    auto tempty_bar = [&](uint32_t a) { return bar_base + 8u * (3 * STAGES + 2 + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + BAR_OFFSET + 192);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + BAR_OFFSET + 196);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    // Trace build (TRACE_CLK), stages 10..12 of the block's first tile: slots 9..11 producer has issued the stage, 12..14 first unpack warp
    // sees it landed, 15..17 it has expanded it, 18..20 MMA warp starts on it; tiles 0, 1, 2 of the first epilogue warp: accumulators
    // seen / released / outputs handed over in slots 21..23, 24..26, 27..29; slot 30 entry.
    if (threadIdx.x == 0) TRACE_CLK(p.status, 30);
    const int num_m_blocks = (p.M + BM - 1) / BM;
    const int num_n_blocks = (p.N + BN - 1) / BN;
    const int num_tiles = num_m_blocks * num_n_blocks;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(unp_bar(s), NUM_UNPACK_WARPS * 32);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < NACC; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), NUM_EPI_WARPS * 32);
        }
        mbar_init(bar_base + 200u, 1);  // spare: see umma_drain
        *abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmap_codes);
        tma_prefetch_desc(&tmap_wpacked);
        tma_prefetch_desc(&tmap_xh);
        tma_prefetch_desc(&tmap_wh);
        if constexpr (!kPartials) tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // everything above touched only this CTA's own shared and tensor memory; what follows reads the first kernel's output
    grid_dependency_wait();
    // the next layer's first kernel may be scheduled as this grid's CTAs leave their SMs (it waits for this whole grid)
    grid_launch_dependents();
    const int items = p.num_kb + p.lr_chunks;  // pipeline items per tile

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // (the whole warp walks the loops and waits, one elected lane issues: counters, addresses and coordinates stay
        // warp-uniform, which shortens the chain of instructions per stage; the same in the MMA warp)
        {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int m0 = (tile % num_m_blocks) * BM;
                const int n0 = (tile / num_m_blocks) * BN;
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(empty_bar(s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    if (!elect_one()) continue;
                    if (i < p.num_kb) {
                        mbar_arrive_expect_tx(full_bar(s), A_BYTES + BP_BYTES);
                        tma_load_2d(st, &tmap_codes, full_bar(s), i * BKC, m0);
                        tma_load_2d(st + BP_OFFSET, &tmap_wpacked, full_bar(s), i * (BKC / 2), n0);
                        if (it >= 10 && it <= 12) TRACE_CLK(p.status, it - 1);
                    } else {
                        mbar_arrive_expect_tx(full_bar(s), A_BYTES + BU_BYTES);
                        tma_load_2d(st, &tmap_xh, full_bar(s), (i - p.num_kb) * 64, m0);
                        tma_load_2d(st + A_BYTES, &tmap_wh, full_bar(s), (i - p.num_kb) * 64, n0);
                    }
                }
            }
            if (!ok && lane == 0) {  // let the copies in flight land before the CTA's shared memory goes away
                const uint32_t first = it > STAGES ? it - STAGES : 0;
                for (uint32_t j = first; j < it; ++j) {
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full_bar(j % STAGES), (j / STAGES) & 1) && globaltimer_ns() - t0 < 100000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        {
            constexpr uint32_t idesc_i8 = umma_idesc(2 /*s32*/, 1 /*s8*/, BM, BN);
            constexpr uint32_t idesc_bf = umma_idesc(1 /*f32*/, 1 /*bf16*/, BM, BN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++tcount) {
                // with narrow tiles two accumulator pairs alternate: a tile's epilogue runs under the next tile's MMAs
                const uint32_t acc = tcount % NACC, tacc = tmem_base + acc * 2 * BN;
                if (!mbar_wait(tempty_bar(acc), ((tcount / NACC) & 1) ^ 1, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                tc_fence_after_sync();
                for (int i = 0; i < items; ++i, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    // (the unpack warps arrive after they have seen the stage's loads land, and one barrier counts both operands'
                    // bytes: their barrier covers the activation codes as well)
                    if (!mbar_wait(unp_bar(s), ph, abort_flag, p.status, DEV_TIMEOUT_MMA)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    const uint64_t adesc = umma_desc_sw128(st);
                    const uint64_t bdesc = umma_desc_sw128(st + A_BYTES);
                    if (!elect_one()) continue;
                    if (it >= 10 && it <= 12) TRACE_CLK(p.status, it + 8);
                    if (i < p.num_kb) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) umma_i8(tacc, adesc + 2 * k, bdesc + 2 * k, idesc_i8, (i | k) != 0);
                    } else {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(tacc + BN, adesc + 2 * k, bdesc + 2 * k, idesc_bf, ((i - p.num_kb) | k) != 0);
                    }
                    umma_commit(empty_bar(s));
                }
                if (ok && elect_one()) umma_commit(tfull_bar(acc));
            }
        }
    } else if (warp < 2 + NUM_UNPACK_WARPS) {
        // ------------------------------------------------------------ nibble -> byte unpack (warps 2..5)
        const int u = threadIdx.x - 64;  // 0..127
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            for (int i = 0; i < items; ++i, ++it) {
                const int s = it % STAGES;
                // The four unpack warps meet at a hardware barrier below, which has no time limit: they must all go on or
                // all give up.  Every thread reaches this reducing barrier once per item whatever its wait returned.
                const bool mine = mbar_wait(full_bar(s), (it / STAGES) & 1, abort_flag, p.status, DEV_TIMEOUT_UNPACK);
                uint32_t any_failed;
                asm volatile(
                    "{\n\t"
                    ".reg .pred pin, pout;\n\t"
                    "setp.eq.u32 pin, %1, 0;\n\t"
                    "bar.red.or.pred pout, 1, %2, pin;\n\t"
                    "selp.u32 %0, 1, 0, pout;\n\t"
                    "}\n"
                    : "=r"(any_failed)
                    : "r"(static_cast<uint32_t>(mine)), "n"(NUM_UNPACK_WARPS * 32)
                    : "memory");
                ok = any_failed == 0;
                if (!ok) break;
                if (u == 0 && it >= 10 && it <= 12) TRACE_CLK(p.status, it + 2);
                if (i < p.num_kb) {
                    // 16-byte piece idx = u + 128 j of the packed tile: row = idx / 4 = u / 4 + 32 j, piece c = u % 4; the
                    // swizzle phase row % 8 and the piece do not depend on j
                    uint8_t* st = smem_gen + s * STAGE_BYTES;
                    const uint4* src = reinterpret_cast<const uint4*>(st + BP_OFFSET) + u;
                    const int c = u & 3, sw = (u >> 2) & 7;
                    uint8_t* d0 = st + A_BYTES + (u >> 2) * 128 + (((2 * c) ^ sw) << 4);
                    uint8_t* d1 = st + A_BYTES + (u >> 2) * 128 + (((2 * c + 1) ^ sw) << 4);
                    // The packed codes sit in the upper half of the buffer they are expanded into: every unpack thread
                    // takes its pieces into registers, the four warps meet at a named barrier, and only then is
                    // anything stored.
                    uint4 pk[PIECES];
#pragma unroll
                    for (int j = 0; j < PIECES; ++j) pk[j] = src[128 * j];
                    asm volatile("bar.sync 2, %0;" ::"n"(NUM_UNPACK_WARPS * 32) : "memory");  // reached by all four warps (see above)
#pragma unroll
                    for (int j = 0; j < PIECES; ++j) {
                        // nibble q + 8 -> byte 16 q: into the high half, then flip bit 7 (16 (q + 8) - 128)
                        uint4 o0, o1;
                        o0.x = ((pk[j].x << 4) & 0xF0F0F0F0u) ^ 0x80808080u; o0.y = (pk[j].x & 0xF0F0F0F0u) ^ 0x80808080u;
                        o0.z = ((pk[j].y << 4) & 0xF0F0F0F0u) ^ 0x80808080u; o0.w = (pk[j].y & 0xF0F0F0F0u) ^ 0x80808080u;
                        o1.x = ((pk[j].z << 4) & 0xF0F0F0F0u) ^ 0x80808080u; o1.y = (pk[j].z & 0xF0F0F0F0u) ^ 0x80808080u;
                        o1.z = ((pk[j].w << 4) & 0xF0F0F0F0u) ^ 0x80808080u; o1.w = (pk[j].w & 0xF0F0F0F0u) ^ 0x80808080u;
                        *reinterpret_cast<uint4*>(d0 + j * 4096) = o0;  // 32 rows of 128 bytes further down
                        *reinterpret_cast<uint4*>(d1 + j * 4096) = o1;
                    }
                    fence_proxy_async_smem();
                }
                if (u == 0 && it >= 10 && it <= 12) TRACE_CLK(p.status, it + 5);
                mbar_arrive(unp_bar(s));  // every lane arrives for itself: a warp barrier followed by one elected lane's arrival costs about a hundred cycles more
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 6..13)
        const int q = warp & 3;  // TMEM lane quadrant this warp may read
        const int half = (warp - (2 + NUM_UNPACK_WARPS)) >> 2;
        constexpr int CPH = BN / 32 / 2;  // 32-column chunks per warp
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++tcount) {
            const int m0 = (tile % num_m_blocks) * BM;
            const int n0 = (tile / num_m_blocks) * BN;
            // This tile's column scales and bias go to shared memory while the MMAs are still running (two buffers: a warp
            // can be one tile ahead of the others).  The reducing barrier orders these stores before the reads below and
            // makes the four warps agree on whether to go on: a plain barrier behind a bounded wait could strand a warp.
            float* s_sw = reinterpret_cast<float*>(smem_gen + SCALE_OFFSET) + (tcount & 1) * 2 * BN;
            float* s_b = s_sw + BN;
            {
                const int e = threadIdx.x - (2 + NUM_UNPACK_WARPS) * 32;  // 0..255; the first 128 stage two columns each
                if (e < BN / 2) {
                    const int col = n0 + 2 * e;
                    float2 w2 = make_float2(0.f, 0.f), b2 = make_float2(0.f, 0.f);
                    if (col < p.N) {
                        w2 = __ldg(reinterpret_cast<const float2*>(p.wscale + col));
                        b2 = __ldg(reinterpret_cast<const float2*>(p.bias + col));
                    }
                    *reinterpret_cast<float2*>(s_sw + 2 * e) = w2;
                    *reinterpret_cast<float2*>(s_b + 2 * e) = b2;
                }
            }
            const uint32_t acc_i = tcount % NACC;
            const bool mine = mbar_wait(tfull_bar(acc_i), (tcount / NACC) & 1, abort_flag, p.status, DEV_TIMEOUT_EPILOGUE);
            uint32_t any_failed;
            asm volatile(
                "{\n\t"
                ".reg .pred pin, pout;\n\t"
                "setp.eq.u32 pin, %1, 0;\n\t"
                "bar.red.or.pred pout, 3, %2, pin;\n\t"
                "selp.u32 %0, 1, 0, pout;\n\t"
                "}\n"
                : "=r"(any_failed)
                : "r"(static_cast<uint32_t>(mine)), "n"(NUM_EPI_WARPS * 32)
                : "memory");
            ok = any_failed == 0;
            if (!ok) break;
            tc_fence_after_sync();
            if (warp == 2 + NUM_UNPACK_WARPS && lane == 0 && tcount < 3) TRACE_CLK(p.status, 21 + 3 * tcount);
            const int row = m0 + q * 32 + lane;
            const float sx = row < p.M ? __ldg(p.xscale + row) : 0.f;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc_i * 2 * BN;
#pragma unroll 1
            for (int c = half * CPH; c < (half + 1) * CPH; ++c) {
                uint32_t acc[32], lr[32];
                tmem_ld_32x32b_x32(taddr + c * 32, acc);
                tmem_ld_32x32b_x32(taddr + BN + c * 32, lr);
                tmem_ld_wait();
                tmem_ld_fence32(acc);
                tmem_ld_fence32(lr);
                if (c == (half + 1) * CPH - 1) {
                    tc_fence_before_sync();
                    mbar_arrive(tempty_bar(acc_i));
                    if (warp == 2 + NUM_UNPACK_WARPS && lane == 0 && tcount < 3) TRACE_CLK(p.status, 22 + 3 * tcount);
                }
                const int col = n0 + c * 32;
                if (row < p.M) {
                    if constexpr (kPartials) {
                        int32_t* dst = p.partials + static_cast<size_t>(row) * p.N + col;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (col + j < p.N)
                                *reinterpret_cast<int4*>(dst + j) =
                                    make_int4(static_cast<int32_t>(acc[j]) >> 4, static_cast<int32_t>(acc[j + 1]) >> 4,
                                              static_cast<int32_t>(acc[j + 2]) >> 4, static_cast<int32_t>(acc[j + 3]) >> 4);
                    }
                }
                if constexpr (!kPartials) {
                    // Outputs leave through shared memory: a thread holds one token row, so direct stores would be 32 scattered
                    // 16-byte pieces per instruction (in the NVFP4 kernel a clock trace showed such stores taking thousands of
                    // cycles per tile and slowing the operand loads).  The warp converts 32 columns of its 32 rows into its
                    // staging tile (64-byte swizzle: a quarter-warp's pieces fall into different banks) and one lane hands
                    // it to a TMA store, which writes whole sectors and clips at M and N.
                    const uint32_t sbuf = smem_base + P::STORE_OFFSET + static_cast<uint32_t>(warp - (2 + NUM_UNPACK_WARPS)) * 2048u;
                    // the chunk is converted first; only then does the warp wait for the copy engine to have read the staging
                    // tile's previous contents (this epilogue is exposed: nothing else hides that read)
                    uint32_t packed[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        float o[8];
#pragma unroll
                        for (int t = 0; t < 8; t += 4) {
                            const float4 sw = *reinterpret_cast<const float4*>(s_sw + c * 32 + j + t);
                            const float4 b = *reinterpret_cast<const float4*>(s_b + c * 32 + j + t);
                            const float sws[4] = {sw.x, sw.y, sw.z, sw.w}, bs[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                // the accumulator holds 16 P (exact); |P| < 2^24, so the conversion is exact too
                                const float pf = static_cast<float>(static_cast<int32_t>(acc[j + t + e]) >> 4);
                                o[t + e] = fmaf(pf * sx, sws[e], __uint_as_float(lr[j + t + e])) + bs[e];
                            }
                        }
                        packed[(j >> 1) + 0] = pack_bf16x2(o[0], o[1]);
                        packed[(j >> 1) + 1] = pack_bf16x2(o[2], o[3]);
                        packed[(j >> 1) + 2] = pack_bf16x2(o[4], o[5]);
                        packed[(j >> 1) + 3] = pack_bf16x2(o[6], o[7]);
                    }
                    if (lane == 0) bulk_wait_group_read_all();  // the tile's previous contents have been read
                    __syncwarp();
#pragma unroll
                    for (int pc = 0; pc < 4; ++pc) {
                        const uint32_t dst = sbuf + static_cast<uint32_t>(lane) * 64u + (static_cast<uint32_t>(pc ^ ((lane >> 1) & 3)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(packed[4 * pc]), "r"(packed[4 * pc + 1]),
                                     "r"(packed[4 * pc + 2]), "r"(packed[4 * pc + 3])
                                     : "memory");
                    }
                    fence_proxy_async_smem();  // these writes -> visible to the copy engine
                    __syncwarp();
                    if (lane == 0 && m0 + q * 32 < p.M && col < p.N) {
                        tma_store_2d(&tmap_y, sbuf, col, m0 + q * 32);
                        bulk_commit_group();
                    }
                }
            }
            if (warp == 2 + NUM_UNPACK_WARPS && lane == 0 && tcount < 3) TRACE_CLK(p.status, 23 + 3 * tcount);
        }
        if constexpr (!kPartials) {
            if (lane == 0) bulk_wait_group_all();  // this warp's stores are performed before the CTA leaves
        }
    }

    if (warp == 1 && lane == 0 && *abort_flag != 0) umma_drain(bar_base + 200u);  // a wait gave up: let issued MMAs finish first
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

template <int BN>
static dirotq_status_t launch_w4a8_gemm_bn(const dirotq_layer* L, const A8GemmArgs& a, cudaStream_t stream) {
    const Geometry& g = L->geo;
    CUtensorMap tmap_codes, tmap_xh;
    dirotq_status_t st;
    st = encode_tmap_2d(&tmap_codes, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, a.codes, (uint64_t)g.K_lp, (uint64_t)a.M,
                        (uint64_t)g.K_lp, BKC, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    st = encode_tmap_2d(&tmap_xh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.xh, (uint64_t)g.r_pad, (uint64_t)a.M,
                        (uint64_t)g.r_pad * 2, 64, BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st != DIROTQ_OK) return st;
    A8KernelParams p;
    p.M = a.M; p.N = g.N;
    p.num_kb = g.K_lp / BKC;
    p.lr_chunks = g.r_pad / 64;
    p.xscale = a.xscale;
    p.wscale = reinterpret_cast<const float*>(L->blob + L->lay.off_wscale);
    p.bias = reinterpret_cast<const float*>(L->blob + L->lay.off_bias);
    p.y = a.y; p.partials = a.partials; p.status = a.status;
    const int num_tiles = ((a.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
    const int grid = num_tiles < sm_count(L->device) ? num_tiles : sm_count(L->device);
    const bool dbg = a.partials != nullptr;
    auto kern = dbg ? w4a8_gemm_kernel<true, BN> : w4a8_gemm_kernel<false, BN>;
    static SmemOptIn<2> opt_in;
    if (!opt_in.ensure(kern, dbg ? 1 : 0, L->device, Plan<BN>::SMEM_BYTES)) return DIROTQ_ERR_CUDA;
    const bool narrow = BN == 128;
    // the outputs leave as TMA stores of 32 rows x 32 columns (64-byte swizzle in shared memory); the debug export of the
    // integer sums stores directly and is given the activation map in its place
    CUtensorMap tmap_y = tmap_xh;
    if (!dbg) {
        st = encode_tmap_2d(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.y, (uint64_t)g.N, (uint64_t)a.M, (uint64_t)g.N * 2, 32, 32,
                            CU_TENSOR_MAP_SWIZZLE_64B);
        if (st != DIROTQ_OK) return st;
    }
    const cudaError_t err = launch_kernel(kern, grid, NUM_THREADS, Plan<BN>::SMEM_BYTES, stream, true, tmap_codes,
                                          narrow ? L->tmap_wpacked128 : L->tmap_wpacked, tmap_xh,
                                          narrow ? L->tmap_wh128 : L->tmap_wh, tmap_y, p);
    return err == cudaSuccess ? DIROTQ_OK : DIROTQ_ERR_CUDA;
}

static std::atomic<int> g_a8_tile_columns{0};  // 0: chosen per call; 128 / 256: forced

}  // namespace

dirotq_status_t set_w4a8_tile_columns(int columns) {
    if (columns != 0 && columns != 128 && columns != 256) return DIROTQ_ERR_INVALID_ARG;
    g_a8_tile_columns.store(columns);
    return DIROTQ_OK;
}

dirotq_status_t launch_w4a8_gemm(const dirotq_layer* L, const A8GemmArgs& a, cudaStream_t stream) {
    // narrow tiles only where the wide ones leave SMs idle: a 128-column tile costs about NARROW_COST of a 256-column one
    constexpr double NARROW_COST = 0.68;  // measured: 0.220 against 0.162 ms with twice as many tiles (4608 x 3072 -> 9216)
    const int forced = g_a8_tile_columns.load();
    const int sms = sm_count(L->device);
    const long m_blocks = (a.M + BM - 1) / BM;
    const long t_wide = m_blocks * ((L->geo.N + 255) / 256), t_narrow = m_blocks * ((L->geo.N + 127) / 128);
    const bool narrow_pays =
        NARROW_COST * static_cast<double>((t_narrow + sms - 1) / sms) < 0.98 * static_cast<double>((t_wide + sms - 1) / sms);
    const bool narrow = forced ? forced == 128 : narrow_pays;
    return narrow ? launch_w4a8_gemm_bn<128>(L, a, stream) : launch_w4a8_gemm_bn<256>(L, a, stream);
}

}  // namespace dirotq
