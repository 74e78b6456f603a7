// Internal definitions shared by the translation units of libdirotq (not part of the C ABI).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <utility>
#include <stddef.h>
#include <stdint.h>

#include "../../include/dirotq.h"

namespace dirotq {

// ------------------------------------------------------------------ geometry of one layer
//
// Column order after the online rotation ("permuted" order): the K_l = K - r low-precision
// coefficients come first, the r high-precision ones last.  Group g of the low block is the
// permuted columns [g*G, (g+1)*G); when K_l is not a multiple of G the last group is ragged and
// the slots up to K_lp = n_g*G (which are high columns in this order) carry zero codes.
struct Geometry {
    int K, N, r, G;
    int K_l;    // K - r
    int n_g;    // ceil(K_l / G)
    int K_lp;   // n_g * G  (<= K)
    int r_pad;  // width of the bf16 rank-r operands: r rounded up to 64, plus (fmt 2) the zero-point columns, rounded up to 64
    int r_pad0; // r rounded up to a multiple of 64: where the zero-point columns of fmt 2 start
    // NVFP4 variant only (fmt == 1): blocks of 16, MMA K = 64, TMA k-blocks of 256 elements
    int fmt;     // 0 = INT4 groups with bf16 scales, 1 = NVFP4 (E2M1 elements, E4M3 block scales),
                 // 2 = INT4 with asymmetric activation codes (0..15, bf16 scale and zero-point per group),
                 // 3 = W4A8: INT8 activations with one scale per token, INT4 weights with one scale per output column
                 // 4 = projection form: only U_h [K, r] is applied densely, the residual (all K columns) is rotated by a
                 //     block Hadamard per group and quantized like fmt 0; then K_l = K_lp = K and there is no K x K rotation
                 //     (G = 128 is then only the packing granularity: K_lp = K_l rounded up to 128, n_g = K_lp / 128)
    int K4;      // K_l rounded up to 64 (<= K): width of the packed E2M1 rows
    int nkb64;   // K4 / 64: scale-factor atoms (128 rows x 4 scales) per row block
    int nkb64p;  // nkb64 rounded up to 4: one TMA k-block = 256 elements = 4 atoms
    int ph;      // 1: projection form in front of the format's quantizer (fmt 4 is ph with the INT4 quantizer; fmt 1 + ph is NVFP4)
    int no_rot;  // 1: the blob holds no rotation (a layer that only consumes a workspace rotated through a sibling layer)
};

inline Geometry make_geometry(int K, int N, int r, int G) {
    Geometry g;
    g.K = K; g.N = N; g.r = r; g.G = G;
    g.K_l = K - r;
    g.n_g = (g.K_l + G - 1) / G;
    g.K_lp = g.n_g * G;
    g.r_pad = (r + 63) / 64 * 64;
    g.r_pad0 = g.r_pad;
    g.fmt = 0;
    g.K4 = (g.K_l + 63) / 64 * 64;
    g.nkb64 = g.K4 / 64;
    g.nkb64p = (g.nkb64 + 3) / 4 * 4;
    g.no_rot = 0;
    g.ph = 0;
    return g;
}

// ------------------------------------------------------------------ weight-side layouts of the grouped INT4 formats
//
// Group scales of the weight codes, f32 [n_g][N32] (N32 = N rounded up to 32).  Two things are folded in offline:
//   * the value stored is 2^18 s_w (exact): the second kernel's accumulators hold 2^-18 times the integer group sums;
//   * inside every aligned run of 32 output columns the scales are permuted so that the 8 a thread of the second
//     kernel's epilogue needs (columns 8 b + 2 p + e, b = 0..3, e = 0..1, for its p = lane % 4) lie side by side:
//     column 8 b + 2 p + e of the run is stored at position 8 p + 2 b + e.
// (W4A8 layers keep one plain scale per output column: f32 [N].)
constexpr float kWScaleFold = 262144.0f;  // 2^18
__host__ __device__ inline int wscale_row_len(int N) { return (N + 31) / 32 * 32; }
__host__ __device__ inline size_t wscale_index(int N, int grp, int n) {
    const int c = n & 31;
    return static_cast<size_t>(grp) * wscale_row_len(N) + (n & ~31) + ((c >> 1) & 3) * 8 + (c >> 3) * 2 + (c & 1);
}

// Packed weight codes of the grouped INT4 formats: a 32-bit word holds eight codes as sign + 3-bit magnitude.  Code t < 4
// sits in byte t with its magnitude in bits 2..0 and its sign in bit 7; code t >= 4 is the same picture rotated left
// by four bit positions (magnitude in bits 6..4 of byte t - 4, sign in bit 3 of the next byte, wrapping around), so that
//     w & 0x87878787  and  rotate_right(w, 4) & 0x87878787
// are codes 0..3 and 4..7 as one byte each, s0000mmm: read as E4M3 that byte is q * 2^-9 exactly.
__host__ __device__ inline uint32_t signmag_nibble_bits(int t, int q) {  // bits of code t (0..7), q in [-7, 7]
    const uint32_t mag = static_cast<uint32_t>(q < 0 ? -q : q), sign = q < 0 ? 1u : 0u;
    const uint32_t v = mag | (sign << 7);                 // s0000mmm in byte 0
    const uint32_t placed = v << (8 * (t & 3));
    return t < 4 ? placed : ((placed << 4) | (placed >> 28));
}
__host__ __device__ inline int signmag_nibble_decode(uint32_t word, int t) {
    const uint32_t w = t < 4 ? word : ((word >> 4) | (word << 28));
    const uint32_t v = (w >> (8 * (t & 3))) & 0x87u;
    const int mag = static_cast<int>(v & 7u);
    return (v & 0x80u) ? -mag : mag;
}

// Fallback build of the library (-DDIROTQ_I8_PATH): the W4A4 group sums run on the integer tensor-core path
// (tcgen05.mma kind::i8, int32 accumulators) instead of the 8-bit float one, whose exact integer accumulation is a
// measured property of the hardware rather than a documented one.  The activation codes in the workspace are then
// two's-complement bytes, the unpack warps turn the weights' sign-magnitude bytes into two's complement, and the
// epilogue converts every group sum to fp32 before it is scaled (2^18 s_w is stored either way, so the token scale
// is multiplied by 2^-18 once per group instead).  Same blob, same interface, bit-identical results; slower.
#ifdef DIROTQ_I8_PATH
constexpr bool kI8Path = true;
#else
constexpr bool kI8Path = false;
#endif

constexpr size_t kAlign = 1024;
inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }

// Projection form (fmt 4): every one of the K residual coefficients is low-precision.
inline void make_ph(Geometry& g) {
    g.fmt = 4;
    g.ph = 1;
    g.K_l = g.K;
    g.n_g = g.K / g.G;
    g.K_lp = g.K;
}
// ... and with NVFP4 operands (G = 64 is then the Hadamard block and the epilogue's chunk)
inline void make_ph_nvfp4(Geometry& g) {
    make_ph(g);
    g.fmt = 1;
    g.K4 = g.K;
    g.nkb64 = g.K / 64;
    g.nkb64p = (g.nkb64 + 3) / 4 * 4;
}

// Sections of the device blob that holds a prepared layer.
// Asymmetric activations (fmt 2): x^ = s u + z per group.  The zero-point term sum_g z[m,g] * (s_w[g,n] sum_{j in g} q_w[j,n])
// is a rank-n_g product; it rides on the bf16 rank-r branch as 3 n_g extra columns: the activation side holds z (bf16,
// exact) three times, the weight side the three bf16 pieces of s_w * sum q_w (17 significant bits, split exactly).
inline void make_asym(Geometry& g) {
    g.fmt = 2;
    g.r_pad = (g.r_pad0 + 3 * g.n_g + 63) / 64 * 64;
}

// NVFP4 weight scale atoms (512 bytes: 128 output columns x the 4 block scales of one 64-element MMA step).  Atom `ak` (index
// along K) of 128-column block `nb` sits at [nb / 2][ak / 4][nb % 2][ak % 4]: the eight atoms a 256-column tile needs for one
// k-block of 256 elements are contiguous (one bulk load), and so are the four of either of its 128-column blocks.
__host__ __device__ inline size_t wsf_atom_offset(int nb, int ak, int nkb64p) {
    return ((((static_cast<size_t>(nb >> 1) * (nkb64p >> 2) + (ak >> 2)) * 2 + (nb & 1)) * 4) + (ak & 3)) * 512;
}
inline size_t wsf_bytes(int N, int nkb64p) { return static_cast<size_t>((N + 255) / 256) * 2 * nkb64p * 512; }

struct BlobLayout {
    size_t off_qt;       // bf16 [K][K]: row c' = permuted output column, K-major over the input channel
    size_t off_wpacked;  // u8   [N][K_lp/2]: two INT4 codes per byte, K-major, see prepare.cu for the nibble order
    size_t off_wscale;   // f32  [n_g][N32]: bf16-valued group scales of the weight codes times 2^18, see wscale_index
    size_t off_wh;       // bf16 [N][r_pad]: high-precision rows of the folded weight, K-major, zero padded
    size_t off_bias;     // f32  [N]
    // NVFP4 variant: off_wpacked = E2M1 codes u8 [N][K4/2] (even k in the low nibble); off_wscale = E4M3 scale
    // atoms u8, ordered as wsf_atom_offset says; off_meta = {float out_scale = 2^(ex+ew), int ew, int ex, uint amax bits}
    size_t off_meta;
    // projection form only: off_qt holds U_hb^T, bf16 [r_pad][K]; off_uh holds -V^T, bf16 [K][r_pad], with
    // V = bf16(U_hb^T H+-); off_had holds one +-1 Hadamard block, bf16 [G][G] (G = 64 for NVFP4 layers)
    size_t off_uh;
    size_t off_had;
    size_t total;
};

inline BlobLayout make_blob_layout(const Geometry& g) {
    BlobLayout b;
    size_t o = 0;
    b.off_qt = o;      o = align_up(o + (g.fmt == 4 ? (size_t)g.r_pad * g.K * 2 : g.no_rot ? 0 : (size_t)g.K * g.K * 2));
    b.off_uh = o;      o = align_up(o + (g.fmt == 4 ? (size_t)g.K * g.r_pad * 2 : 0));
    b.off_had = o;     o = align_up(o + (g.fmt == 4 ? (size_t)g.G * g.G * 2 : 0));
    b.off_wpacked = o; o = align_up(o + (size_t)g.N * (g.K_lp / 2));
    b.off_wscale = o;  o = align_up(o + (size_t)g.n_g * wscale_row_len(g.N) * 4);
    b.off_wh = o;      o = align_up(o + (size_t)g.N * g.r_pad * 2);
    b.off_bias = o;    o = align_up(o + (size_t)g.N * 4);
    b.off_meta = o;    o = align_up(o + 64);
    b.total = o;
    return b;
}

inline BlobLayout make_blob_layout_nvfp4(const Geometry& g) {
    BlobLayout b;
    size_t o = 0;
    b.off_qt = o;      o = align_up(o + (g.ph ? (size_t)g.r_pad * g.K * 2 : (size_t)g.K * g.K * 2));
    b.off_uh = o;      o = align_up(o + (g.ph ? (size_t)g.K * g.r_pad * 2 : 0));
    b.off_had = o;     o = align_up(o + (g.ph ? (size_t)64 * 64 * 2 : 0));
    b.off_wpacked = o; o = align_up(o + (size_t)g.N * (g.K4 / 2));
    b.off_wscale = o;  o = align_up(o + wsf_bytes(g.N, g.nkb64p));
    b.off_wh = o;      o = align_up(o + (size_t)g.N * g.r_pad * 2);
    b.off_bias = o;    o = align_up(o + (size_t)g.N * 4);
    b.off_meta = o;    o = align_up(o + 64);
    b.total = o;
    return b;
}

// Workspace of one dirotq_linear call (device memory owned by the caller).
struct WorkspaceLayout {
    int ldm;            // leading dimension (tokens) of the transposed activation-scale array
    size_t off_status;  // int32[64]: word 0 = device status
    size_t off_codes;   // u8  [M][K_lp]: activation codes, one per byte, sign-magnitude (bit 7 = sign, bits 2..0 = |q|)
    size_t off_xscale;  // f32 [n_g][ldm]: the bf16-valued activation scales s, group-major
    size_t off_xh;      // bf16 [M][r_pad]
    // NVFP4 variant: off_codes = E2M1 codes u8 [M][K4/2]; off_xscale = E4M3 scale atoms u8 [ceil(M/128)][nkb64p][512]
    size_t total;
};

inline WorkspaceLayout make_workspace_layout(const Geometry& g, int M) {
    WorkspaceLayout w;
    w.ldm = (M + 63) / 64 * 64;
    size_t o = 0;
    w.off_status = o;  o = align_up(o + 256);
    w.off_codes = o;   o = align_up(o + (size_t)M * g.K_lp);
    w.off_xscale = o;  o = align_up(o + (size_t)g.n_g * w.ldm * 4);
    w.off_xh = o;      o = align_up(o + (size_t)M * g.r_pad * 2);
    w.total = o;
    return w;
}

// W4A8 (fmt 3): off_codes = int8 [M][K_lp]; off_xscale = f32 [M] token scales; off_xtilde = f32 [M][K_lp] rotated
// low-precision coefficients (first pass); off_rowmax = u32 [M] bit patterns of the tokens' max |x~| (atomic max).
struct WorkspaceLayoutA8 {
    size_t off_status, off_codes, off_xscale, off_rowmax, off_xh, off_xtilde, total;
};
inline WorkspaceLayoutA8 make_workspace_layout_w4a8(const Geometry& g, int M) {
    WorkspaceLayoutA8 w;
    size_t o = 0;
    w.off_status = o;  o = align_up(o + 256);
    w.off_codes = o;   o = align_up(o + (size_t)M * g.K_lp);
    w.off_xscale = o;  o = align_up(o + (size_t)M * 4);
    w.off_rowmax = o;  o = align_up(o + (size_t)M * 4);
    w.off_xh = o;      o = align_up(o + (size_t)M * g.r_pad * 2);
    w.off_xtilde = o;  o = align_up(o + (size_t)M * g.K_lp * 4);
    w.total = o;
    return w;
}

inline WorkspaceLayout make_workspace_layout_nvfp4(const Geometry& g, int M) {
    WorkspaceLayout w;
    w.ldm = 0;
    size_t o = 0;
    w.off_status = o;  o = align_up(o + 256);
    w.off_codes = o;   o = align_up(o + (size_t)M * (g.K4 / 2));
    w.off_xscale = o;  o = align_up(o + (size_t)((M + 127) / 128) * g.nkb64p * 512);
    w.off_xh = o;      o = align_up(o + (size_t)M * g.r_pad * 2);
    w.total = o;
    return w;
}

}  // namespace dirotq

// The opaque handle of the C ABI: host-side description of a prepared layer.
struct dirotq_layer {
    uint32_t magic;
    int device;
    dirotq::Geometry geo;
    dirotq::BlobLayout lay;
    char* blob;  // device
    CUtensorMap tmap_qt;       // bf16 [K][K], box 64 x 256, 128B swizzle
    CUtensorMap tmap_qt128;    // the same tensor with box 64 x 128 (narrow tiles of the rotation kernel)
    CUtensorMap tmap_had;      // projection form: the +-1 Hadamard block, bf16 [G][G], box 64 x G, 128B swizzle
    CUtensorMap tmap_wpacked;  // u8 [N][K_lp/2] (two codes per byte), box 64 x kGemmBN, no swizzle
    CUtensorMap tmap_wscale;   // f32 [n_g][N32], box kGemmBN x (128/G)
    CUtensorMap tmap_wh;       // bf16 [N][r_pad], box 64 x kGemmBN, 128B swizzle
    CUtensorMap tmap_wpacked128, tmap_wscale128, tmap_wh128;  // the same three with 128-row boxes (narrow W4A4 tiles)
    CUtensorMap tmap_wpacked192, tmap_wscale192, tmap_wh192;  // ... and with 192-row boxes (grouped INT4 formats)
    CUtensorMap tmap_wpacked64, tmap_wscale64, tmap_wh64;     // ... and with 64-row boxes (calls with few token rows)
    CUtensorMap tmap_qt64;     // the rotation with box 64 x 64 (calls with few token rows, groups of 64)
    int act_scale_log2;        // NVFP4 variant: exponent of the activations' per-tensor power-of-two scale
};

namespace dirotq {

constexpr uint32_t kLayerMagic = 0x44695251u;  // "DiRQ"
constexpr int kGemmBN = 256;   // output columns per tile of the W4A4 kernel (rows of its weight-side TMA boxes)
constexpr int kNvfp4BN = 128;  // output columns per tile of the NVFP4 kernel

// ------------------------------------------------------------------ kernel launch interfaces

struct RotateArgs {
    const void* x;  // bf16 [M][K]
    int M;
    int8_t* codes;
    float* xscale;
    int ldm;
    uint16_t* xh;
    float* xrot;  // optional fp32 [M][K], columns in the caller's (unpermuted) order
    int* status;
    uint8_t* xsf = nullptr;  // NVFP4 variant: scale-factor atoms (codes then holds packed E2M1)
    float* xtilde = nullptr;       // W4A8: fp32 [M][K_lp] rotated low-precision coefficients
    unsigned int* rowmax = nullptr;  // W4A8: bit patterns of the tokens' max |x~| (zeroed before the launch)
};

struct A8GemmArgs {
    int M;
    const int8_t* codes;   // [M][K_lp]
    const float* xscale;   // [M]
    const uint16_t* xh;    // bf16 [M][r_pad]
    uint16_t* y;           // bf16 [M][N]
    int32_t* partials;     // debug: int32 [M][N]; when set, y is not written
    int* status;
};

struct GemmArgs {
    int M;
    const int8_t* codes;
    const float* xscale;
    int ldm;
    const uint16_t* xh;
    uint16_t* y;        // bf16 [M][N]
    int32_t* partials;  // debug: int32 [n_g][M][N]; when set, y is not written
    int* status;
};

// tensor-map factory (api.cu)
dirotq_status_t encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dt, size_t elem_bytes, const void* base,
                               uint64_t dim0, uint64_t dim1, uint64_t stride1_bytes, uint32_t box0, uint32_t box1,
                               CUtensorMapSwizzle swz);

// launchers (each returns after enqueueing on `stream`)
dirotq_status_t launch_rotate_quantize(const dirotq_layer* L, const RotateArgs& a, cudaStream_t stream);
dirotq_status_t launch_w4a4_gemm(const dirotq_layer* L, const GemmArgs& a, cudaStream_t stream);
dirotq_status_t set_w4a4_tile_columns(int columns);
// Launches `kern`; with `dependent` (and unless switched off process-wide) as a programmatic dependent launch: the
// kernel may be scheduled while the previous kernel of the stream drains, and orders itself with
// grid_dependency_wait().
bool dependent_launch_enabled();
void set_dependent_launch(bool on);
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream, bool dependent,
                                 Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    const bool pdl = dependent && dependent_launch_enabled();
    cfg.attrs = pdl ? attr : nullptr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// The same launch as clusters of `cluster` CTAs (`grid` a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_clusters(void (*kern)(KArgs...), int grid, int cluster, int block, size_t smem, cudaStream_t stream,
                                          bool dependent, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    const bool pdl = dependent && dependent_launch_enabled();
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// How many clusters of `cluster` CTAs of `kern` the current device holds at once (0 on error).
template <typename... KArgs>
inline int max_active_clusters(void (*kern)(KArgs...), int cluster, int block, size_t smem) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(cluster));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n;
}

// The same launch as clusters of two CTAs (`grid` must be even).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_pairs(void (*kern)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream, bool dependent,
                                       Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(static_cast<unsigned>(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    const bool pdl = dependent && dependent_launch_enabled();
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// Raising a kernel's dynamic shared-memory limit (cudaFuncSetAttribute) applies to the CURRENT device only, so what has been
// done is remembered per device: one table of flags per launch site, indexed by device and kernel variant.  Safe to
// call from several host threads (the attribute call is idempotent; the flag only saves repeating it).
template <int VARIANTS>
struct SmemOptIn {
    std::atomic<bool> done[64][VARIANTS];
    template <typename Kernel>
    bool ensure(Kernel kern, int variant, int device, int bytes) {
        const bool cached = device >= 0 && device < 64;
        if (cached && done[device][variant].load(std::memory_order_acquire)) return true;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
        if (cached) done[device][variant].store(true, std::memory_order_release);
        return true;
    }
};

dirotq_status_t set_nvfp4_tile_columns(int columns);
dirotq_status_t set_w4a8_tile_columns(int columns);
dirotq_status_t set_rotation_plan(int plan);
void set_first_step_split(bool on);
dirotq_status_t launch_prepare_ph(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                  const void* bias, double* scratch, cudaStream_t stream);
dirotq_status_t launch_uh_export(const dirotq_layer* L, uint16_t* uh, uint16_t* v, cudaStream_t stream);
dirotq_status_t launch_prepare_nvfp4_ph(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                        const void* bias, double* scratch, cudaStream_t stream);
dirotq_status_t launch_project_quantize(const dirotq_layer* L, const RotateArgs& a, cudaStream_t stream);
struct Nvfp4GemmArgs {
    int M;
    const uint8_t* codes;  // [M][K4/2]
    const uint8_t* xsf;    // scale-factor atoms
    const uint16_t* xh;    // bf16 [M][r_pad]
    uint16_t* y;           // bf16 [M][N]
    int* status;
};
dirotq_status_t launch_nvfp4_gemm(const dirotq_layer* L, const Nvfp4GemmArgs& a, cudaStream_t stream);
dirotq_status_t launch_prepare_nvfp4(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                                     int q_dtype, const void* bias, double* scratch, cudaStream_t stream);
dirotq_status_t launch_layer_export_nvfp4(const dirotq_layer* L, uint8_t* wcodes, uint8_t* wsf, uint16_t* wh, uint16_t* qb,
                                          int* ew, cudaStream_t stream);
dirotq_status_t launch_workspace_export_nvfp4(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                              uint8_t* codes, uint8_t* sf, cudaStream_t stream);
dirotq_status_t launch_prepare(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                               int q_dtype, const void* bias, const int8_t* wcodes, const void* wscales, double* scratch,
                               cudaStream_t stream);
dirotq_status_t launch_pack_codes(const dirotq_layer* L, const int8_t* wcodes, const uint16_t* wscales, cudaStream_t stream);
size_t gptq_scratch_bytes(int K, int N, int r, int T);
dirotq_status_t launch_gptq_round(const dirotq_layer* L, const void* calib_bf16, int T, double damp, int block, char* scratch,
                                  cudaStream_t stream, const int8_t** codes_out, const uint16_t** scales_out);
dirotq_status_t launch_layer_export(const dirotq_layer* L, int8_t* wcodes, uint16_t* wscales, uint16_t* wh,
                                    uint16_t* qb, cudaStream_t stream);
dirotq_status_t launch_workspace_export(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                        int8_t* codes, uint16_t* scales, cudaStream_t stream);
dirotq_status_t launch_workspace_export_asym(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh,
                                             uint8_t* codes, uint16_t* scales, uint16_t* zeros, cudaStream_t stream);
dirotq_status_t launch_zero_term_export(const dirotq_layer* L, float* d, cudaStream_t stream);
dirotq_status_t launch_w4a8_gemm(const dirotq_layer* L, const A8GemmArgs& a, cudaStream_t stream);
dirotq_status_t launch_a8_quantize(const dirotq_layer* L, int M, const float* xtilde, const unsigned int* rowmax, int8_t* codes,
                                   float* xscale, cudaStream_t stream);
dirotq_status_t launch_prepare_w4a8(const dirotq_layer* L, const void* W, int w_dtype, int w_layout, const void* Q,
                                    int q_dtype, const void* bias, double* scratch, cudaStream_t stream);
dirotq_status_t launch_workspace_export_w4a8(const dirotq_layer* L, int M, const char* workspace, uint16_t* xh, int8_t* codes,
                                             uint16_t* scales, cudaStream_t stream);
dirotq_status_t launch_debug_codes(const dirotq_layer* L, int M, const int8_t* act_codes, char* workspace,
                                   cudaStream_t stream);
int sm_count(int device);

}  // namespace dirotq
