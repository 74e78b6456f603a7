// C ABI of libdirotq: argument validation, tensor-map construction, launch sequencing.
#include "common.h"

#include <atomic>

#include <mutex>

#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

namespace dirotq {
namespace {

thread_local char g_last_error[256] = "";

void set_error(const char* what, cudaError_t e) {
    snprintf(g_last_error, sizeof g_last_error, "%s: %s", what, cudaGetErrorString(e));
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up at run time so that the library loads on machines
// without a driver (build hosts); any call that needs it fails with DIROTQ_ERR_CUDA there.
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres);
        if (e == cudaSuccess && qres == cudaDriverEntryPointSuccess) fn = reinterpret_cast<EncodeTiledFn>(p);
        else set_error("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", e);
    }
    return fn;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

dirotq_status_t check_shape(int K, int N, int r, int G) {
    if (K <= 0 || N <= 0 || r <= 0) return DIROTQ_ERR_INVALID_ARG;
    if (G != 64 && G != 128) return DIROTQ_ERR_UNSUPPORTED_SHAPE;
    if (K % 64 != 0 || K % G != 0 || N % 16 != 0) return DIROTQ_ERR_UNSUPPORTED_SHAPE;
    if (r % 16 != 0 || r > 4096 || r >= K) return DIROTQ_ERR_UNSUPPORTED_SHAPE;
    return DIROTQ_OK;
}

bool valid_layer(const dirotq_layer* L) { return L != nullptr && L->magic == kLayerMagic; }

dirotq_status_t check_device(int* device_out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_error("cudaGetDevice", e); return DIROTQ_ERR_CUDA; }
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) { set_error("cudaDeviceGetAttribute", e); return DIROTQ_ERR_CUDA; }
    if (major != 10) return DIROTQ_ERR_ARCH;
    *device_out = dev;
    return DIROTQ_OK;
}

}  // namespace

int sm_count(int device) {
    static int cached[64] = {0};
    if (device < 0 || device >= 64) return 148;
    if (cached[device] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) n = 148;
        cached[device] = n;
    }
    return cached[device];
}

dirotq_status_t encode_tmap_2d(CUtensorMap* out, CUtensorMapDataType dt, size_t elem_bytes, const void* base,
                               uint64_t dim0, uint64_t dim1, uint64_t stride1_bytes, uint32_t box0, uint32_t box1,
                               CUtensorMapSwizzle swz) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return DIROTQ_ERR_CUDA;
    if (!aligned16(base) || stride1_bytes % 16 != 0 || (box0 * elem_bytes) % 16 != 0) return DIROTQ_ERR_INVALID_ARG;
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {stride1_bytes};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_last_error, sizeof g_last_error, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return DIROTQ_ERR_CUDA;
    }
    return DIROTQ_OK;
}

static std::atomic<bool> g_dependent_launch{true};
bool dependent_launch_enabled() { return g_dependent_launch.load(); }
void set_dependent_launch(bool on) { g_dependent_launch.store(on); }

}  // namespace dirotq

using namespace dirotq;

extern "C" {

const char* dirotq_status_string(dirotq_status_t s) {
    switch (s) {
        case DIROTQ_OK: return "ok";
        case DIROTQ_ERR_INVALID_ARG: return "invalid argument";
        case DIROTQ_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case DIROTQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case DIROTQ_ERR_ARCH: return "device is not sm_100";
        case DIROTQ_ERR_CUDA: return "CUDA error";
        case DIROTQ_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int dirotq_version(void) { return 100; }

const char* dirotq_last_error(void) { return g_last_error; }

dirotq_status_t dirotq_layer_bytes(int K, int N, int r, int group, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, group);
    if (st != DIROTQ_OK) return st;
    *bytes = make_blob_layout(make_geometry(K, N, r, group)).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_scratch_bytes(int K, int N, size_t* bytes) {
    if (!bytes || K <= 0 || N <= 0) return DIROTQ_ERR_INVALID_ARG;
    *bytes = static_cast<size_t>(K) * N * sizeof(double);
    return DIROTQ_OK;
}

static size_t workspace_need(const dirotq_layer_t* layer, int M) {
    switch (layer->geo.fmt) {
        case 1: return make_workspace_layout_nvfp4(layer->geo, M).total;
        case 3: return make_workspace_layout_w4a8(layer->geo, M).total;
        default: return make_workspace_layout(layer->geo, M).total;
    }
}

dirotq_status_t dirotq_workspace_bytes(const dirotq_layer_t* layer, int M, size_t* bytes) {
    if (!valid_layer(layer) || !bytes || M < 1) return DIROTQ_ERR_INVALID_ARG;
    *bytes = workspace_need(layer, M);
    return DIROTQ_OK;
}

// Weight-side tensor maps with 192-row boxes (the 192-column tile plan of the grouped INT4 second kernel) and with 64-row
// boxes (its plan for calls with few token rows).
static dirotq_status_t encode_tmaps_rows(dirotq_layer* L, int N, int group, int rows, CUtensorMap* wpacked, CUtensorMap* wscale,
                                         CUtensorMap* wh) {
    const Geometry& g = L->geo;
    const BlobLayout& lay = L->lay;
    dirotq_status_t st = encode_tmap_2d(wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                                        (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, rows, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(wscale, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, rows, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, rows, CU_TENSOR_MAP_SWIZZLE_128B);
    return st;
}

static dirotq_status_t encode_tmaps_192(dirotq_layer* L, int N, int group) {
    dirotq_status_t st64 = encode_tmaps_rows(L, N, group, 64, &L->tmap_wpacked64, &L->tmap_wscale64, &L->tmap_wh64);
    if (st64 != DIROTQ_OK) return st64;
    const Geometry& g = L->geo;
    const BlobLayout& lay = L->lay;
    dirotq_status_t st = encode_tmap_2d(&L->tmap_wpacked192, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                                        (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, 192, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wscale192, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, 192, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh192, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, 192, CU_TENSOR_MAP_SWIZZLE_128B);
    return st;
}

struct GptqArgs {
    const void* calib;  // bf16 [T][K] calibration tokens (device); NULL: round to nearest
    int T;
    double damp;
    int block;
};

static dirotq_status_t prepare_int4(bool asym, bool sibling, const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                    const void* bias, const int8_t* wcodes, const void* wscales, int K, int N, int r,
                                    int group, void* blob, size_t blob_bytes,
                                    void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                    dirotq_layer_t** layer_out, const GptqArgs* gptq = nullptr) {
    if (!W || !Q || !blob || !scratch || !layer_out) return DIROTQ_ERR_INVALID_ARG;
    if (w_dtype != DIROTQ_DTYPE_F32 && w_dtype != DIROTQ_DTYPE_BF16) return DIROTQ_ERR_INVALID_ARG;
    if (q_dtype != DIROTQ_DTYPE_F64 && q_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    if (w_layout != DIROTQ_LAYOUT_KN && w_layout != DIROTQ_LAYOUT_NK) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, group);
    if (st != DIROTQ_OK) return st;
    if (!aligned16(W) || !aligned16(Q) || !aligned16(scratch) || (bias && !aligned16(bias))) return DIROTQ_ERR_INVALID_ARG;
    if ((wcodes == nullptr) != (wscales == nullptr)) return DIROTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    Geometry g = make_geometry(K, N, r, group);
    if (asym) make_asym(g);
    g.no_rot = sibling ? 1 : 0;
    const BlobLayout lay = make_blob_layout(g);
    if (blob_bytes < lay.total) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (scratch_bytes < static_cast<size_t>(K) * N * sizeof(double)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (gptq) {
        if (!gptq->calib || !aligned16(gptq->calib) || gptq->T < 1 || !(gptq->damp > 0.0) || gptq->block < group ||
            gptq->block > 128 || gptq->block % group != 0)
            return DIROTQ_ERR_INVALID_ARG;
        if (scratch_bytes < gptq_scratch_bytes(K, N, r, gptq->T)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    }
    int dev = 0;
    st = check_device(&dev);
    if (st != DIROTQ_OK) return st;

    dirotq_layer* L = new (std::nothrow) dirotq_layer;
    if (!L) return DIROTQ_ERR_INVALID_ARG;
    memset(L, 0, sizeof *L);
    L->magic = kLayerMagic;
    L->device = dev;
    L->geo = g;
    L->lay = lay;
    L->blob = static_cast<char*>(blob);

    st = DIROTQ_OK;
    if (!sibling) {
        st = encode_tmap_2d(&L->tmap_qt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                            (uint64_t)K * 2, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
        if (st == DIROTQ_OK)
            st = encode_tmap_2d(&L->tmap_qt128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K,
                                (uint64_t)K, (uint64_t)K * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
        if (st == DIROTQ_OK)
            st = encode_tmap_2d(&L->tmap_qt64, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K,
                                (uint64_t)K, (uint64_t)K * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wscale, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, kGemmBN, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked128, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wscale128, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, 128, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK) st = encode_tmaps_192(L, N, group);
    if (st == DIROTQ_OK)
        st = launch_prepare(L, W, w_dtype, w_layout, Q, q_dtype, bias, wcodes, wscales, static_cast<double*>(scratch),
                            static_cast<cudaStream_t>(stream));
    if (st == DIROTQ_OK && gptq) {
        // the round-to-nearest layer above left the folded weight in the scratch and the bf16 rotation in the blob: round
        // the residual rows again with error feedback and put those codes and scales in place of the first ones
        const int8_t* codes = nullptr;
        const uint16_t* scales = nullptr;
        st = launch_gptq_round(L, gptq->calib, gptq->T, gptq->damp, gptq->block, static_cast<char*>(scratch),
                               static_cast<cudaStream_t>(stream), &codes, &scales);
        if (st == DIROTQ_OK) st = launch_pack_codes(L, codes, scales, static_cast<cudaStream_t>(stream));
    }
    if (st != DIROTQ_OK) {
        delete L;
        return st;
    }
    *layer_out = L;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_scratch_bytes_gptq(int K, int N, int r, int calib_tokens, size_t* bytes) {
    if (!bytes || K <= 0 || N <= 0 || r <= 0 || r >= K || calib_tokens < 1) return DIROTQ_ERR_INVALID_ARG;
    *bytes = gptq_scratch_bytes(K, N, r, calib_tokens);
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_gptq(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                          const void* bias, const void* calib_x, int calib_tokens, double damp, int block,
                                          int asym, int K, int N, int r, int group, void* blob, size_t blob_bytes,
                                          void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                          dirotq_layer_t** layer_out) {
    const GptqArgs ga = {calib_x, calib_tokens, damp, block};
    return prepare_int4(asym != 0, false, W, w_dtype, w_layout, Q, q_dtype, bias, nullptr, nullptr, K, N, r, group, blob,
                        blob_bytes, scratch, scratch_bytes, stream, layer_out, &ga);
}

dirotq_status_t dirotq_prepare_layer(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                     const void* bias, int K, int N, int r, int group, void* blob, size_t blob_bytes,
                                     void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                     dirotq_layer_t** layer_out) {
    return prepare_int4(false, false, W, w_dtype, w_layout, Q, q_dtype, bias, nullptr, nullptr, K, N, r, group, blob, blob_bytes,
                        scratch, scratch_bytes, stream, layer_out);
}

dirotq_status_t dirotq_prepare_layer_codes(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                           const void* bias, const int8_t* wcodes, const void* wscales, int asym, int K,
                                           int N, int r, int group, void* blob, size_t blob_bytes, void* scratch,
                                           size_t scratch_bytes, dirotq_stream_t stream, dirotq_layer_t** layer_out) {
    if (!wcodes || !wscales) return DIROTQ_ERR_INVALID_ARG;
    return prepare_int4(asym != 0, false, W, w_dtype, w_layout, Q, q_dtype, bias, wcodes, wscales, K, N, r, group, blob,
                        blob_bytes, scratch, scratch_bytes, stream, layer_out);
}

dirotq_status_t dirotq_layer_bytes_asym(int K, int N, int r, int group, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, group);
    if (st != DIROTQ_OK) return st;
    Geometry g = make_geometry(K, N, r, group);
    make_asym(g);
    *bytes = make_blob_layout(g).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_asym(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                          const void* bias, int K, int N, int r, int group, void* blob, size_t blob_bytes,
                                          void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                          dirotq_layer_t** layer_out) {
    return prepare_int4(true, false, W, w_dtype, w_layout, Q, q_dtype, bias, nullptr, nullptr, K, N, r, group, blob, blob_bytes,
                        scratch, scratch_bytes, stream, layer_out);
}

dirotq_status_t dirotq_layer_bytes_sibling(int K, int N, int r, int group, int asym, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, group);
    if (st != DIROTQ_OK) return st;
    Geometry g = make_geometry(K, N, r, group);
    if (asym) make_asym(g);
    g.no_rot = 1;
    *bytes = make_blob_layout(g).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_sibling(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                             const void* bias, int asym, int K, int N, int r, int group, void* blob,
                                             size_t blob_bytes, void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                             dirotq_layer_t** layer_out) {
    return prepare_int4(asym != 0, true, W, w_dtype, w_layout, Q, q_dtype, bias, nullptr, nullptr, K, N, r, group, blob,
                        blob_bytes, scratch, scratch_bytes, stream, layer_out);
}

// ---- projection form (fmt 4): U_h only, block-Hadamard residual ----

static dirotq_status_t ph_geometry(int K, int N, int r, int group, Geometry* out) {
    dirotq_status_t st = check_shape(K, N, r, group);
    if (st != DIROTQ_OK) return st;
    Geometry g = make_geometry(K, N, r, group);
    make_ph(g);
    *out = g;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_layer_bytes_ph(int K, int N, int r, int group, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    Geometry g;
    dirotq_status_t st = ph_geometry(K, N, r, group, &g);
    if (st != DIROTQ_OK) return st;
    *bytes = make_blob_layout(g).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_scratch_bytes_ph(int K, int N, int r, size_t* bytes) {
    if (!bytes || K <= 0 || N <= 0 || r <= 0) return DIROTQ_ERR_INVALID_ARG;
    *bytes = (static_cast<size_t>(K) + r) * N * sizeof(double);
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_ph(const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                        const void* bias, int K, int N, int r, int group, void* blob, size_t blob_bytes,
                                        void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                        dirotq_layer_t** layer_out) {
    if (!W || !Uh || !blob || !scratch || !layer_out) return DIROTQ_ERR_INVALID_ARG;
    if (w_dtype != DIROTQ_DTYPE_F32 && w_dtype != DIROTQ_DTYPE_BF16) return DIROTQ_ERR_INVALID_ARG;
    if (uh_dtype != DIROTQ_DTYPE_F64 && uh_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    if (w_layout != DIROTQ_LAYOUT_KN && w_layout != DIROTQ_LAYOUT_NK) return DIROTQ_ERR_INVALID_ARG;
    Geometry g;
    dirotq_status_t st = ph_geometry(K, N, r, group, &g);
    if (st != DIROTQ_OK) return st;
    if (!aligned16(W) || !aligned16(Uh) || !aligned16(scratch) || (bias && !aligned16(bias))) return DIROTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    const BlobLayout lay = make_blob_layout(g);
    if (blob_bytes < lay.total) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (scratch_bytes < (static_cast<size_t>(K) + r) * N * sizeof(double)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    int dev = 0;
    st = check_device(&dev);
    if (st != DIROTQ_OK) return st;
    dirotq_layer* L = new (std::nothrow) dirotq_layer;
    if (!L) return DIROTQ_ERR_INVALID_ARG;
    memset(L, 0, sizeof *L);
    L->magic = kLayerMagic;
    L->device = dev;
    L->geo = g;
    L->lay = lay;
    L->blob = static_cast<char*>(blob);
    // first stage, step 1: x [M,K] times U_hb^T stored as [r_pad][K] (a 128-row box reads zeros past r_pad);
    // step 2: x~_h [M,r_pad] times -V^T stored as [K][r_pad], then x times the +-1 Hadamard block, group by group
    st = encode_tmap_2d(&L->tmap_qt128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K,
                        (uint64_t)g.r_pad, (uint64_t)K * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_uh, (uint64_t)g.r_pad,
                            (uint64_t)K, (uint64_t)g.r_pad * 2, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_had, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_had, (uint64_t)g.G,
                            (uint64_t)g.G, (uint64_t)g.G * 2, 64, g.G, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wscale, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, kGemmBN, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked128, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wscale128, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, L->blob + lay.off_wscale,
                            (uint64_t)wscale_row_len(N), (uint64_t)g.n_g, (uint64_t)wscale_row_len(N) * 4, 128, 128 / group,
                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK) st = encode_tmaps_192(L, N, group);
    if (st == DIROTQ_OK)
        st = launch_prepare_ph(L, W, w_dtype, w_layout, Uh, uh_dtype, bias, static_cast<double*>(scratch),
                               static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) {
        delete L;
        return st;
    }
    *layer_out = L;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_layer_export_uh(const dirotq_layer_t* layer, void* uh_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || !layer->geo.ph || !uh_bf16) return DIROTQ_ERR_INVALID_ARG;
    return launch_uh_export(layer, static_cast<uint16_t*>(uh_bf16), nullptr, static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_export_v(const dirotq_layer_t* layer, void* v_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || !layer->geo.ph || !v_bf16) return DIROTQ_ERR_INVALID_ARG;
    return launch_uh_export(layer, nullptr, static_cast<uint16_t*>(v_bf16), static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_bytes_w4a8(int K, int N, int r, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    Geometry g = make_geometry(K, N, r, 128);
    g.fmt = 3;
    *bytes = make_blob_layout(g).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_w4a8(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                          const void* bias, int K, int N, int r, void* blob, size_t blob_bytes, void* scratch,
                                          size_t scratch_bytes, dirotq_stream_t stream, dirotq_layer_t** layer_out) {
    if (!W || !Q || !blob || !scratch || !layer_out) return DIROTQ_ERR_INVALID_ARG;
    if (w_dtype != DIROTQ_DTYPE_F32 && w_dtype != DIROTQ_DTYPE_BF16) return DIROTQ_ERR_INVALID_ARG;
    if (q_dtype != DIROTQ_DTYPE_F64 && q_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    if (w_layout != DIROTQ_LAYOUT_KN && w_layout != DIROTQ_LAYOUT_NK) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    if (!aligned16(W) || !aligned16(Q) || !aligned16(scratch) || (bias && !aligned16(bias))) return DIROTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    Geometry g = make_geometry(K, N, r, 128);  // 128: packing granularity of the codes only
    g.fmt = 3;
    const BlobLayout lay = make_blob_layout(g);
    if (blob_bytes < lay.total) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (scratch_bytes < static_cast<size_t>(K) * N * sizeof(double)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    int dev = 0;
    st = check_device(&dev);
    if (st != DIROTQ_OK) return st;
    dirotq_layer* L = new (std::nothrow) dirotq_layer;
    if (!L) return DIROTQ_ERR_INVALID_ARG;
    memset(L, 0, sizeof *L);
    L->magic = kLayerMagic;
    L->device = dev;
    L->geo = g;
    L->lay = lay;
    L->blob = static_cast<char*>(blob);
    st = encode_tmap_2d(&L->tmap_qt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                        (uint64_t)K * 2, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                            (uint64_t)K * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt64, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                            (uint64_t)K * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, kGemmBN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked128, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked,
                            (uint64_t)g.K_lp / 2, (uint64_t)N, (uint64_t)g.K_lp / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = launch_prepare_w4a8(L, W, w_dtype, w_layout, Q, q_dtype, bias, static_cast<double*>(scratch),
                                 static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) {
        delete L;
        return st;
    }
    *layer_out = L;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_workspace_export_w4a8(const dirotq_layer_t* layer, int M, const void* workspace, void* xh_bf16,
                                             int8_t* codes, void* scales_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt != 3 || !workspace || M < 1 || M > 65535) return DIROTQ_ERR_INVALID_ARG;
    return launch_workspace_export_w4a8(layer, M, static_cast<const char*>(workspace), static_cast<uint16_t*>(xh_bf16), codes,
                                        static_cast<uint16_t*>(scales_bf16), static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_workspace_export_asym(const dirotq_layer_t* layer, int M, const void* workspace, void* xh_bf16,
                                             uint8_t* codes, void* scales_bf16, void* zeros_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt != 2 || !workspace || M < 1 || M > 65535) return DIROTQ_ERR_INVALID_ARG;
    return launch_workspace_export_asym(layer, M, static_cast<const char*>(workspace), static_cast<uint16_t*>(xh_bf16), codes,
                                        static_cast<uint16_t*>(scales_bf16), static_cast<uint16_t*>(zeros_bf16),
                                        static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_export_zero_term(const dirotq_layer_t* layer, float* zero_term, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt != 2 || !zero_term) return DIROTQ_ERR_INVALID_ARG;
    return launch_zero_term_export(layer, zero_term, static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_destroy(dirotq_layer_t* layer) {
    if (!valid_layer(layer)) return DIROTQ_ERR_INVALID_ARG;
    layer->magic = 0;
    delete layer;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_layer_info(const dirotq_layer_t* layer, int* K, int* N, int* r, int* group, int* n_g, int* K_lp) {
    if (!valid_layer(layer)) return DIROTQ_ERR_INVALID_ARG;
    if (K) *K = layer->geo.K;
    if (N) *N = layer->geo.N;
    if (r) *r = layer->geo.r;
    if (group) *group = layer->geo.G;
    if (n_g) *n_g = layer->geo.n_g;
    if (K_lp) *K_lp = layer->geo.K_lp;
    return DIROTQ_OK;
}

static dirotq_status_t check_call(const dirotq_layer_t* layer, int M, const void* workspace, size_t workspace_bytes,
                                  bool rotates = true) {
    if (!valid_layer(layer) || !workspace || M < 1) return DIROTQ_ERR_INVALID_ARG;
    if (rotates && layer->geo.no_rot) return DIROTQ_ERR_INVALID_ARG;  // a sibling layer holds no rotation
    if ((reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    if (workspace_bytes < workspace_need(layer, M)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    // the layer's blob and tensor maps belong to the device it was prepared on: that device must be current
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIROTQ_ERR_CUDA;
    if (dev != layer->device) return DIROTQ_ERR_INVALID_ARG;
    return DIROTQ_OK;
}

static RotateArgs rotate_args(const dirotq_layer_t* layer, const void* x, int M, char* ws, float* xrot) {
    if (layer->geo.fmt == 3) {
        const WorkspaceLayoutA8 w = make_workspace_layout_w4a8(layer->geo, M);
        RotateArgs a;
        a.x = x; a.M = M;
        a.codes = reinterpret_cast<int8_t*>(ws + w.off_codes);
        a.xscale = reinterpret_cast<float*>(ws + w.off_xscale);
        a.ldm = 0;
        a.xh = reinterpret_cast<uint16_t*>(ws + w.off_xh);
        a.xrot = xrot;
        a.status = reinterpret_cast<int*>(ws + w.off_status);
        a.xtilde = reinterpret_cast<float*>(ws + w.off_xtilde);
        a.rowmax = reinterpret_cast<unsigned int*>(ws + w.off_rowmax);
        return a;
    }
    const bool nv = layer->geo.fmt == 1;
    const WorkspaceLayout w = nv ? make_workspace_layout_nvfp4(layer->geo, M) : make_workspace_layout(layer->geo, M);
    RotateArgs a;
    a.x = x; a.M = M;
    a.codes = reinterpret_cast<int8_t*>(ws + w.off_codes);
    a.xscale = reinterpret_cast<float*>(ws + w.off_xscale);
    a.ldm = w.ldm;
    a.xh = reinterpret_cast<uint16_t*>(ws + w.off_xh);
    a.xrot = xrot;
    a.status = reinterpret_cast<int*>(ws + w.off_status);
    a.xsf = nv ? reinterpret_cast<uint8_t*>(ws + w.off_xscale) : nullptr;
    return a;
}

// First kernel(s): rotation + split + quantization.  W4A8 needs the token's whole row before it can quantize: the rotation
// kernel writes fp32 coefficients and the row maxima, a second small kernel quantizes.
static dirotq_status_t first_kernel(const dirotq_layer_t* layer, const RotateArgs& ra, int M, cudaStream_t s) {
    if (layer->geo.ph) return launch_project_quantize(layer, ra, s);
    if (layer->geo.fmt == 3) {
        if (cudaMemsetAsync(ra.rowmax, 0, static_cast<size_t>(M) * 4, s) != cudaSuccess) return DIROTQ_ERR_CUDA;
        dirotq_status_t st = launch_rotate_quantize(layer, ra, s);
        if (st != DIROTQ_OK) return st;
        return launch_a8_quantize(layer, M, ra.xtilde, ra.rowmax, ra.codes, ra.xscale, s);
    }
    return launch_rotate_quantize(layer, ra, s);
}

static dirotq_status_t second_kernel(const dirotq_layer_t* layer, const RotateArgs& ra, int M, void* y, cudaStream_t s) {
    if (layer->geo.fmt == 3) {
        A8GemmArgs ga;
        ga.M = M; ga.codes = ra.codes; ga.xscale = ra.xscale; ga.xh = ra.xh;
        ga.y = static_cast<uint16_t*>(y); ga.partials = nullptr; ga.status = ra.status;
        return launch_w4a8_gemm(layer, ga, s);
    }
    if (layer->geo.fmt == 1) {
        Nvfp4GemmArgs na;
        na.M = M; na.codes = reinterpret_cast<const uint8_t*>(ra.codes); na.xsf = ra.xsf; na.xh = ra.xh;
        na.y = static_cast<uint16_t*>(y); na.status = ra.status;
        return launch_nvfp4_gemm(layer, na, s);
    }
    GemmArgs ga;
    ga.M = M; ga.codes = ra.codes; ga.xscale = ra.xscale; ga.ldm = ra.ldm; ga.xh = ra.xh;
    ga.y = static_cast<uint16_t*>(y); ga.partials = nullptr; ga.status = ra.status;
    return launch_w4a4_gemm(layer, ga, s);
}

dirotq_status_t dirotq_set_rotation_tile(int plan) { return set_rotation_plan(plan); }

dirotq_status_t dirotq_set_first_step_split(int enabled) {
    dirotq::set_first_step_split(enabled != 0);
    return DIROTQ_OK;
}

dirotq_status_t dirotq_set_dependent_launch(int enabled) {
    dirotq::set_dependent_launch(enabled != 0);
    return DIROTQ_OK;
}

dirotq_status_t dirotq_set_gemm_tile(int columns) {
    // 64 and 192: plans of the grouped INT4 second kernel only; 512: 256 columns per pair of CTAs, NVFP4 second kernel only
    const bool int4_only = columns == 64 || columns == 66 || columns == 192;  // 66: 64 columns with the reduction split over a cluster
    dirotq_status_t st = set_w4a4_tile_columns(columns == 512 ? 0 : columns);
    if (st == DIROTQ_OK) st = set_nvfp4_tile_columns(int4_only ? 0 : columns);
    return st != DIROTQ_OK ? st : set_w4a8_tile_columns(int4_only || columns == 512 ? 0 : columns);
}

dirotq_status_t dirotq_rotate_quantize(const void* x, int M, const dirotq_layer_t* layer, void* workspace,
                                       size_t workspace_bytes, float* xrot_f32, dirotq_stream_t stream) {
    dirotq_status_t st = check_call(layer, M, workspace, workspace_bytes);
    if (st != DIROTQ_OK) return st;
    if (!x || !aligned16(x) || (xrot_f32 && !aligned16(xrot_f32))) return DIROTQ_ERR_INVALID_ARG;
    return first_kernel(layer, rotate_args(layer, x, M, static_cast<char*>(workspace), xrot_f32), M,
                        static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_linear(const void* x, int M, const dirotq_layer_t* layer, void* y, void* workspace,
                              size_t workspace_bytes, dirotq_stream_t stream) {
    dirotq_status_t st = check_call(layer, M, workspace, workspace_bytes);
    if (st != DIROTQ_OK) return st;
    if (!x || !y || !aligned16(x) || !aligned16(y)) return DIROTQ_ERR_INVALID_ARG;
    char* ws = static_cast<char*>(workspace);
    const RotateArgs ra = rotate_args(layer, x, M, ws, nullptr);
    st = first_kernel(layer, ra, M, static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) return st;
    return second_kernel(layer, ra, M, y, static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_w4a4_gemm(int M, const dirotq_layer_t* layer, const void* workspace, size_t workspace_bytes,
                                 void* y, dirotq_stream_t stream) {
    dirotq_status_t st = check_call(layer, M, workspace, workspace_bytes, false);
    if (st != DIROTQ_OK) return st;
    if (!y || !aligned16(y)) return DIROTQ_ERR_INVALID_ARG;
    char* ws = const_cast<char*>(static_cast<const char*>(workspace));
    const RotateArgs ra = rotate_args(layer, nullptr, M, ws, nullptr);
    return second_kernel(layer, ra, M, y, static_cast<cudaStream_t>(stream));
}

namespace {

// Copy streams and events of dirotq_linear_host, created once per device (no device memory involved).
struct HostPipe {
    bool ready = false;
    cudaStream_t h2d = nullptr, d2h = nullptr;
    static constexpr int kMaxChunks = 8;
    cudaEvent_t start = nullptr, done = nullptr, copied[kMaxChunks] = {}, computed[kMaxChunks] = {};
};
std::mutex g_pipe_mutex;
HostPipe g_pipe[64];

// Caller holds g_pipe_mutex (also while it enqueues on the pipe: its events are shared by all calls on the device).
dirotq_status_t host_pipe(int dev, HostPipe** out) {
    if (dev < 0 || dev >= 64) return DIROTQ_ERR_INVALID_ARG;
    HostPipe& p = g_pipe[dev];
    if (!p.ready) {
        cudaError_t e = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming);
        for (int i = 0; i < HostPipe::kMaxChunks && e == cudaSuccess; ++i) {
            e = cudaEventCreateWithFlags(&p.copied[i], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p.computed[i], cudaEventDisableTiming);
        }
        if (e != cudaSuccess) { set_error("host pipeline set-up", e); return DIROTQ_ERR_CUDA; }
        p.ready = true;
    }
    *out = &p;
    return DIROTQ_OK;
}

}  // namespace

dirotq_status_t dirotq_linear_host(const void* x_host, int M, const dirotq_layer_t* layer, void* y_host, void* x_dev,
                                   void* y_dev, void* workspace, size_t workspace_bytes, dirotq_stream_t stream) {
    dirotq_status_t st = check_call(layer, M, workspace, workspace_bytes);
    if (st != DIROTQ_OK) return st;
    if (!x_host || !y_host || !x_dev || !y_dev) return DIROTQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t xrow = static_cast<size_t>(layer->geo.K) * 2, yrow = static_cast<size_t>(layer->geo.N) * 2;
    // Token rows are independent: the call is cut into row chunks whose host-to-device copy, computation and
    // device-to-host copy overlap (copy engines in both directions + SMs).  The chunks' kernels run one after another on
    // `stream`, so they can share the workspace.
    int chunks = M / 1024;
    if (chunks > HostPipe::kMaxChunks) chunks = HostPipe::kMaxChunks;
    if (chunks <= 1) {
        cudaError_t e = cudaMemcpyAsync(x_dev, x_host, xrow * M, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) { set_error("cudaMemcpyAsync(H2D)", e); return DIROTQ_ERR_CUDA; }
        st = dirotq_linear(x_dev, M, layer, y_dev, workspace, workspace_bytes, stream);
        if (st != DIROTQ_OK) return st;
        e = cudaMemcpyAsync(y_host, y_dev, yrow * M, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) { set_error("cudaMemcpyAsync(D2H)", e); return DIROTQ_ERR_CUDA; }
        return DIROTQ_OK;
    }
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe* p = nullptr;
    st = host_pipe(layer->device, &p);
    if (st != DIROTQ_OK) return st;
    const int rows_per_chunk = ((M + chunks - 1) / chunks + 127) / 128 * 128;
    cudaError_t e = cudaEventRecord(p->start, s);  // the staging buffers may still be in use by earlier work on `stream`
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p->h2d, p->start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(p->d2h, p->start, 0);
    int c = 0;
    for (int m0 = 0; m0 < M && e == cudaSuccess; m0 += rows_per_chunk, ++c) {
        const int mc = M - m0 < rows_per_chunk ? M - m0 : rows_per_chunk;
        char* xd = static_cast<char*>(x_dev) + xrow * m0;
        char* yd = static_cast<char*>(y_dev) + yrow * m0;
        e = cudaMemcpyAsync(xd, static_cast<const char*>(x_host) + xrow * m0, xrow * mc, cudaMemcpyHostToDevice, p->h2d);
        if (e == cudaSuccess) e = cudaEventRecord(p->copied[c], p->h2d);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, p->copied[c], 0);
        if (e != cudaSuccess) break;
        st = dirotq_linear(xd, mc, layer, yd, workspace, workspace_bytes, stream);
        if (st != DIROTQ_OK) return st;
        e = cudaEventRecord(p->computed[c], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(p->d2h, p->computed[c], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(static_cast<char*>(y_host) + yrow * m0, yd, yrow * mc, cudaMemcpyDeviceToHost, p->d2h);
    }
    if (e == cudaSuccess) e = cudaEventRecord(p->done, p->d2h);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, p->done, 0);  // later work on `stream` (and its synchronisation) sees y_host
    if (e != cudaSuccess) { set_error("host pipeline", e); return DIROTQ_ERR_CUDA; }
    return DIROTQ_OK;
}

dirotq_status_t dirotq_workspace_status(const void* workspace, dirotq_stream_t stream, int* device_code) {
    if (!workspace) return DIROTQ_ERR_INVALID_ARG;
    int code = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&code, workspace, sizeof code, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { set_error("status read", e); return DIROTQ_ERR_CUDA; }
    if (device_code) *device_code = code;
    return code == 0 ? DIROTQ_OK : DIROTQ_ERR_DEVICE_TIMEOUT;
}

dirotq_status_t dirotq_workspace_wait_counters(const void* workspace, dirotq_stream_t stream, unsigned long long out[8]) {
    if (!workspace || !out) return DIROTQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(out, static_cast<const char*>(workspace) + 8, 8 * sizeof(unsigned long long),
                                    cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { set_error("wait counter read", e); return DIROTQ_ERR_CUDA; }
    return DIROTQ_OK;
}

dirotq_status_t dirotq_workspace_export(const dirotq_layer_t* layer, int M, const void* workspace, void* xh_bf16,
                                        int8_t* codes, void* scales_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || (layer->geo.fmt != 0 && layer->geo.fmt != 4) || !workspace || M < 1 || M > 65535) return DIROTQ_ERR_INVALID_ARG;
    return launch_workspace_export(layer, M, static_cast<const char*>(workspace), static_cast<uint16_t*>(xh_bf16), codes,
                                   static_cast<uint16_t*>(scales_bf16), static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_int_gemm_debug(const int8_t* act_codes, int M, const dirotq_layer_t* layer, int32_t* partials,
                                      void* workspace, size_t workspace_bytes, dirotq_stream_t stream) {
    dirotq_status_t st = check_call(layer, M, workspace, workspace_bytes, false);
    if (st != DIROTQ_OK) return st;
    if (layer->geo.fmt == 1) return DIROTQ_ERR_INVALID_ARG;
    if (layer->geo.fmt == 3) {  // one sum per output: partials [M][N]; the caller's codes are read in place
        if (!act_codes || !partials || !aligned16(act_codes) || !aligned16(partials)) return DIROTQ_ERR_INVALID_ARG;
        const WorkspaceLayoutA8 w8 = make_workspace_layout_w4a8(layer->geo, M);
        char* ws8 = static_cast<char*>(workspace);
        A8GemmArgs ga;
        ga.M = M; ga.codes = act_codes; ga.xscale = reinterpret_cast<const float*>(ws8 + w8.off_xscale);
        ga.xh = reinterpret_cast<const uint16_t*>(ws8 + w8.off_xh);
        ga.y = nullptr; ga.partials = partials; ga.status = reinterpret_cast<int*>(ws8 + w8.off_status);
        return launch_w4a8_gemm(layer, ga, static_cast<cudaStream_t>(stream));
    }
    if (!act_codes || !partials || !aligned16(act_codes) || !aligned16(partials)) return DIROTQ_ERR_INVALID_ARG;
    char* ws = static_cast<char*>(workspace);
    const WorkspaceLayout w = make_workspace_layout(layer->geo, M);
    st = launch_debug_codes(layer, M, act_codes, ws, static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) return st;
    GemmArgs ga;
    ga.M = M; ga.codes = reinterpret_cast<const int8_t*>(ws + w.off_codes);
    ga.xscale = reinterpret_cast<const float*>(ws + w.off_xscale);
    ga.ldm = w.ldm;
    ga.xh = reinterpret_cast<const uint16_t*>(ws + w.off_xh);
    ga.y = nullptr; ga.partials = partials;
    ga.status = reinterpret_cast<int*>(ws + w.off_status);
    return launch_w4a4_gemm(layer, ga, static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_export(const dirotq_layer_t* layer, int8_t* wcodes, void* wscales_bf16, void* wh_bf16,
                                    void* q_bf16, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt == 1) return DIROTQ_ERR_INVALID_ARG;
    if (q_bf16 && (layer->geo.no_rot || layer->geo.fmt == 4)) return DIROTQ_ERR_INVALID_ARG;  // no K x K rotation in the blob
    return launch_layer_export(layer, wcodes, static_cast<uint16_t*>(wscales_bf16), static_cast<uint16_t*>(wh_bf16),
                               static_cast<uint16_t*>(q_bf16), static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------- NVFP4 variant

dirotq_status_t dirotq_layer_bytes_nvfp4(int K, int N, int r, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    *bytes = make_blob_layout_nvfp4(make_geometry(K, N, r, 64)).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_nvfp4(const void* W, int w_dtype, int w_layout, const void* Q, int q_dtype,
                                           const void* bias, int K, int N, int r, int act_scale_log2, void* blob,
                                           size_t blob_bytes, void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                           dirotq_layer_t** layer_out) {
    if (!W || !Q || !blob || !scratch || !layer_out) return DIROTQ_ERR_INVALID_ARG;
    if (w_dtype != DIROTQ_DTYPE_F32 && w_dtype != DIROTQ_DTYPE_BF16) return DIROTQ_ERR_INVALID_ARG;
    if (q_dtype != DIROTQ_DTYPE_F64 && q_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    if (w_layout != DIROTQ_LAYOUT_KN && w_layout != DIROTQ_LAYOUT_NK) return DIROTQ_ERR_INVALID_ARG;
    if (act_scale_log2 < -100 || act_scale_log2 > 100) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    if (!aligned16(W) || !aligned16(Q) || !aligned16(scratch) || (bias && !aligned16(bias))) return DIROTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    Geometry g = make_geometry(K, N, r, 64);
    g.fmt = 1;
    const BlobLayout lay = make_blob_layout_nvfp4(g);
    if (blob_bytes < lay.total) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (scratch_bytes < static_cast<size_t>(K) * N * sizeof(double)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    int dev = 0;
    st = check_device(&dev);
    if (st != DIROTQ_OK) return st;
    dirotq_layer* L = new (std::nothrow) dirotq_layer;
    if (!L) return DIROTQ_ERR_INVALID_ARG;
    memset(L, 0, sizeof *L);
    L->magic = kLayerMagic;
    L->device = dev;
    L->geo = g;
    L->lay = lay;
    L->blob = static_cast<char*>(blob);
    L->act_scale_log2 = act_scale_log2;
    st = encode_tmap_2d(&L->tmap_qt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                        (uint64_t)K * 2, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                            (uint64_t)K * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt64, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K, (uint64_t)K,
                            (uint64_t)K * 2, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked, (uint64_t)g.K4 / 2,
                            (uint64_t)N, (uint64_t)g.K4 / 2, 128, kNvfp4BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, kNvfp4BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = launch_prepare_nvfp4(L, W, w_dtype, w_layout, Q, q_dtype, bias, static_cast<double*>(scratch),
                                  static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) {
        delete L;
        return st;
    }
    *layer_out = L;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_workspace_export_nvfp4(const dirotq_layer_t* layer, int M, const void* workspace, void* xh_bf16,
                                              uint8_t* codes, uint8_t* scales_e4m3, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt != 1 || !workspace || M < 1 || M > 65535) return DIROTQ_ERR_INVALID_ARG;
    return launch_workspace_export_nvfp4(layer, M, static_cast<const char*>(workspace), static_cast<uint16_t*>(xh_bf16), codes,
                                         scales_e4m3, static_cast<cudaStream_t>(stream));
}

dirotq_status_t dirotq_layer_bytes_nvfp4_ph(int K, int N, int r, size_t* bytes) {
    if (!bytes) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    Geometry g = make_geometry(K, N, r, 64);
    make_ph_nvfp4(g);
    *bytes = make_blob_layout_nvfp4(g).total;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_prepare_layer_nvfp4_ph(const void* W, int w_dtype, int w_layout, const void* Uh, int uh_dtype,
                                              const void* bias, int K, int N, int r, int act_scale_log2, void* blob,
                                              size_t blob_bytes, void* scratch, size_t scratch_bytes, dirotq_stream_t stream,
                                              dirotq_layer_t** layer_out) {
    if (!W || !Uh || !blob || !scratch || !layer_out) return DIROTQ_ERR_INVALID_ARG;
    if (w_dtype != DIROTQ_DTYPE_F32 && w_dtype != DIROTQ_DTYPE_BF16) return DIROTQ_ERR_INVALID_ARG;
    if (uh_dtype != DIROTQ_DTYPE_F64 && uh_dtype != DIROTQ_DTYPE_F32) return DIROTQ_ERR_INVALID_ARG;
    if (w_layout != DIROTQ_LAYOUT_KN && w_layout != DIROTQ_LAYOUT_NK) return DIROTQ_ERR_INVALID_ARG;
    if (act_scale_log2 < -100 || act_scale_log2 > 100) return DIROTQ_ERR_INVALID_ARG;
    dirotq_status_t st = check_shape(K, N, r, 64);
    if (st != DIROTQ_OK) return st;
    if (!aligned16(W) || !aligned16(Uh) || !aligned16(scratch) || (bias && !aligned16(bias))) return DIROTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(blob) & (kAlign - 1)) != 0) return DIROTQ_ERR_INVALID_ARG;
    Geometry g = make_geometry(K, N, r, 64);
    make_ph_nvfp4(g);
    const BlobLayout lay = make_blob_layout_nvfp4(g);
    if (blob_bytes < lay.total) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    if (scratch_bytes < (static_cast<size_t>(K) + r) * N * sizeof(double)) return DIROTQ_ERR_BUFFER_TOO_SMALL;
    int dev = 0;
    st = check_device(&dev);
    if (st != DIROTQ_OK) return st;
    dirotq_layer* L = new (std::nothrow) dirotq_layer;
    if (!L) return DIROTQ_ERR_INVALID_ARG;
    memset(L, 0, sizeof *L);
    L->magic = kLayerMagic;
    L->device = dev;
    L->geo = g;
    L->lay = lay;
    L->blob = static_cast<char*>(blob);
    L->act_scale_log2 = act_scale_log2;
    st = encode_tmap_2d(&L->tmap_qt128, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_qt, (uint64_t)K,
                        (uint64_t)g.r_pad, (uint64_t)K * 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_qt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_uh, (uint64_t)g.r_pad,
                            (uint64_t)K, (uint64_t)g.r_pad * 2, 64, 256, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_had, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_had, (uint64_t)g.G,
                            (uint64_t)g.G, (uint64_t)g.G * 2, 64, g.G, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wpacked, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, L->blob + lay.off_wpacked, (uint64_t)g.K4 / 2,
                            (uint64_t)N, (uint64_t)g.K4 / 2, 128, kNvfp4BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = encode_tmap_2d(&L->tmap_wh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, L->blob + lay.off_wh, (uint64_t)g.r_pad,
                            (uint64_t)N, (uint64_t)g.r_pad * 2, 64, kNvfp4BN, CU_TENSOR_MAP_SWIZZLE_128B);
    if (st == DIROTQ_OK)
        st = launch_prepare_nvfp4_ph(L, W, w_dtype, w_layout, Uh, uh_dtype, bias, static_cast<double*>(scratch),
                                     static_cast<cudaStream_t>(stream));
    if (st != DIROTQ_OK) {
        delete L;
        return st;
    }
    *layer_out = L;
    return DIROTQ_OK;
}

dirotq_status_t dirotq_layer_export_nvfp4(const dirotq_layer_t* layer, uint8_t* wcodes, uint8_t* wscales_e4m3, void* wh_bf16,
                                          void* q_bf16, int* weight_scale_log2, dirotq_stream_t stream) {
    if (!valid_layer(layer) || layer->geo.fmt != 1) return DIROTQ_ERR_INVALID_ARG;
    if (q_bf16 && layer->geo.ph) return DIROTQ_ERR_INVALID_ARG;  // no K x K rotation in the blob
    return launch_layer_export_nvfp4(layer, wcodes, wscales_e4m3, static_cast<uint16_t*>(wh_bf16),
                                     static_cast<uint16_t*>(q_bf16), weight_scale_log2, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
