// Host side of the C ABI: argument checks, tensor maps, workspace carving, launches.
#include "internal.cuh"

#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

using namespace rudder;

namespace rudder {
int device_sm_count()
{
    static std::atomic<int> cache[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}
}  // namespace rudder

namespace {

// ---- cuTensorMapEncodeTiled through the runtime (no link-time dependency on the driver library) --
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Row-major 2D tensor [rows, cols] of `esize`-byte elements; box = {box_cols, box_rows}.
bool make_tmap_2d(CUtensorMap* tm, CUtensorMapDataType dt, int esize, const void* base, uint64_t cols, uint64_t rows,
                  uint64_t row_stride_bytes, uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    (void)esize;
    cuuint64_t gdim[2] = {cols, rows};
    cuuint64_t gstride[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(tm, dt, 2, const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Block scales in the tensor core's order seen as [atoms][K/64][128 words of 4 bytes]; box = {128, 4, box_atoms}:
// the four 512-byte chunks of one 256-channel stage, for box_atoms 128-row atoms.
bool make_tmap_sf(CUtensorMap* tm, const void* base, uint64_t k64, uint64_t atoms, uint32_t box_atoms)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {128, k64, atoms};
    cuuint64_t gstride[2] = {512, k64 * 512};
    cuuint32_t box[3] = {128, 4, box_atoms};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Per-device state created on first use (function attributes, SM count, copy streams, the address of the
// static workspace): guarded by one mutex, so that host threads may make their first calls concurrently.
std::mutex g_state_mutex;
bool g_gemm_ready[64] = {false};


int sm_count() { return rudder::device_sm_count(); }

rudder_status ensure_init()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RUDDER_ERR_CUDA;
    if (dev < 0 || dev >= 64) return RUDDER_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_state_mutex);
    if (!g_gemm_ready[dev]) {
        if (gemm_i8_init() != cudaSuccess || gemm_fp4_init() != cudaSuccess || actq_init() != cudaSuccess) return RUDDER_ERR_CUDA;
        g_gemm_ready[dev] = true;
    }
    return RUDDER_OK;
}

// A packed weight lives on the device that was current when it was packed; every call that launches on it
// must be made with that device current (its tensor maps and pointers mean nothing elsewhere).
bool on_weights_device(const rudder_weight* w)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == w->device;
}

rudder_status check_table_and_segments(const rudder_segments* seg, int step, const rudder_scale_table* tab, int M,
                                       SegParams* out)
{
    if (!seg || !tab || !tab->gamma || !seg->seg_offsets || !seg->seg_stream) return RUDDER_ERR_ARG;
    if (tab->T < 1 || tab->S < 1 || tab->S > kMaxStreams) return RUDDER_ERR_ARG;
    if (step < 0 || step >= tab->T) return RUDDER_ERR_ARG;
    if (tab->mode != RUDDER_RANGE_PER_TOKEN && tab->mode != RUDDER_RANGE_STATIC) return RUDDER_ERR_ARG;
    if (tab->mode == RUDDER_RANGE_STATIC && !tab->clip) return RUDDER_ERR_ARG;
    if (seg->n_seg < 1 || seg->n_seg > kMaxSeg) return RUDDER_ERR_ARG;
    if (seg->seg_offsets[0] != 0 || seg->seg_offsets[seg->n_seg] != M) return RUDDER_ERR_ARG;
    out->n_seg = seg->n_seg;
    for (int i = 0; i < seg->n_seg; ++i) {
        if (seg->seg_offsets[i + 1] < seg->seg_offsets[i]) return RUDDER_ERR_ARG;
        if (seg->seg_stream[i] < 0 || seg->seg_stream[i] >= tab->S) return RUDDER_ERR_ARG;
        out->offset[i] = seg->seg_offsets[i];
        out->stream[i] = seg->seg_stream[i];
    }
    out->offset[seg->n_seg] = M;
    for (int i = seg->n_seg + 1; i <= kMaxSeg; ++i) out->offset[i] = M;
    for (int i = seg->n_seg; i < kMaxSeg; ++i) out->stream[i] = 0;
    return RUDDER_OK;
}

int qmax_of(int scheme) { return scheme == RUDDER_W4A8_INT ? 127 : 7; }

size_t workspace_bytes_for(const rudder_weight* w, int M)
{
    if (!w || M < 1) return 0;
    const size_t r = align_up(static_cast<size_t>(M) * sizeof(float), 256);
    if (w->scheme == RUDDER_W4A4_NVFP4) {
        // packed E2M1 codes [M, K/2], block scales in tiled order for ceil(M/128) atoms, row scales
        const size_t codes = align_up(static_cast<size_t>(M) * (w->K / 2), 256);
        const size_t sf = align_up(static_cast<size_t>((M + 127) / 128) * (w->K / 64) * 512, 256);
        return codes + sf + r;
    }
    const size_t codes = align_up(static_cast<size_t>(M) * w->K, 256);
    return codes + r + gemm_i8_scratch_bytes(M, w->N, w->K, false, nullptr);
}

rudder_status linear_impl(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M, const rudder_segments* seg,
                          int step, const rudder_scale_table* tab, const float* bias, uint16_t* Y, int64_t ldy,
                          void* workspace, size_t workspace_bytes, cudaStream_t st, int32_t* acc, int row0, int rows,
                          int col0, int cols, cudaEvent_t* ev = nullptr /* ev[1] recorded after the prologue, ev[2] after the GEMM */,
                          bool gelu_first = false /* X is the tensor before the GELU: the prologue applies it (static range only) */)
{
    if (!w || !X || !Y) return RUDDER_ERR_ARG;
    if (!on_weights_device(w)) return RUDDER_ERR_ARG;
    if (M < 1) return RUDDER_ERR_SHAPE;
    SegParams sp;
    rudder_status s = check_table_and_segments(seg, step, tab, M, &sp);
    if (s != RUDDER_OK) return s;
    if (!aligned(X, 16) || !aligned(Y, 16) || ldx % 8 != 0 || ldy % 8 != 0 || ldx < w->K || ldy < w->N) return RUDDER_ERR_ALIGN;
    if (bias && !aligned(bias, 16)) return RUDDER_ERR_ALIGN;
    if (w->scheme == RUDDER_W4A4_NVFP4 && acc) return RUDDER_ERR_UNSUPPORTED;   // fp32 accumulation: nothing exact to dump
    const size_t need = workspace_bytes_for(w, M);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return RUDDER_ERR_WORKSPACE;
    if (acc) {
        if (rows < 1 || cols < 1 || row0 < 0 || col0 < 0 || row0 % 128 != 0 || col0 % 64 != 0) return RUDDER_ERR_ARG;
    }
    s = ensure_init();
    if (s != RUDDER_OK) return s;

    ActqArgs a;
    a.zero_ints = nullptr; a.n_zero = 0;
    a.X = X; a.ldx = ldx; a.M = M; a.K = w->K; a.dinv = w->dinv;
    a.gamma_step = tab->gamma + static_cast<size_t>(step) * tab->S;
    a.clip_step = (tab->mode == RUDDER_RANGE_STATIC) ? tab->clip + step : nullptr;
    a.seg = sp;

    if (gelu_first && (a.clip_step == nullptr || w->scheme == RUDDER_W4A4_NVFP4)) return RUDDER_ERR_UNSUPPORTED;
    if (w->scheme == RUDDER_W4A4_NVFP4) {
        uint8_t* ws = static_cast<uint8_t*>(workspace);
        uint8_t* codes4 = ws;
        uint8_t* sfx = ws + align_up(static_cast<size_t>(M) * (w->K / 2), 256);
        float* r4 = reinterpret_cast<float*>(sfx + align_up(static_cast<size_t>((M + 127) / 128) * (w->K / 64) * 512, 256));
        if (launch_actq_nvfp4(a, codes4, sfx, true, r4, st) != cudaSuccess) return RUDDER_ERR_CUDA;
        if (ev && cudaEventRecord(ev[1], st) != cudaSuccess) return RUDDER_ERR_CUDA;
        GemmFp4Args g;
        const bool pair = gemm_fp4_use_pair(M, w->N, w->K);
        const int tt = pair ? 128 : gemm_fp4_token_tile(M, w->N);      // token rows of one activation box
        const int st_rows = pair ? 64 : gemm_fp4_store_rows(M, w->N);  // token rows of one output store box
        const uint32_t box_tok = static_cast<uint32_t>(M < tt ? M : tt);
        const uint64_t kb = static_cast<uint64_t>(w->K / 2);
        if (!make_tmap_2d(&g.tm_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes4, kb, static_cast<uint64_t>(M), kb, 128, box_tok,
                          CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap_2d(&g.tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w->codes, kb, static_cast<uint64_t>(w->N), kb, 128,
                          static_cast<uint32_t>(w->N < 128 ? w->N : 128), CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tmap_2d(&g.tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, static_cast<uint64_t>(w->N), static_cast<uint64_t>(M),
                          static_cast<uint64_t>(ldy) * 2, static_cast<uint32_t>(w->N < 128 ? w->N : 128),
                          static_cast<uint32_t>(M < st_rows ? M : st_rows), CU_TENSOR_MAP_SWIZZLE_NONE))
            return RUDDER_ERR_CUDA;
        if (pair && (!make_tmap_sf(&g.tm_sfx, sfx, static_cast<uint64_t>(w->K / 64), static_cast<uint64_t>((M + 127) / 128), 2) ||
                     !make_tmap_sf(&g.tm_sfw, w->sf_tiled, static_cast<uint64_t>(w->K / 64), static_cast<uint64_t>((w->N + 127) / 128), 1)))
            return RUDDER_ERR_CUDA;
        g.sm_count = sm_count();
        g.sf_x = sfx; g.sf_w = w->sf_tiled;
        g.M = M; g.N = w->N; g.K = w->K;
        g.row_scale = r4; g.tensor_scale = w->tensor_scale; g.bias = bias;
        if (launch_gemm_fp4(g, st) != cudaSuccess) return RUDDER_ERR_CUDA;
        if (ev && cudaEventRecord(ev[2], st) != cudaSuccess) return RUDDER_ERR_CUDA;
        return RUDDER_OK;
    }

    int8_t* codes = static_cast<int8_t*>(workspace);
    float* r = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + align_up(static_cast<size_t>(M) * w->K, 256));
    if (gemm_i8_register_path(M, w->N, w->K, w->G, w->f8 != 0)) {
        // Up to a few hundred rows: the light prologue (int8 codes, whatever the weight layout) and a register-level GEMM.
        if ((gelu_first ? launch_actq_gelu_static(a, qmax_of(w->scheme), false, codes, w->K, r, sm_count(), st)
                        : launch_actq_int(a, qmax_of(w->scheme), false, codes, w->K, r, st)) != cudaSuccess) return RUDDER_ERR_CUDA;
        if (ev && cudaEventRecord(ev[1], st) != cudaSuccess) return RUDDER_ERR_CUDA;
        GemmI8FewRowsArgs f;
        f.codes = codes; f.ldc = w->K; f.row_scale = r; f.wq = w->codes; f.signmag = w->f8 != 0;
        f.w_scales_t = w->scales_t; f.bias = bias; f.Y = Y; f.ldy = ldy;
        f.M = M; f.N = w->N; f.K = w->K; f.G = w->G;
        f.acc = acc; f.row0 = row0; f.rows = rows; f.col0 = col0; f.cols = cols;
        if ((gemm_i8_fewrows_applies(M, w->N, w->K, w->G) ? launch_gemm_i8_fewrows(f, st) : launch_gemm_i8_midrows(f, st)) != cudaSuccess) return RUDDER_ERR_CUDA;
        if (ev && cudaEventRecord(ev[2], st) != cudaSuccess) return RUDDER_ERR_CUDA;
        return RUDDER_OK;
    }
    const GemmI8Plan plan = gemm_i8_plan(M, w->N, w->K, w->G, w->f8 != 0, acc != nullptr);
    GemmI8Args g;
    g.partials = nullptr; g.counters = nullptr;
    if (plan.splitk > 1) {
        size_t counters_off = 0;
        gemm_i8_scratch_bytes(M, w->N, w->K, false, &counters_off);
        uint8_t* scratch = reinterpret_cast<uint8_t*>(r) + align_up(static_cast<size_t>(M) * sizeof(float), 256);
        g.partials = reinterpret_cast<float*>(scratch);
        g.counters = reinterpret_cast<int*>(scratch + counters_off);
        a.zero_ints = g.counters;
        a.n_zero = ((M + plan.token_tile - 1) / plan.token_tile) * ((w->N + 127) / 128);
    }
    if ((gelu_first ? launch_actq_gelu_static(a, qmax_of(w->scheme), w->f8 != 0, codes, w->K, r, sm_count(), st)
                    : launch_actq_int(a, qmax_of(w->scheme), w->f8 != 0, codes, w->K, r, st)) != cudaSuccess) return RUDDER_ERR_CUDA;
    if (ev && cudaEventRecord(ev[1], st) != cudaSuccess) return RUDDER_ERR_CUDA;

    const int tt = plan.token_tile;
    const uint32_t box_tok = static_cast<uint32_t>(M < tt ? M : tt);
    if (!make_tmap_2d(&g.tm_x, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, codes, static_cast<uint64_t>(w->K), static_cast<uint64_t>(M),
                      static_cast<uint64_t>(w->K), 128, box_tok, CU_TENSOR_MAP_SWIZZLE_128B))
        return RUDDER_ERR_CUDA;
    if (!make_tmap_2d(&g.tm_y, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Y, static_cast<uint64_t>(w->N), static_cast<uint64_t>(M),
                      static_cast<uint64_t>(ldy) * 2, static_cast<uint32_t>(w->N < 128 ? w->N : 128),
                      plan.persist ? 64u : box_tok, CU_TENSOR_MAP_SWIZZLE_NONE))
        return RUDDER_ERR_CUDA;
    g.sm_count = sm_count();
    g.w_scales_t = w->scales_t; g.tm_w = w->tm_codes; g.f8 = w->f8 != 0;
    g.y = Y; g.ldy = ldy;
    g.M = M; g.N = w->N; g.K = w->K; g.G = w->G;
    g.row_scale = r; g.bias = bias;
    g.acc = acc; g.row0 = row0; g.rows = rows; g.col0 = col0; g.cols = cols;
    if (launch_gemm_i8(g, st) != cudaSuccess) return RUDDER_ERR_CUDA;
    if (ev && cudaEventRecord(ev[2], st) != cudaSuccess) return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

}  // namespace

extern "C" {

const char* rudder_status_string(rudder_status s)
{
    switch (s) {
        case RUDDER_OK: return "ok";
        case RUDDER_ERR_ARG: return "invalid argument";
        case RUDDER_ERR_SHAPE: return "unsupported shape";
        case RUDDER_ERR_ALIGN: return "misaligned pointer or leading dimension";
        case RUDDER_ERR_UNSUPPORTED: return "unsupported scheme or mode";
        case RUDDER_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case RUDDER_ERR_CUDA: return "CUDA call failed";
        case RUDDER_ERR_TIMEOUT: return "bounded device-side wait gave up";
    }
    return "unknown status";
}

// Shape / scheme checks shared by pack and import; normalises `group` (16 for NVFP4).
static rudder_status check_weight_shape(int N, int K, rudder_scheme scheme, int* group)
{
    if (N < 64 || N % 64 != 0 || K < 128 || K % 128 != 0) return RUDDER_ERR_SHAPE;
    if (scheme != RUDDER_W4A8_INT && scheme != RUDDER_W4A4_INT && scheme != RUDDER_W4A4_NVFP4) return RUDDER_ERR_UNSUPPORTED;
    if (scheme == RUDDER_W4A4_NVFP4) {
        if (K % 256 != 0) return RUDDER_ERR_SHAPE;        // the block-scaled GEMM moves 256 input channels per stage
        *group = 16;
    } else if (!(*group == 64 || *group == 128 || *group == K)) {
        return RUDDER_ERR_SHAPE;
    }
    return RUDDER_OK;
}

// Allocates the handle and its device arrays (nothing is filled in).  nullptr if an allocation failed.
static rudder_weight* alloc_weight(int N, int K, rudder_scheme scheme, int group)
{
    rudder_weight* w = static_cast<rudder_weight*>(calloc(1, sizeof(rudder_weight)));
    if (!w) return nullptr;
    w->N = N; w->K = K; w->G = group; w->scheme = scheme;
    cudaGetDevice(&w->device);
    const size_t n_groups = static_cast<size_t>(K / group);
    const size_t code_bytes = static_cast<size_t>(N) * (K / 2);
    bool ok = cudaMalloc(&w->codes, code_bytes) == cudaSuccess &&
              cudaMalloc(&w->dinv, static_cast<size_t>(K) * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&w->tensor_scale, sizeof(float)) == cudaSuccess;
    if (scheme == RUDDER_W4A4_NVFP4) {
        const size_t sf_bytes = static_cast<size_t>((N + 127) / 128) * (K / 64) * 512;
        ok = ok && cudaMalloc(&w->scales_c, n_groups * N) == cudaSuccess && cudaMalloc(&w->sf_tiled, sf_bytes) == cudaSuccess;
        w->bytes = code_bytes + n_groups * N + sf_bytes + static_cast<size_t>(K) * sizeof(float) + sizeof(float);
    } else {
        // W4A4 with group scales: |C^(g)| <= 128 * 49, so E4M3 operands and FP32 accumulators hold the
        // integers exactly and the per-group drain needs no integer-to-float conversion.
        w->f8 = (scheme == RUDDER_W4A4_INT && group <= 128) ? 1 : 0;
        ok = ok && cudaMalloc(&w->scales_t, n_groups * N * sizeof(float)) == cudaSuccess &&
             cudaMalloc(&w->scales_c, n_groups * N * sizeof(uint16_t)) == cudaSuccess &&
             cudaMalloc(&w->tm_codes, sizeof(CUtensorMap)) == cudaSuccess;
        w->bytes = code_bytes + n_groups * N * (sizeof(float) + sizeof(uint16_t)) + static_cast<size_t>(K) * sizeof(float) + sizeof(float);
    }
    if (!ok) {
        rudder_weight_free(w);
        return nullptr;
    }
    return w;
}

// Integer schemes: the tensor map over the packed codes, kept in device memory so that the GEMM takes it by pointer.
static bool finish_int4(rudder_weight* w)
{
    CUtensorMap tm;
    return make_tmap_2d(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, w->codes, static_cast<uint64_t>(w->K / 2), static_cast<uint64_t>(w->N),
                        static_cast<uint64_t>(w->K / 2), 64, static_cast<uint32_t>(w->N < 128 ? w->N : 128), CU_TENSOR_MAP_SWIZZLE_NONE) &&
           cudaMemcpy(w->tm_codes, &tm, sizeof(CUtensorMap), cudaMemcpyHostToDevice) == cudaSuccess;
}

rudder_status rudder_pack_weights(const float* W, const float* d, int N, int K, rudder_scheme scheme, int group,
                                  void* stream, rudder_weight** out)
{
    if (out) *out = nullptr;
    if (!W || !out) return RUDDER_ERR_ARG;
    rudder_status s = check_weight_shape(N, K, scheme, &group);
    if (s != RUDDER_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_init();
    if (s != RUDDER_OK) return s;
    rudder_weight* w = alloc_weight(N, K, scheme, group);
    if (!w) return RUDDER_ERR_CUDA;
    bool ok;
    if (scheme == RUDDER_W4A4_NVFP4) {
        const size_t sf_bytes = static_cast<size_t>((N + 127) / 128) * (K / 64) * 512;
        unsigned int* amax_bits = nullptr;
        ok = cudaMalloc(&amax_bits, sizeof(unsigned int)) == cudaSuccess &&
             launch_pack_nvfp4(W, d, N, K, w->codes, static_cast<uint8_t*>(w->scales_c), w->sf_tiled, sf_bytes, w->dinv,
                               w->tensor_scale, amax_bits, st) == cudaSuccess &&
             cudaStreamSynchronize(st) == cudaSuccess;
        if (amax_bits) cudaFree(amax_bits);
    } else {
        int8_t* tmp = nullptr;
        const float one = 1.0f;
        ok = cudaMalloc(&tmp, static_cast<size_t>(N) * K) == cudaSuccess &&
             cudaMemcpyAsync(w->tensor_scale, &one, sizeof(float), cudaMemcpyHostToDevice, st) == cudaSuccess &&
             launch_pack_int4(W, d, N, K, group, w->codes, w->scales_t, static_cast<uint16_t*>(w->scales_c), w->dinv, tmp, w->f8 != 0, st) == cudaSuccess &&
             cudaStreamSynchronize(st) == cudaSuccess;
        if (tmp) cudaFree(tmp);
        ok = ok && finish_int4(w);
    }
    if (!ok) {
        rudder_weight_free(w);
        return RUDDER_ERR_CUDA;
    }
    *out = w;
    return RUDDER_OK;
}

rudder_status rudder_weight_import(const uint8_t* codes, const void* scales, const float* dinv, const float* tensor_scale,
                                   int N, int K, rudder_scheme scheme, int group, void* stream, rudder_weight** out)
{
    if (out) *out = nullptr;
    if (!codes || !scales || !dinv || !out) return RUDDER_ERR_ARG;
    if (scheme == RUDDER_W4A4_NVFP4 && !tensor_scale) return RUDDER_ERR_ARG;
    rudder_status s = check_weight_shape(N, K, scheme, &group);
    if (s != RUDDER_OK) return s;
    if (!aligned(codes, 4) || !aligned(scales, 2)) return RUDDER_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    s = ensure_init();
    if (s != RUDDER_OK) return s;
    rudder_weight* w = alloc_weight(N, K, scheme, group);
    if (!w) return RUDDER_ERR_CUDA;
    const size_t n_groups = static_cast<size_t>(K / group);
    bool ok = cudaMemcpyAsync(w->dinv, dinv, static_cast<size_t>(K) * sizeof(float), cudaMemcpyDeviceToDevice, st) == cudaSuccess;
    if (scheme == RUDDER_W4A4_NVFP4) {
        const size_t sf_bytes = static_cast<size_t>((N + 127) / 128) * (K / 64) * 512;
        ok = ok && cudaMemcpyAsync(w->codes, codes, static_cast<size_t>(N) * (K / 2), cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(w->scales_c, scales, n_groups * N, cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(w->tensor_scale, tensor_scale, sizeof(float), cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
             launch_import_nvfp4_scales(static_cast<const uint8_t*>(scales), N, K, w->sf_tiled, sf_bytes, st) == cudaSuccess &&
             cudaStreamSynchronize(st) == cudaSuccess;
    } else {
        int8_t* tmp = nullptr;
        const float one = 1.0f;
        ok = ok && cudaMalloc(&tmp, static_cast<size_t>(N) * K) == cudaSuccess &&
             cudaMemcpyAsync(w->tensor_scale, &one, sizeof(float), cudaMemcpyHostToDevice, st) == cudaSuccess &&
             cudaMemcpyAsync(w->scales_c, scales, n_groups * N * sizeof(uint16_t), cudaMemcpyDeviceToDevice, st) == cudaSuccess &&
             launch_import_int4(codes, static_cast<const uint16_t*>(scales), N, K, group, w->codes, w->scales_t, tmp, w->f8 != 0, st) == cudaSuccess &&
             cudaStreamSynchronize(st) == cudaSuccess;
        if (tmp) cudaFree(tmp);
        ok = ok && finish_int4(w);
    }
    if (!ok) {
        rudder_weight_free(w);
        return RUDDER_ERR_CUDA;
    }
    *out = w;
    return RUDDER_OK;
}

rudder_status rudder_weight_free(rudder_weight* w)
{
    if (!w) return RUDDER_OK;
    cudaFree(w->codes);
    cudaFree(w->scales_t);
    cudaFree(w->scales_c);
    cudaFree(w->sf_tiled);
    cudaFree(w->dinv);
    cudaFree(w->tensor_scale);
    cudaFree(w->tm_codes);
    free(w);
    return RUDDER_OK;
}

rudder_status rudder_weight_info(const rudder_weight* w, int* N, int* K, int* group, int* scheme, size_t* device_bytes)
{
    if (!w) return RUDDER_ERR_ARG;
    if (N) *N = w->N;
    if (K) *K = w->K;
    if (group) *group = w->G;
    if (scheme) *scheme = w->scheme;
    if (device_bytes) *device_bytes = w->bytes;
    return RUDDER_OK;
}

rudder_status rudder_weight_export(const rudder_weight* w, uint8_t* codes, void* scales, float* dinv, float* tensor_scale,
                                   void* stream)
{
    if (!w) return RUDDER_ERR_ARG;
    if (!on_weights_device(w)) return RUDDER_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t n_groups = static_cast<size_t>(w->K / w->G);
    if (w->scheme == RUDDER_W4A4_NVFP4) {
        if (codes && cudaMemcpyAsync(codes, w->codes, static_cast<size_t>(w->N) * (w->K / 2), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return RUDDER_ERR_CUDA;
        if (scales && cudaMemcpyAsync(scales, w->scales_c, n_groups * w->N, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return RUDDER_ERR_CUDA;
    } else {
        if (codes && launch_export_int4(w->codes, w->N, w->K, codes, w->f8 != 0, st) != cudaSuccess) return RUDDER_ERR_CUDA;
        if (scales && cudaMemcpyAsync(scales, w->scales_c, n_groups * w->N * sizeof(uint16_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return RUDDER_ERR_CUDA;
    }
    if (dinv && cudaMemcpyAsync(dinv, w->dinv, static_cast<size_t>(w->K) * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    if (tensor_scale && cudaMemcpyAsync(tensor_scale, w->tensor_scale, sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

size_t rudder_linear_workspace_bytes(const rudder_weight* w, int M) { return workspace_bytes_for(w, M); }

rudder_status rudder_linear(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M, const rudder_segments* seg,
                            int step, const rudder_scale_table* tab, const float* bias, uint16_t* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* stream)
{
    return linear_impl(w, X, ldx, M, seg, step, tab, bias, Y, ldy, workspace, workspace_bytes,
                       static_cast<cudaStream_t>(stream), nullptr, 0, 0, 0, 0);
}

rudder_status rudder_linear_dump_acc(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                     const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                     const float* bias, uint16_t* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                                     void* stream, int row0, int rows, int col0, int cols, int32_t* acc)
{
    if (!acc) return RUDDER_ERR_ARG;
    return linear_impl(w, X, ldx, M, seg, step, tab, bias, Y, ldy, workspace, workspace_bytes,
                       static_cast<cudaStream_t>(stream), acc, row0, rows, col0, cols);
}

size_t rudder_block_workspace_bytes(const rudder_block_args* args, int M)
{
    if (!args || M < 1) return 0;
    size_t total = 0;
    for (int l = 0; l < 4; ++l) {
        if (!args->w[l]) return 0;
        total += workspace_bytes_for(args->w[l], M);
    }
    if (args->x[3] == nullptr)       // chained: GELU(up output) is staged here as the down projection's input
        total += align_up(static_cast<size_t>(M) * args->w[3]->K * 2, 256);
    return total;
}

// The GELU in front of a chained layer moves into that layer's prologue when the range is static and the codes are integers.
static bool gelu_fuses(const rudder_weight* w, const rudder_scale_table* tab)
{
    return tab->mode == RUDDER_RANGE_STATIC && tab->clip != nullptr && w->scheme != RUDDER_W4A4_NVFP4;
}

// Workspace of rudder_block_dit: the four linears, the staged GELU output (M x F) and three M x H buffers
// (normalised input of the attention half, the first residual sum, normalised input of the MLP half).
static size_t dit_workspace_bytes(const rudder_block_args* args, int M)
{
    if (!args || M < 1) return 0;
    size_t total = 0;
    for (int l = 0; l < 4; ++l) {
        if (!args->w[l]) return 0;
        total += workspace_bytes_for(args->w[l], M);
    }
    total += align_up(static_cast<size_t>(M) * args->w[3]->K * 2, 256);
    total += 3 * align_up(static_cast<size_t>(M) * args->w[0]->K * 2, 256);
    return total;
}

static rudder_status block_dit_impl(const rudder_block_args* args, const rudder_block_glue* glue, int M, const rudder_segments* seg,
                                    int step, void* workspace, size_t workspace_bytes, cudaStream_t st)
{
    if (!args || !glue || !glue->norm1_weight || !glue->norm2_weight || !glue->out) return RUDDER_ERR_ARG;
    for (int l = 0; l < 4; ++l)
        if (!args->w[l] || !args->tab[l] || !args->y[l] || !on_weights_device(args->w[l])) return RUDDER_ERR_ARG;
    if (!args->x[0] || args->x[1] || args->x[2] || args->x[3]) return RUDDER_ERR_ARG;      // the block runs from x[0] alone
    const int H = args->w[0]->K, F = args->w[2]->N;
    if (args->w[0]->N != 3 * H || args->w[1]->K != H || args->w[1]->N != H || args->w[2]->K != H || args->w[3]->K != F || args->w[3]->N != H)
        return RUDDER_ERR_SHAPE;
    if (!(glue->eps >= 0.0f)) return RUDDER_ERR_ARG;
    const size_t need = dit_workspace_bytes(args, M);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need || need == 0) return RUDDER_ERR_WORKSPACE;
    if (!aligned(args->x[0], 16) || args->ldx[0] % 8 != 0 || args->ldx[0] < H || !aligned(glue->out, 16) || glue->ldout % 8 != 0 || glue->ldout < H ||
        !aligned(glue->norm1_weight, 16) || !aligned(glue->norm2_weight, 16))
        return RUDDER_ERR_ALIGN;
    for (int l = 0; l < 4; ++l) {
        SegParams sp;
        rudder_status s = check_table_and_segments(seg, step, args->tab[l], M, &sp);
        if (s != RUDDER_OK) return s;
        if (!aligned(args->y[l], 16) || args->ldy[l] % 8 != 0 || args->ldy[l] < args->w[l]->N) return RUDDER_ERR_ALIGN;
    }
    rudder_status s = ensure_init();
    if (s != RUDDER_OK) return s;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    size_t lin_off[4], off = 0;
    for (int l = 0; l < 4; ++l) { lin_off[l] = off; off += workspace_bytes_for(args->w[l], M); }
    uint16_t* gelu_buf = reinterpret_cast<uint16_t*>(ws + off); off += align_up(static_cast<size_t>(M) * F * 2, 256);
    uint16_t* n1 = reinterpret_cast<uint16_t*>(ws + off);       off += align_up(static_cast<size_t>(M) * H * 2, 256);
    uint16_t* h1 = reinterpret_cast<uint16_t*>(ws + off);       off += align_up(static_cast<size_t>(M) * H * 2, 256);
    uint16_t* n2 = reinterpret_cast<uint16_t*>(ws + off);
    const int sms = sm_count();
    auto lin = [&](int l, const uint16_t* x, int64_t ldx) {
        return linear_impl(args->w[l], x, ldx, M, seg, step, args->tab[l], args->bias[l], args->y[l], args->ldy[l], ws + lin_off[l],
                           workspace_bytes_for(args->w[l], M), st, nullptr, 0, 0, 0, 0, nullptr);
    };
    // attention half: h = x + O(V(QKV(norm1(x))))   (the V third of the QKV output stands in for attention, which stays outside)
    if (launch_rmsnorm(args->x[0], args->ldx[0], glue->norm1_weight, glue->eps, n1, H, M, H, st) != cudaSuccess) return RUDDER_ERR_CUDA;
    if ((s = lin(0, n1, H)) != RUDDER_OK) return s;
    if ((s = lin(1, args->y[0] + 2 * static_cast<size_t>(H), args->ldy[0])) != RUDDER_OK) return s;
    if (launch_add(args->x[0], args->ldx[0], args->y[1], args->ldy[1], h1, H, M, H, sms, st) != cudaSuccess) return RUDDER_ERR_CUDA;
    // MLP half: out = h + down(gelu(up(norm2(h))))
    if (launch_rmsnorm(h1, H, glue->norm2_weight, glue->eps, n2, H, M, H, st) != cudaSuccess) return RUDDER_ERR_CUDA;
    if ((s = lin(2, n2, H)) != RUDDER_OK) return s;
    if (gelu_fuses(args->w[3], args->tab[3])) {
        s = linear_impl(args->w[3], args->y[2], args->ldy[2], M, seg, step, args->tab[3], args->bias[3], args->y[3], args->ldy[3], ws + lin_off[3],
                        workspace_bytes_for(args->w[3], M), st, nullptr, 0, 0, 0, 0, nullptr, true);
        if (s != RUDDER_OK) return s;
    } else {
        if (launch_gelu(args->y[2], args->ldy[2], gelu_buf, F, M, F, sms, st) != cudaSuccess) return RUDDER_ERR_CUDA;
        if ((s = lin(3, gelu_buf, F)) != RUDDER_OK) return s;
    }
    if (launch_add(h1, H, args->y[3], args->ldy[3], glue->out, glue->ldout, M, H, sms, st) != cudaSuccess) return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

static rudder_status block_impl(const rudder_block_args* args, int M, const rudder_segments* seg, int step, void* workspace,
                                size_t workspace_bytes, void* stream, cudaEvent_t* ev /* [9] or nullptr */)
{
    if (!args) return RUDDER_ERR_ARG;
    for (int l = 0; l < 4; ++l)
        if (!args->w[l] || !args->tab[l] || (!args->x[l] && l == 0) || !args->y[l] || !on_weights_device(args->w[l])) return RUDDER_ERR_ARG;
    const size_t need = rudder_block_workspace_bytes(args, M);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need || need == 0) return RUDDER_ERR_WORKSPACE;
    // Chained layers (x[l] == NULL, l >= 1) take the previous output through the minimal glue: the V third
    // of the QKV output stands in for attention, the O output feeds the up projection as it is, GELU of the
    // up output (staged at the end of the workspace) feeds the down projection.
    const uint16_t* x_eff[4];
    int64_t ldx_eff[4];
    size_t lin_bytes = 0;
    for (int l = 0; l < 4; ++l) lin_bytes += workspace_bytes_for(args->w[l], M);
    uint16_t* gelu_buf = reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(workspace) + lin_bytes);
    for (int l = 0; l < 4; ++l) {
        x_eff[l] = args->x[l];
        ldx_eff[l] = args->ldx[l];
        if (args->x[l] != nullptr) continue;
        const int K = args->w[l]->K, Np = args->w[l - 1]->N;
        if (l == 1) {
            if (Np != 3 * K) return RUDDER_ERR_SHAPE;
            x_eff[l] = args->y[0] + 2 * static_cast<size_t>(K);
            ldx_eff[l] = args->ldy[0];
        } else {
            if (Np != K) return RUDDER_ERR_SHAPE;
            x_eff[l] = (l == 3) ? gelu_buf : args->y[l - 1];
            ldx_eff[l] = (l == 3) ? K : args->ldy[l - 1];
        }
    }
    // validate everything before the first launch
    for (int l = 0; l < 4; ++l) {
        SegParams sp;
        rudder_status s = check_table_and_segments(seg, step, args->tab[l], M, &sp);
        if (s != RUDDER_OK) return s;
        const rudder_weight* w = args->w[l];
        if (!aligned(x_eff[l], 16) || !aligned(args->y[l], 16) || ldx_eff[l] % 8 != 0 || args->ldy[l] % 8 != 0 ||
            ldx_eff[l] < w->K || args->ldy[l] < w->N)
            return RUDDER_ERR_ALIGN;
    }
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    for (int l = 0; l < 4; ++l) {
        const size_t bytes = workspace_bytes_for(args->w[l], M);
        // Chained down projection.  With a static range (the paper's calibrated threshold) its prologue has no row
        // reduction, so the GELU is applied inside it, straight from the up output: no activated tensor is written
        // or read back and the GELU launch goes away.  Otherwise GELU runs as a pass of its own into the staging buffer.
        const bool fuse_gelu = l == 3 && args->x[3] == nullptr && gelu_fuses(args->w[3], args->tab[3]);
        if (l == 3 && args->x[3] == nullptr && !fuse_gelu &&
            launch_gelu(args->y[2], args->ldy[2], gelu_buf, args->w[3]->K, M, args->w[3]->K, sm_count(), static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return RUDDER_ERR_CUDA;
        rudder_status s = linear_impl(args->w[l], fuse_gelu ? args->y[2] : x_eff[l], fuse_gelu ? args->ldy[2] : ldx_eff[l], M, seg, step,
                                      args->tab[l], args->bias[l], args->y[l], args->ldy[l], ws, bytes, static_cast<cudaStream_t>(stream),
                                      nullptr, 0, 0, 0, 0, ev ? ev + 2 * l : nullptr, fuse_gelu);
        if (s != RUDDER_OK) return s;
        ws += bytes;
    }
    return RUDDER_OK;
}

rudder_status rudder_block(const rudder_block_args* args, int M, const rudder_segments* seg, int step, void* workspace,
                           size_t workspace_bytes, void* stream)
{
    return block_impl(args, M, seg, step, workspace, workspace_bytes, stream, nullptr);
}

size_t rudder_block_dit_workspace_bytes(const rudder_block_args* args, int M) { return dit_workspace_bytes(args, M); }

rudder_status rudder_block_dit(const rudder_block_args* args, const rudder_block_glue* glue, int M, const rudder_segments* seg, int step,
                               void* workspace, size_t workspace_bytes, void* stream)
{
    return block_dit_impl(args, glue, M, seg, step, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

rudder_status rudder_block_profile(const rudder_block_args* args, int M, const rudder_segments* seg, int step,
                                   void* workspace, size_t workspace_bytes, void* stream, float* ms)
{
    if (!ms) return RUDDER_ERR_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaEvent_t ev[9];
    for (int i = 0; i < 9; ++i)
        if (cudaEventCreate(&ev[i]) != cudaSuccess) return RUDDER_ERR_CUDA;
    rudder_status s = RUDDER_OK;
    if (cudaEventRecord(ev[0], st) != cudaSuccess) s = RUDDER_ERR_CUDA;
    if (s == RUDDER_OK) s = block_impl(args, M, seg, step, workspace, workspace_bytes, stream, ev);
    if (s == RUDDER_OK && cudaStreamSynchronize(st) != cudaSuccess) s = RUDDER_ERR_CUDA;
    if (s == RUDDER_OK)
        for (int i = 0; i < 8; ++i)
            if (cudaEventElapsedTime(&ms[i], ev[i], ev[i + 1]) != cudaSuccess) s = RUDDER_ERR_CUDA;
    for (int i = 0; i < 9; ++i) cudaEventDestroy(ev[i]);
    return s;
}

// Copy streams and events of rudder_block_host, one set per device, created on first use.  Calls on one
// device share them: concurrent host threads must not call rudder_block_host on the same device.
struct HostPipe {
    cudaStream_t in, out;
    cudaEvent_t start, in_done[4], lin_done[4], out_done;
    bool ready;
};
static HostPipe g_host_pipe[64];

static HostPipe* host_pipe()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe* hp = &g_host_pipe[dev];
    std::lock_guard<std::mutex> lock(g_state_mutex);
    if (!hp->ready) {
        if (cudaStreamCreateWithFlags(&hp->in, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&hp->out, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&hp->start, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&hp->out_done, cudaEventDisableTiming) != cudaSuccess)
            return nullptr;
        for (int l = 0; l < 4; ++l)
            if (cudaEventCreateWithFlags(&hp->in_done[l], cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&hp->lin_done[l], cudaEventDisableTiming) != cudaSuccess)
                return nullptr;
        hp->ready = true;
    }
    return hp;
}

size_t rudder_block_host_staging_bytes(const rudder_block_args* args, int M)
{
    if (!args || M < 1) return 0;
    size_t total = 0;
    for (int l = 0; l < 4; ++l) {
        if (!args->w[l]) return 0;
        total += align_up(static_cast<size_t>(M) * args->w[l]->K * 2, 256) + align_up(static_cast<size_t>(M) * args->w[l]->N * 2, 256);
    }
    return total;
}

rudder_status rudder_block_host(const rudder_block_args* args, int M, const rudder_segments* seg, int step, void* staging,
                                size_t staging_bytes, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!args) return RUDDER_ERR_ARG;
    for (int l = 0; l < 4; ++l)
        if (!args->w[l] || !args->x[l] || !args->y[l] || args->ldx[l] < args->w[l]->K || args->ldy[l] < args->w[l]->N)
            return RUDDER_ERR_ARG;
    const size_t need = rudder_block_host_staging_bytes(args, M);
    if (!staging || !aligned(staging, 256) || staging_bytes < need || need == 0) return RUDDER_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rudder_block_args dev = *args;
    uint8_t* p = static_cast<uint8_t*>(staging);
    for (int l = 0; l < 4; ++l) {
        const int K = args->w[l]->K, N = args->w[l]->N;
        dev.x[l] = reinterpret_cast<const uint16_t*>(p);
        dev.ldx[l] = K;
        p += align_up(static_cast<size_t>(M) * K * 2, 256);
        dev.y[l] = reinterpret_cast<uint16_t*>(p);
        dev.ldy[l] = N;
        p += align_up(static_cast<size_t>(M) * N * 2, 256);
    }
    // validate on the host before the first copy is enqueued (block_impl checks again)
    for (int l = 0; l < 4; ++l) {
        SegParams sp;
        if (!args->tab[l]) return RUDDER_ERR_ARG;
        rudder_status s = check_table_and_segments(seg, step, args->tab[l], M, &sp);
        if (s != RUDDER_OK) return s;
    }
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < rudder_block_workspace_bytes(args, M)) return RUDDER_ERR_WORKSPACE;
    // Uploads, the four linears and downloads run on three streams (PCIe is full duplex): linear l starts
    // when its input has landed, its output goes back while later inputs are still coming in.  `st` waits
    // for the last download, so the call keeps the usual stream semantics.
    HostPipe* hp = host_pipe();
    if (!hp) return RUDDER_ERR_CUDA;
    if (cudaEventRecord(hp->start, st) != cudaSuccess || cudaStreamWaitEvent(hp->in, hp->start, 0) != cudaSuccess ||
        cudaStreamWaitEvent(hp->out, hp->start, 0) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    for (int l = 0; l < 4; ++l) {
        const int K = args->w[l]->K;
        if (cudaMemcpy2DAsync(const_cast<uint16_t*>(dev.x[l]), static_cast<size_t>(K) * 2, args->x[l], static_cast<size_t>(args->ldx[l]) * 2,
                              static_cast<size_t>(K) * 2, M, cudaMemcpyHostToDevice, hp->in) != cudaSuccess ||
            cudaEventRecord(hp->in_done[l], hp->in) != cudaSuccess)
            return RUDDER_ERR_CUDA;
    }
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    for (int l = 0; l < 4; ++l) {
        const int N = args->w[l]->N;
        const size_t bytes = workspace_bytes_for(args->w[l], M);
        if (cudaStreamWaitEvent(st, hp->in_done[l], 0) != cudaSuccess) return RUDDER_ERR_CUDA;
        rudder_status s = linear_impl(dev.w[l], dev.x[l], dev.ldx[l], M, seg, step, dev.tab[l], dev.bias[l], dev.y[l], dev.ldy[l],
                                      ws, bytes, st, nullptr, 0, 0, 0, 0, nullptr);
        if (s != RUDDER_OK) return s;
        ws += bytes;
        if (cudaEventRecord(hp->lin_done[l], st) != cudaSuccess || cudaStreamWaitEvent(hp->out, hp->lin_done[l], 0) != cudaSuccess ||
            cudaMemcpy2DAsync(args->y[l], static_cast<size_t>(args->ldy[l]) * 2, dev.y[l], static_cast<size_t>(N) * 2,
                              static_cast<size_t>(N) * 2, M, cudaMemcpyDeviceToHost, hp->out) != cudaSuccess)
            return RUDDER_ERR_CUDA;
    }
    if (cudaEventRecord(hp->out_done, hp->out) != cudaSuccess || cudaStreamWaitEvent(st, hp->out_done, 0) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

rudder_status rudder_quantize_activations(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M,
                                          const rudder_segments* seg, int step, const rudder_scale_table* tab,
                                          void* codes, uint8_t* block_scales, float* row_scale, void* stream)
{
    if (!w || !X || !codes || !row_scale) return RUDDER_ERR_ARG;
    if (w->scheme == RUDDER_W4A4_NVFP4 && !block_scales) return RUDDER_ERR_ARG;
    if (!on_weights_device(w)) return RUDDER_ERR_ARG;
    if (M < 1) return RUDDER_ERR_SHAPE;
    SegParams sp;
    rudder_status s = check_table_and_segments(seg, step, tab, M, &sp);
    if (s != RUDDER_OK) return s;
    if (!aligned(X, 16) || ldx % 8 != 0 || ldx < w->K || !aligned(codes, 16)) return RUDDER_ERR_ALIGN;
    ActqArgs a;
    a.zero_ints = nullptr; a.n_zero = 0;
    a.X = X; a.ldx = ldx; a.M = M; a.K = w->K; a.dinv = w->dinv;
    a.gamma_step = tab->gamma + static_cast<size_t>(step) * tab->S;
    a.clip_step = (tab->mode == RUDDER_RANGE_STATIC) ? tab->clip + step : nullptr;
    a.seg = sp;
    if (w->scheme == RUDDER_W4A4_NVFP4) {
        // same kernel as production; the block scales go out row-major instead of in the tiled order
        if (launch_actq_nvfp4(a, static_cast<uint8_t*>(codes), block_scales, false, row_scale, static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return RUDDER_ERR_CUDA;
        return RUDDER_OK;
    }
    // The kernel writes what production writes for this weight: int8, or (W4A4 on the E4M3 tensor path) the
    // E4M3 bytes of the same integers, which are then decoded in place so that the caller sees integers.
    const bool e4m3 = w->f8 != 0 && !gemm_i8_register_path(M, w->N, w->K, w->G, w->f8 != 0);     // the register-level GEMMs read int8 whatever the weight layout
    if (launch_actq_int(a, qmax_of(w->scheme), e4m3, static_cast<int8_t*>(codes), w->K, row_scale, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    if (e4m3 && launch_e4m3_to_int8(static_cast<int8_t*>(codes), static_cast<size_t>(M) * w->K, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

rudder_status rudder_gelu_quantize_activations(const rudder_weight* w, const uint16_t* X, int64_t ldx, int M, const rudder_segments* seg,
                                               int step, const rudder_scale_table* tab, void* codes, float* row_scale, void* stream)
{
    if (!w || !X || !codes || !row_scale) return RUDDER_ERR_ARG;
    if (!on_weights_device(w)) return RUDDER_ERR_ARG;
    if (M < 1) return RUDDER_ERR_SHAPE;
    SegParams sp;
    rudder_status s = check_table_and_segments(seg, step, tab, M, &sp);
    if (s != RUDDER_OK) return s;
    if (!gelu_fuses(w, tab)) return RUDDER_ERR_UNSUPPORTED;
    if (!aligned(X, 16) || ldx % 8 != 0 || ldx < w->K || !aligned(codes, 16)) return RUDDER_ERR_ALIGN;
    ActqArgs a;
    a.zero_ints = nullptr; a.n_zero = 0;
    a.X = X; a.ldx = ldx; a.M = M; a.K = w->K; a.dinv = w->dinv;
    a.gamma_step = tab->gamma + static_cast<size_t>(step) * tab->S;
    a.clip_step = tab->clip + step;
    a.seg = sp;
    const bool e4m3 = w->f8 != 0 && !gemm_i8_register_path(M, w->N, w->K, w->G, w->f8 != 0);     // what production writes for this weight and shape
    if (launch_actq_gelu_static(a, qmax_of(w->scheme), e4m3, static_cast<int8_t*>(codes), w->K, row_scale, sm_count(), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    if (e4m3 && launch_e4m3_to_int8(static_cast<int8_t*>(codes), static_cast<size_t>(M) * w->K, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return RUDDER_ERR_CUDA;
    return RUDDER_OK;
}

rudder_status rudder_gelu(const uint16_t* X, int64_t ldx, int M, int N, uint16_t* Y, int64_t ldy, void* stream)
{
    if (!X || !Y) return RUDDER_ERR_ARG;
    if (M < 1 || N < 8 || N % 8 != 0) return RUDDER_ERR_SHAPE;
    if (!aligned(X, 16) || !aligned(Y, 16) || ldx % 8 != 0 || ldy % 8 != 0 || ldx < N || ldy < N) return RUDDER_ERR_ALIGN;
    rudder_status s = ensure_init();
    if (s != RUDDER_OK) return s;
    return launch_gelu(X, ldx, Y, ldy, M, N, sm_count(), static_cast<cudaStream_t>(stream)) == cudaSuccess ? RUDDER_OK : RUDDER_ERR_CUDA;
}

rudder_status rudder_rmsnorm(const uint16_t* X, int64_t ldx, int M, int N, const float* weight, float eps, uint16_t* Y, int64_t ldy, void* stream)
{
    if (!X || !Y || !weight || !(eps >= 0.0f)) return RUDDER_ERR_ARG;
    if (M < 1 || N < 8 || N % 8 != 0) return RUDDER_ERR_SHAPE;
    if (!aligned(X, 16) || !aligned(Y, 16) || !aligned(weight, 16) || ldx % 8 != 0 || ldy % 8 != 0 || ldx < N || ldy < N) return RUDDER_ERR_ALIGN;
    return launch_rmsnorm(X, ldx, weight, eps, Y, ldy, M, N, static_cast<cudaStream_t>(stream)) == cudaSuccess ? RUDDER_OK : RUDDER_ERR_CUDA;
}

rudder_status rudder_add(const uint16_t* A, int64_t lda, const uint16_t* B, int64_t ldb, int M, int N, uint16_t* Y, int64_t ldy, void* stream)
{
    if (!A || !B || !Y) return RUDDER_ERR_ARG;
    if (M < 1 || N < 8 || N % 8 != 0) return RUDDER_ERR_SHAPE;
    if (!aligned(A, 16) || !aligned(B, 16) || !aligned(Y, 16) || lda % 8 != 0 || ldb % 8 != 0 || ldy % 8 != 0 || lda < N || ldb < N || ldy < N)
        return RUDDER_ERR_ALIGN;
    return launch_add(A, lda, B, ldb, Y, ldy, M, N, sm_count(), static_cast<cudaStream_t>(stream)) == cudaSuccess ? RUDDER_OK : RUDDER_ERR_CUDA;
}

rudder_status rudder_selftest_wait_timeout(long long limit_cycles, void* stream)
{
    if (limit_cycles < 1000 || limit_cycles > 100000000ll) return RUDDER_ERR_ARG;     // at most ~50 ms of SM clocks
    return launch_wait_timeout_selftest(limit_cycles, static_cast<cudaStream_t>(stream)) == cudaSuccess ? RUDDER_OK : RUDDER_ERR_CUDA;
}

rudder_status rudder_device_status(int* last, int* where)
{
    if (!last) return RUDDER_ERR_ARG;
    int v[2] = {0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) return RUDDER_ERR_CUDA;
    if (cudaMemcpyFromSymbol(v, rudder::g_device_status, sizeof(v)) != cudaSuccess) return RUDDER_ERR_CUDA;
    const int zero[2] = {0, 0};
    if (cudaMemcpyToSymbol(rudder::g_device_status, zero, sizeof(zero)) != cudaSuccess) return RUDDER_ERR_CUDA;
    *last = v[0];
    if (where) *where = v[1];
    return RUDDER_OK;
}

}  // extern "C"
