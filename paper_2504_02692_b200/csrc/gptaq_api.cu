// C ABI of the GPTAQ layer solve: handle, argument checks, launch sequences.
// Every arithmetic step runs in the kernels of this library; the host code
// below only validates, carves the caller's workspace and enqueues launches.
#include "../../include/gptaq.h"

#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "kernels.cuh"
#include "simt_gemm.cuh"
#include "umma_gemm.cuh"
#include "tc_gemm.cuh"

using namespace gptaq;

namespace {

constexpr size_t ALIGN = 256;
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

enum Stage { STAGE_ACCUM = 0, STAGE_FACTORED = 1, STAGE_P = 2 };
constexpr int64_t ACT_ORDER_MAX_N = 57344;     // a weight row (float32) has to fit the shared memory of one CTA
constexpr int64_t P_ROWWISE_MAX_N = 16384;     // two rows (float32) in the shared memory of one CTA

}  // namespace

struct gptaq_ctx {
    int64_t n;
    int device;
    int num_sms;
    char *state;
    size_t state_bytes;
    char *ws;
    size_t ws_bytes;
    StateHeader *hd;
    float *H, *D;
    uint8_t *dead;         // dead-input flags in working (possibly sorted) column order
    uint8_t *dead_raw;     // ... in the caller's column order
    int *perm;             // act_order: working column c is the caller's column perm[c]
    bool act_order;
    int stage;
    int64_t tokens;
    int64_t launches;
    int stats_precision;   // GPTAQ_STATS_*
    bool tensor;           // float32-grade tensor-core GEMMs for factor / P / trailing update
    bool f16;              // ... with FP16-split operands where the producer can record their range (n % 8 == 0)
    TcSched sched;         // tile numbering of the float32-grade GEMM launches (see StateHeader::sched_counter)
    int terms;             // GPTAQ_TERM_* switches of gptaq_quantize
    bool static_groups;    // group grids from the original weights, per group of the caller's columns
    int clip_steps; float clip_min;   // clipping-range search of the grids
    // Statistics pipeline: the conversion of a token batch runs on the caller's stream, the
    // tensor-core product on `gemm_stream`, so that the (memory-bound) conversion of the next
    // batch overlaps the (tensor-bound) product of this one.  Two operand buffers alternate.
    cudaStream_t gemm_stream;
    cudaEvent_t conv_done[2], gemm_done[2];
    bool gemm_pending[2];
    bool relayout;         // the operand buffers change size: wait for the products in flight first
    int next_buf;
    // partial sums of the cut tiles of the statistics products wait in the workspace (fix_args.scratch) until
    // the sums are needed or the cut changes; fix_pending: they have not been added to H / dXX^T yet
    bool fix_pending;
    StatsGemmArgs fix_args;
    bool d_upper_only;     // a token batch went in without the tiles of dXX^T below the diagonal
    // optional timing of the statistics kernel alone: one event pair per launch, on the stream it runs on
    bool kernel_timing;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timing_events;   // pool; the first timing_used are recorded
    size_t timing_used;
    std::string cuda_error;
};

namespace {

struct Layout {
    size_t h_off, d_off, dead_off, dead_raw_off, perm_off, total;
};

Layout state_layout(int64_t n) {
    Layout l;
    size_t mat = round_up((size_t)n * (size_t)n * sizeof(float), ALIGN);
    l.h_off = ALIGN;
    l.d_off = l.h_off + mat;
    l.dead_off = l.d_off + mat;
    l.dead_raw_off = l.dead_off + round_up((size_t)n, ALIGN);
    l.perm_off = l.dead_raw_off + round_up((size_t)n, ALIGN);
    l.total = l.perm_off + round_up((size_t)n * sizeof(int), ALIGN);
    return l;
}

// float32-grade tensor-core path (tc_gemm.cuh): widths whose rows are 16-byte multiples (a TMA
// stride rule) and that are large enough for 128 x 256 tiles to pay.
constexpr int64_t TC_MIN_N = 512;
inline bool tc_shape_ok(int64_t n) { return n >= TC_MIN_N && (n % 4) == 0; }

struct WsLayout {
    size_t t_off, rinv_off;
    size_t s_off[6];        // split operand matrices (n x n each): S1 hi/lo, S2 hi/lo, S3 hi/lo
    size_t pan_off[2];      // split copy of factor panels, hi/lo: n x 128 float32 (TF32) or n x SUPER_NB fp16
    // [-Err | Wpre]: float32 (m x 2B, or m x 2 * QSUPER * B for the FP16-split update), second part
    // (TF32 remainder, or the fp16 hi / lo parts of the wide matrix), fp16 hi / lo of one block, row scales
    size_t ew_off, ew_lo_off, ew16_off, rs_off, total;
    bool tensor;
};

// FP16-split factorisation: panels are grouped in super-panels of SUPER_NB columns; inside a super-panel
// the rank-128 update only touches the super-panel's remaining columns, the rest of the matrix receives
// one rank-SUPER_NB update per super-panel (8x less read-modify-write traffic, longer contractions)
constexpr int SUPER_NB = 8 * NB;
// The lazy-batch update of gptaq_quantize likewise: QSUPER blocks form a super-block; a block's errors
// are applied to the rest of its super-block at once and to everything beyond once per super-block.
constexpr int QSUPER = 8;

WsLayout ws_layout(int64_t n, int64_t m_max, int blocksize) {
    WsLayout w;
    size_t nb = (size_t)((n + NB - 1) / NB);
    const size_t mat = round_up((size_t)n * (size_t)n * sizeof(float), ALIGN);
    w.tensor = tc_shape_ok(n);
    w.t_off = 0;
    w.rinv_off = w.t_off + mat;
    size_t off = w.rinv_off + round_up(nb * NB * NB * sizeof(float), ALIGN);
    const bool f16 = w.tensor && (n % 8) == 0;
    // split operand copies: six float32-sized regions for TF32 parts; fp16 hi / lo parts use three
    // (S0 = U^T, S1 = U then P^T, S4 = dXX^T then O; hi and lo of one matrix fill one region)
    for (int i = 0; i < 6; ++i) {
        w.s_off[i] = off;
        if (w.tensor && (!f16 || i == 0 || i == 1 || i == 4)) off += mat;
    }
    const size_t pan = std::max((size_t)n * NB * sizeof(float), (size_t)n * SUPER_NB * sizeof(__half));
    for (int i = 0; i < 2; ++i) { w.pan_off[i] = off; if (w.tensor) off += round_up(pan, ALIGN); }
    const size_t ew1 = round_up((size_t)m_max * 2 * (size_t)blocksize * sizeof(float), ALIGN);
    const size_t ew = f16 ? QSUPER * ew1 : ew1;
    w.ew_off = off;
    w.ew_lo_off = off + ew;
    w.ew16_off = off + (w.tensor ? 2 * ew : ew);
    w.rs_off = w.ew16_off + (f16 ? ew1 : 0);
    w.total = w.rs_off + (f16 ? round_up(2 * (size_t)m_max * sizeof(float), ALIGN) : 0);
    return w;
}

gptaq_status_t cuda_fail(gptaq_ctx *h, cudaError_t e) {
    if (h) h->cuda_error = cudaGetErrorString(e);
    return GPTAQ_ERR_CUDA;
}

#define CU(call)                                             \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) return cuda_fail(h, e__);    \
    } while (0)

#define LAUNCHED()                                           \
    do {                                                     \
        cudaError_t e__ = cudaGetLastError();                \
        if (e__ != cudaSuccess) return cuda_fail(h, e__);    \
        h->launches++;                                       \
    } while (0)

gptaq_status_t gemm(gptaq_ctx *h, const GemmProblem &p, bool a_rc, bool b_rc, cudaStream_t s) {
    if (p.M <= 0 || p.N <= 0 || p.nbatch <= 0) return GPTAQ_OK;
    cudaError_t e = launch_simt_gemm(p, a_rc, b_rc, s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches++;
    return GPTAQ_OK;
}

#define OK(call)                                  \
    do {                                          \
        gptaq_status_t s__ = (call);              \
        if (s__ != GPTAQ_OK) return s__;          \
    } while (0)

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// fp16 matrix [rows][kp] (K contiguous), box = 64 x box_rows, 128-byte swizzle.
bool make_kmajor_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t kp, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kp, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kp * 2};
    cuuint32_t box[2] = {(cuuint32_t)UBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// float32 matrix [rows][ld] with `cols` valid K-contiguous elements per row; box = 32 x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_f32_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {(cuuint32_t)TBK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A split operand (hi / lo arrays of the same shape) as seen by the tensor-core GEMM.
struct SplitOperand {
    const void *hi, *lo;       // float32 arrays holding TF32 values, or __half arrays (f16)
    int64_t rows, cols, ld;
    bool f16 = false;
};

// __half matrix [rows][ld] with `cols` valid K-contiguous elements per row; box = 64 x box_rows.
bool make_f16_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)(2 * TBK), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_operand_map(CUtensorMap *map, const void *ptr, const SplitOperand &o, int box_rows) {
    return o.f16 ? make_f16_map(map, ptr, o.rows, o.cols, o.ld, box_rows)
                 : make_f32_map(map, ptr, o.rows, o.cols, o.ld, box_rows);
}

struct TcMaps {
    CUtensorMap a_hi, a_lo, b_hi, b_lo, b2_hi, b2_lo;
    bool f16 = false;
};

bool make_tc_maps(TcMaps *m, const SplitOperand &A, const SplitOperand &B, const SplitOperand *B2) {
    const SplitOperand &b2 = B2 ? *B2 : B;
    m->f16 = A.f16;
    return make_operand_map(&m->a_hi, A.hi, A, TBM) && make_operand_map(&m->a_lo, A.lo, A, TBM) &&
           make_operand_map(&m->b_hi, B.hi, B, TBN) && make_operand_map(&m->b_lo, B.lo, B, TBN) &&
           make_operand_map(&m->b2_hi, b2.hi, b2, TBN) && make_operand_map(&m->b2_lo, b2.lo, b2, TBN);
}

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor
// drains; it calls pdl_wait() before it touches anything the predecessor wrote.
// (Measured on a 4096-wide layer: the factorisation's chain of short launches gains 4 %, the quantize
// chain loses 4 %, so only the former uses it.)
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

TcGemmArgs tc_args(float *C, int64_t ldc, int M, int N, int K, float alpha, float beta, int mode, int mask,
                   StateHeader *hd) {
    TcGemmArgs a;
    std::memset(&a, 0, sizeof(a));
    a.C = C; a.ldc = ldc; a.M = M; a.N = N; a.K = K; a.nbatch = 1;
    a.alpha = alpha; a.beta = beta; a.mode = mode; a.mask = mask; a.hd = hd;
    return a;
}

// float32 matrix C [M][ldc] with N valid columns as the target of bulk reductions: box = 32 x 128,
// 128-byte swizzle (the layout the epilogue writes its staging boxes in).
bool make_c_map(CUtensorMap *map, float *C, int64_t M, int64_t N, int64_t ldc) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
    cuuint32_t box[2] = {32, (cuuint32_t)TBM};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t launch_tc_gemm(const TcMaps &m, const TcGemmArgs &a_in, TcSched &sched, int num_sms, cudaStream_t s, bool pdl = true) {
    if (a_in.M <= 0 || a_in.N <= 0 || a_in.nbatch <= 0) return cudaSuccess;
    TcGemmArgs a = a_in;
    const int64_t tiles = (int64_t)a.nbatch * ((a.M + TBM - 1) / TBM) * ((a.N + TBN - 1) / TBN);
    const int grid = (int)std::min<int64_t>(tiles, num_sms);
    // "C += ...": bulk tensor reductions where the target qualifies for a tensor map (16-byte aligned base
    // and row pitch); scattered per-thread reductions otherwise
    a.sched = &a.hd->sched_counter;
    a.sched_base = sched.base;
    sched.base += (unsigned)tiles;           // (grid <= tiles)
    CUtensorMap mapC = m.a_hi;       // placeholder, not dereferenced unless c_tma is set
    a.c_tma = 0;
    if (a.beta == 1.f && a.nbatch == 1 && !a.amax_out && (a.mask == TC_MASK_NONE || a.mask == TC_MASK_UPPER_KEEP) &&
        (reinterpret_cast<uintptr_t>(a.C) & 15) == 0 && (a.ldc & 3) == 0 && make_c_map(&mapC, a.C, a.M, a.N, a.ldc))
        a.c_tma = 1;
    if (m.f16) return launch_pdl(pdl, tc_gemm_kernel<true>, dim3(grid), dim3(TC_THREADS), TC_SMEM, s, m.a_hi, m.a_lo, m.b_hi, m.b_lo, m.b2_hi, m.b2_lo, mapC, a);
    return launch_pdl(pdl, tc_gemm_kernel<false>, dim3(grid), dim3(TC_THREADS), TC_SMEM, s, m.a_hi, m.a_lo, m.b_hi, m.b_lo, m.b2_hi, m.b2_lo, mapC, a);
}

// Slots of StateHeader::tc_amax (largest magnitudes of FP16-split operands).

cudaError_t launch_absmax(const float *src, int64_t lds, int rows, int cols, int mask, float scale, unsigned *slot,
                          int num_sms, cudaStream_t s) {
    const int grid = std::max(1, std::min(rows, 8 * num_sms));
    absmax_kernel<<<grid, 256, 0, s>>>(src, lds, rows, cols, mask, scale, slot);
    return cudaGetLastError();
}

struct SplitBatch {
    int nbatch = 1;
    int64_t src_bstride = 0, dst_bstride = 0;
    int rows_last = 0, cols_last = 0;
};

// hi_t / lo_t non-null: the transposed form goes there in the same pass (transpose is then ignored)
cudaError_t launch_split16(const float *src, int64_t lds, __half *hi, __half *lo, int64_t ldd, int rows, int cols,
                           bool transpose, int mask, float scale, const unsigned *amax, cudaStream_t s,
                           const SplitBatch &b = SplitBatch(), __half *hi_t = nullptr, __half *lo_t = nullptr) {
    if (rows <= 0 || cols <= 0 || b.nbatch <= 0) return cudaSuccess;
    Split16Args a;
    a.src = src; a.lds = lds; a.src_bstride = b.src_bstride; a.hi = hi; a.lo = lo; a.ldd = ldd;
    a.dst_bstride = b.dst_bstride;
    a.rows = rows; a.cols = cols; a.rows_last = b.rows_last; a.cols_last = b.cols_last; a.nbatch = b.nbatch;
    a.transpose = hi_t ? 2 : (transpose ? 1 : 0); a.mask = mask; a.scale = scale; a.amax = amax;
    a.hi_t = hi_t; a.lo_t = lo_t;
    dim3 grid((cols + 63) / 64, (rows + 63) / 64, b.nbatch);
    split16_kernel<<<grid, 256, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_split(const float *src, int64_t lds, float *hi, float *lo, int64_t ldd, int rows, int cols,
                         bool transpose, int mask, float scale, cudaStream_t s, const SplitBatch &b = SplitBatch()) {
    if (rows <= 0 || cols <= 0 || b.nbatch <= 0) return cudaSuccess;
    SplitArgs a;
    a.src = src; a.lds = lds; a.src_bstride = b.src_bstride; a.hi = hi; a.lo = lo; a.ldd = ldd;
    a.dst_bstride = b.dst_bstride;
    a.rows = rows; a.cols = cols; a.rows_last = b.rows_last; a.cols_last = b.cols_last; a.nbatch = b.nbatch;
    a.transpose = transpose ? 1 : 0; a.mask = mask; a.scale = scale;
    dim3 grid((cols + 63) / 64, (rows + 63) / 64, b.nbatch);
    split_kernel<<<grid, 256, 0, s>>>(a);
    return cudaGetLastError();
}

// Scratch of the statistics kernel's K-split tail: at most one 128 x 256 partial tile per SM.
size_t stats_scratch_bytes(int num_sms) { return round_up((size_t)num_sms * UBM * UBN * sizeof(float), ALIGN); }
constexpr int MAX_SMS_FOR_SIZING = 256;

// fp16 operand arrays per converted batch: X^T, (X~ - X)^T, the low part of X^T, the low part of (X~ - X)^T
int stats_operand_arrays(int precision) {
    return precision == GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR ? 4 : (precision == GPTAQ_STATS_FP16_SPLIT_TENSOR ? 3 : 2);
}

// Largest token chunk (multiple of 64) whose fp16 operand copies fit the workspace next to that scratch.
int64_t tc_chunk_tokens(const gptaq_ctx *h) {
    const int nbuf = stats_operand_arrays(h->stats_precision);
    int64_t per_token = 2 * nbuf * h->n * 2;   // two buffers of X^T, dX^T (and their low parts), fp16
    const size_t reserve = stats_scratch_bytes(h->num_sms);
    if (h->ws_bytes <= reserve + 2 * ALIGN) return 0;
    int64_t cap = (int64_t)((h->ws_bytes - reserve - 2 * ALIGN) / (size_t)per_token);
    cap = cap / UBK * UBK;
    return std::min<int64_t>(cap, 1 << 20);
}

bool tc_eligible(const gptaq_ctx *h) {
    // from 256 input channels on, and for exactly 128 (one half-empty pair tile per sum; the TMA boxes of 128
    // channels then cover the operand exactly)
    return h->stats_precision != GPTAQ_STATS_FP32 && (h->n >= UBN || h->n == UBM) && tc_chunk_tokens(h) >= UBK &&
           encode_tiled_fn() != nullptr;
}

// Adds the waiting partial sums of the cut tiles to H / dXX^T, on the internal stream behind the products.
gptaq_status_t flush_partials(gptaq_ctx *h) {
    if (!h->fix_pending) return GPTAQ_OK;
    const StatsGemmArgs &ga = h->fix_args;
    stats_fixup_kernel<<<dim3((unsigned)(ga.ntiles - ga.full_tiles), FIXUP_SLABS), 256, 0, h->gemm_stream>>>(ga);
    LAUNCHED();
    h->fix_pending = false;
    CU(cudaEventRecord(h->gemm_done[0], h->gemm_stream));
    h->gemm_pending[0] = true;
    return GPTAQ_OK;
}

// Orders `s` after every statistics product still running on the internal stream.
gptaq_status_t join_statistics(gptaq_ctx *h, cudaStream_t s) {
    OK(flush_partials(h));
    for (int i = 0; i < 2; ++i)
        if (h->gemm_pending[i]) {
            CU(cudaStreamWaitEvent(s, h->gemm_done[i], 0));
            h->gemm_pending[i] = false;
        }
    return GPTAQ_OK;
}

gptaq_status_t accumulate_tc(gptaq_ctx *h, const float *X, const float *Xfp, int64_t tokens, int64_t ld,
                             cudaStream_t s) {
    const int n = (int)h->n;
    if (h->relayout) {
        OK(join_statistics(h, s));
        h->relayout = false;
    }
    const int64_t chunk = tc_chunk_tokens(h);
    // 256 x 256 tiles of H (upper) and of dXX^T (upper too, unless act_order will permute it)
    const int d_full = h->act_order ? 1 : 0;
    const int64_t ntiles = TileIter::total(n, d_full);
    if (!d_full) h->d_upper_only = true;
    const int npairs = std::max(1, h->num_sms / 2);         // CTA pairs (clusters of two)
    for (int64_t t0 = 0; t0 < tokens; t0 += chunk) {
        const int tk = (int)std::min<int64_t>(chunk, tokens - t0);
        const int kp = (tk + UBK - 1) / UBK * UBK;
        const int narr = stats_operand_arrays(h->stats_precision);
        const bool split = narr >= 3, splitd = narr == 4;
        const int buf = h->next_buf;
        h->next_buf ^= 1;
        const size_t buf_bytes = round_up((size_t)narr * n * (size_t)(chunk) * 2, ALIGN);
        __half *Xt = reinterpret_cast<__half *>(h->ws + (size_t)buf * buf_bytes);
        __half *dXt = Xt + (size_t)n * kp;
        __half *Xlo = split ? dXt + (size_t)n * kp : nullptr;
        __half *dXlo = splitd ? Xlo + (size_t)n * kp : nullptr;
        unsigned *amax = h->hd->amax[buf];
        cudaStream_t gs = h->gemm_stream;
        // this buffer was last read by the product issued two chunks ago
        if (h->gemm_pending[buf]) {
            CU(cudaStreamWaitEvent(s, h->gemm_done[buf], 0));
            h->gemm_pending[buf] = false;
        }
        CU(cudaMemsetAsync(amax, 0, 2 * sizeof(unsigned), s));
        ConvertArgs ca;
        ca.X = X + t0 * ld; ca.Xfp = Xfp + t0 * ld; ca.ld = ld; ca.tokens = tk; ca.n = n; ca.kp = kp;
        ca.Xt = Xt; ca.dXt = dXt; ca.Xlo = Xlo; ca.dXlo = dXlo; ca.amax = amax;
        dim3 cgrid(kp / 64, (n + 63) / 64);
        convert_transpose_kernel<0><<<cgrid, 256, 0, s>>>(ca);
        LAUNCHED();
        convert_transpose_kernel<1><<<std::min<unsigned>(cgrid.x * cgrid.y, 4u * (unsigned)h->num_sms), 256, 0, s>>>(ca);
        LAUNCHED();
        CU(cudaEventRecord(h->conv_done[buf], s));
        CU(cudaStreamWaitEvent(gs, h->conv_done[buf], 0));
        CUtensorMap mX, mD, mL, mDL;
        const __half *lo = split ? Xlo : Xt;    // unused maps still have to be valid
        const __half *dlo = splitd ? dXlo : dXt;
        if (!make_kmajor_map(&mX, Xt, n, kp, UBM) || !make_kmajor_map(&mD, dXt, n, kp, UBM) ||
            !make_kmajor_map(&mL, lo, n, kp, UBM) || !make_kmajor_map(&mDL, dlo, n, kp, UBM)) {
            h->cuda_error = "cuTensorMapEncodeTiled failed";
            return GPTAQ_ERR_CUDA;
        }
        StatsGemmArgs ga;
        ga.H = h->H; ga.D = h->D; ga.n = n; ga.kblocks = kp / UBK; ga.nseg_h = split ? 3 : 1; ga.nseg_d = splitd ? 3 : 1; ga.amax = amax; ga.hd = h->hd;
        // the last, partial wave of tiles is cut along K so that every pair has work
        ga.d_full = d_full;
        ga.ntiles = (int)ntiles;
        ga.full_tiles = (int)(ntiles / npairs) * npairs;
        ga.ksplit = 1;
        const int cut = (int)ntiles - ga.full_tiles;
        if (cut > 0) {
            const int by_pairs = npairs / cut, by_k = ga.kblocks / (2 * UCHUNK);
            ga.ksplit = std::max(1, std::min(std::min(by_pairs, by_k), 8));
        }
        if (ga.ksplit == 1) ga.full_tiles = (int)ntiles;
        // scratch behind the two operand buffers (one partial 128 x 256 tile per CTA at most; the products
        // run one after the other on the internal stream, so one scratch serves both buffers)
        ga.scratch = reinterpret_cast<float *>(h->ws + 2 * buf_bytes);
        const int nitems = ga.full_tiles + ((int)ntiles - ga.full_tiles) * ga.ksplit;
        const int sgrid = 2 * std::min(nitems, npairs);
        std::pair<cudaEvent_t, cudaEvent_t> *tev = nullptr;
        if (h->kernel_timing) {
            if (h->timing_used == h->timing_events.size()) {
                std::pair<cudaEvent_t, cudaEvent_t> ev{nullptr, nullptr};
                CU(cudaEventCreate(&ev.first));
                CU(cudaEventCreate(&ev.second));
                h->timing_events.push_back(ev);
            }
            tev = &h->timing_events[h->timing_used++];
            CU(cudaEventRecord(tev->first, gs));
        }
        if (h->fix_pending && (h->fix_args.ksplit != ga.ksplit || h->fix_args.full_tiles != ga.full_tiles ||
                               h->fix_args.ntiles != ga.ntiles || h->fix_args.d_full != ga.d_full ||
                               h->fix_args.scratch != ga.scratch))
            OK(flush_partials(h));              // another cut: the slots change meaning
        if (ga.ksplit > 1 && !h->fix_pending) {
            CU(cudaMemsetAsync(ga.scratch, 0, (size_t)((int)ntiles - ga.full_tiles) * (ga.ksplit - 1) * 2 * UBM * UBN * sizeof(float), gs));
            h->fix_args = ga;
            h->fix_pending = true;
        }
        stats_umma_kernel<<<sgrid, UMMA_THREADS, UMMA_SMEM, gs>>>(mX, mD, mL, mDL, ga);
        LAUNCHED();
        if (tev) CU(cudaEventRecord(tev->second, gs));
        CU(cudaEventRecord(h->gemm_done[buf], gs));
        h->gemm_pending[buf] = true;
    }
    h->tokens += tokens;
    return GPTAQ_OK;
}

bool valid_block(int b) { return b == 32 || b == 64 || b == 128; }

// What the column loop and the trailing update work on: the factor U, the matrix P, the
// dead-input flags, the device status header and the m x 2B scratch for [-Err | Wpre].
struct QuantizeTarget {
    int n;
    const float *U, *P;
    const uint8_t *dead;
    StateHeader *hd;
    TcSched *sched;            // host-side count of the tile numbers drawn from hd->sched_counter
    float *EW;
    int num_sms;
    // float32-grade tensor-core trailing update: split copies of U^T and P^T (n x n, ld n) and
    // the low part of [-Err | Wpre]; all null on the plain-FMA path
    const float *UT_hi, *UT_lo, *PT_hi, *PT_lo;
    float *EW_lo;
    // the same update with FP16-split operands (takes precedence when set): U^T and P^T as fp16 hi / lo
    // (lo = hi + n * n), each with the scale of its recorded maximum, [-Err | Wpre] as fp16 hi / lo with
    // one scale per row
    const __half *UT16 = nullptr, *PT16 = nullptr;
    __half *EW16 = nullptr;
    float *row_inv = nullptr;
    // ... in super-blocks: EW is then m x 2 * QSUPER * B wide; EWS16 its fp16 hi / lo parts (lo = hi +
    // m * 2 * QSUPER * B) with the row scales row_inv_s
    __half *EWS16 = nullptr;
    float *row_inv_s = nullptr;
    const unsigned *amax_u = nullptr, *amax_p = nullptr;
    int terms = GPTAQ_TERM_ERR | GPTAQ_TERM_ASYM;   // which terms of the weight update are applied
    const int *perm = nullptr;                      // act_order: working column c is the caller's column perm[c]
    int clip_steps = 0; float clip_min = 1.f;       // clipping-range search of the grids (0 steps: min/max)
    const uint8_t *dead_orig = nullptr;             // static groups: dead-input flags in the caller's column order
    bool static_groups = false;
};

gptaq_status_t check_quantize_args(int64_t n, const void *d_W, int w_dtype, int64_t m, int64_t ldw, int bits,
                                   int group, int blocksize, const uint8_t *d_codes, const float *d_scales,
                                   const float *d_zeros, const float *d_Wq) {
    if (bits < 2 || bits > 8 || !valid_block(blocksize) || group < 0 ||
        (w_dtype != GPTAQ_W_FP32 && w_dtype != GPTAQ_W_BF16))
        return GPTAQ_ERR_UNSUPPORTED;
    if (group > 0 && (blocksize % group) != 0) return GPTAQ_ERR_UNSUPPORTED;
    if (m == 0) return GPTAQ_OK;
    if (!d_W || !d_codes || !d_scales || !d_zeros || ldw < n) return GPTAQ_ERR_INVALID_ARG;
    if (w_dtype == GPTAQ_W_BF16 && !d_Wq) return GPTAQ_ERR_INVALID_ARG;
    return GPTAQ_OK;
}

#define QLAUNCHED()                                          \
    do {                                                     \
        cudaError_t e__ = cudaGetLastError();                \
        if (e__ != cudaSuccess) { *err = e__; return GPTAQ_ERR_CUDA; } \
        ++*launches;                                         \
    } while (0)

// Algorithm 1, the blocked loop: launch sequence shared by the entry points that quantize.
gptaq_status_t quantize_core(const QuantizeTarget &t, void *d_W, int w_dtype, int64_t m, int64_t ldw,
                             int bits, int group, int sym, int blocksize, uint8_t *d_codes, float *d_scales,
                             float *d_zeros, float *d_Wq, cudaStream_t s, int64_t *launches, cudaError_t *err) {
    const int n = t.n;
    float *EW = t.EW;
    float *Wk = static_cast<float *>(d_W);
    int64_t ldk = ldw;
    if (t.perm) {
        // working copy in sorted column order (the caller's d_Wq; checked to be a second buffer)
        if (w_dtype == GPTAQ_W_BF16)
            gather_cols_kernel<__nv_bfloat16><<<t.num_sms * 8, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(d_W), ldw,
                                                                           d_Wq, n, (int)m, n, t.perm);
        else
            gather_cols_kernel<float><<<t.num_sms * 8, 256, 0, s>>>(static_cast<const float *>(d_W), ldw, d_Wq, n,
                                                                   (int)m, n, t.perm);
        QLAUNCHED();
        Wk = d_Wq; ldk = n;
    } else if (w_dtype == GPTAQ_W_BF16) {
        bf16_to_f32_kernel<<<t.num_sms * 8, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(d_W), ldw,
                                                        d_Wq, n, (int)m, n);
        QLAUNCHED();
        Wk = d_Wq; ldk = n;
    } else if (d_Wq && d_Wq != d_W) {
        copy2d_kernel<<<t.num_sms * 8, 256, 0, s>>>(static_cast<const float *>(d_W), ldw, d_Wq, n,
                                                   (int)m, n);
        QLAUNCHED();
        Wk = d_Wq; ldk = n;
    }

    const int G = group > 0 ? (n + group - 1) / group : 1;
    const bool static_groups = t.static_groups && group > 0;
    if (static_groups) {
        // grids of the original weights (the caller's d_W in its own column order is still untouched)
        const unsigned sg_grid = (unsigned)(((int64_t)m * G + 7) / 8);
        if (w_dtype == GPTAQ_W_BF16)
            static_group_grid_kernel<__nv_bfloat16><<<sg_grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(d_W), ldw, (int)m, n,
                                                                           group, G, t.dead_orig, bits, sym, d_scales, d_zeros,
                                                                           t.clip_steps, t.clip_min);
        else
            static_group_grid_kernel<float><<<sg_grid, 256, 0, s>>>(static_cast<const float *>(d_W), ldw, (int)m, n, group, G,
                                                                   t.dead_orig, bits, sym, d_scales, d_zeros, t.clip_steps,
                                                                   t.clip_min);
        QLAUNCHED();
    }
    if (group <= 0) {
        row_grid_kernel<<<(unsigned)((m + 7) / 8), 256, 0, s>>>(Wk, ldk, (int)m, n, t.dead, bits, sym,
                                                               d_scales, d_zeros, t.clip_steps, t.clip_min);
        QLAUNCHED();
    }

    int nw = (int)((m + t.num_sms - 1) / t.num_sms);
    nw = std::max(1, std::min(32, nw));
    const unsigned cl_grid = (unsigned)((m + nw - 1) / nw);
    const int T = blocksize / 32;
    // rows per CTA of the block kernel: enough CTAs for every SM, at most 128 rows each
    const int cb_rows = 32 * std::max(1, std::min(4, (int)((m + 32 * (int64_t)t.num_sms - 1) / (32 * (int64_t)t.num_sms))));
    const unsigned cb_grid = (unsigned)((m + cb_rows - 1) / cb_rows);
    const size_t cl_smem = 2 * (size_t)blocksize * blocksize * sizeof(float);

    const bool tensor16 = t.EW16 != nullptr;
    const bool tensor = tensor16 || t.EW_lo != nullptr;
    TcMaps maps, maps_super;
    const int SBW = QSUPER * blocksize;           // super-block width (FP16-split update)
    if (tensor16) {
        const size_t nn = (size_t)n * n, me = (size_t)m * 2 * blocksize;
        const SplitOperand A{t.EW16, t.EW16 + me, m, 2 * blocksize, 2 * blocksize, true};
        const SplitOperand AS{t.EWS16, t.EWS16 + (size_t)m * 2 * SBW, m, 2 * SBW, 2 * SBW, true};
        const SplitOperand B{t.UT16, t.UT16 + nn, n, n, n, true}, B2{t.PT16, t.PT16 + nn, n, n, n, true};
        if (!make_tc_maps(&maps, A, B, &B2) || !make_tc_maps(&maps_super, AS, B, &B2)) {
            *err = cudaErrorUnknown;
            return GPTAQ_ERR_CUDA;
        }
    } else if (tensor) {
        const SplitOperand A{EW, t.EW_lo, m, 2 * blocksize, 2 * blocksize};
        const SplitOperand B{t.UT_hi, t.UT_lo, n, n, n}, B2{t.PT_hi, t.PT_lo, n, n, n};
        if (!make_tc_maps(&maps, A, B, &B2)) { *err = cudaErrorUnknown; return GPTAQ_ERR_CUDA; }
    }
    for (int i0 = 0; i0 < n; i0 += blocksize) {
        ColumnLoopArgs a;
        a.W = Wk; a.ldw = ldk; a.m = (int)m; a.n = n; a.U = t.U; a.P = t.P; a.dead = t.dead;
        a.i0 = i0; a.bw = std::min(blocksize, n - i0);
        a.bits = bits; a.group = group; a.sym = sym;
        a.codes = d_codes; a.scales = d_scales; a.zeros = d_zeros; a.G = G; a.EW = EW; a.EW_lo = tensor16 ? nullptr : t.EW_lo; a.hd = t.hd;
        a.ew_ld = 2 * blocksize; a.ew_pre = blocksize;
        a.EW16_hi = tensor16 ? t.EW16 : nullptr; a.EW16_lo = tensor16 ? t.EW16 + (size_t)m * 2 * blocksize : nullptr;
        a.row_inv = t.row_inv; a.amax_u = t.amax_u; a.amax_p = t.amax_p;
        a.perm = t.perm; a.clip_steps = t.clip_steps; a.clip_min = t.clip_min; a.err_scale = (t.terms & GPTAQ_TERM_ERR) ? 1.f : 0.f; a.asym_scale = (t.terms & GPTAQ_TERM_ASYM) ? 1.f : 0.f;
        a.static_groups = static_groups ? 1 : 0;
        // (every full block of one call takes the same kernel: the conditions do not depend on the block)
        const bool fast = a.bw == blocksize && (group <= 0 || (group % 32) == 0) && (i0 % 4) == 0 &&
                          (reinterpret_cast<uintptr_t>(t.dead) & 3) == 0 && !static_groups;
        const int sb0 = i0 / SBW * SBW, sb_end = std::min(sb0 + SBW, n);
        if (fast && tensor16) {
            // this block's columns of the super-block's [-Err | Wpre]
            a.EW = EW + (i0 - sb0); a.ew_ld = 2 * SBW; a.ew_pre = SBW;
        }
        if (fast) {
            const int lanes = column_block_lanes(cb_rows);
            if (lanes == 4) column_block_kernel<4><<<cb_grid, CB_THREADS, column_block_smem(cb_rows), s>>>(a, cb_rows, blocksize);
            else if (lanes == 2) column_block_kernel<2><<<cb_grid, CB_THREADS, column_block_smem(cb_rows), s>>>(a, cb_rows, blocksize);
            else column_block_kernel<1><<<cb_grid, CB_THREADS, column_block_smem(cb_rows), s>>>(a, cb_rows, blocksize);
        }
        else if (T == 4) column_loop_kernel<4><<<cl_grid, nw * 32, cl_smem, s>>>(a);
        else if (T == 2) column_loop_kernel<2><<<cl_grid, nw * 32, cl_smem, s>>>(a);
        else column_loop_kernel<1><<<cl_grid, nw * 32, cl_smem, s>>>(a);
        QLAUNCHED();
        const int i2 = i0 + blocksize;
        if (tensor16 && !fast) {
            // grids per group of fewer than 32 columns: every full block takes column_loop_kernel, which
            // leaves [-Err | rho Wpre] in float32; scaled row by row and split here, then applied to all
            // columns to the right (the ragged last block has none)
            if (i2 < n) {
                rowscale_split16_kernel<<<(unsigned)((m + 7) / 8), 256, 0, s>>>(EW, 2 * blocksize, (int)m, 2 * blocksize, t.EW16,
                                                                              t.EW16 + (size_t)m * 2 * blocksize, t.row_inv);
                QLAUNCHED();
                TcGemmArgs g = tc_args(Wk + i2, ldk, (int)m, n - i2, 2 * blocksize, 1.f, 1.f, TC_FULL, TC_MASK_NONE, t.hd);
                g.b_row0 = i2; g.b_k0 = i0; g.k_split = blocksize; g.b2_k0 = i0;
                g.row_inv = t.row_inv; g.amax_b = t.amax_u;
                *err = launch_tc_gemm(maps, g, *t.sched, t.num_sms, s, false);
                if (*err != cudaSuccess) return GPTAQ_ERR_CUDA;
                ++*launches;
            }
        } else if (tensor16) {
            if (i2 < sb_end) {
                // rest of the super-block: W[:, i2:sb_end] += [-Err | Wpre] * [U[blk, i2:sb_end] ; P[blk, i2:sb_end]]
                TcGemmArgs g = tc_args(Wk + i2, ldk, (int)m, sb_end - i2, 2 * blocksize, 1.f, 1.f, TC_FULL, TC_MASK_NONE, t.hd);
                g.b_row0 = i2; g.b_k0 = i0; g.k_split = blocksize; g.b2_k0 = i0;
                g.row_inv = t.row_inv; g.amax_b = t.amax_u;
                *err = launch_tc_gemm(maps, g, *t.sched, t.num_sms, s, false);
                if (*err != cudaSuccess) return GPTAQ_ERR_CUDA;
                ++*launches;
            } else if (i2 == sb_end && sb_end < n) {
                // super-block done: everything to its right receives all of its errors at once
                rowscale_split16_kernel<<<(unsigned)((m + 7) / 8), 256, 0, s>>>(EW, 2 * SBW, (int)m, 2 * SBW, t.EWS16,
                                                                              t.EWS16 + (size_t)m * 2 * SBW, t.row_inv_s);
                QLAUNCHED();
                TcGemmArgs g = tc_args(Wk + sb_end, ldk, (int)m, n - sb_end, 2 * SBW, 1.f, 1.f, TC_FULL, TC_MASK_NONE, t.hd);
                g.b_row0 = sb_end; g.b_k0 = sb0; g.k_split = SBW; g.b2_k0 = sb0;
                g.row_inv = t.row_inv_s; g.amax_b = t.amax_u;
                *err = launch_tc_gemm(maps_super, g, *t.sched, t.num_sms, s, false);
                if (*err != cudaSuccess) return GPTAQ_ERR_CUDA;
                ++*launches;
            }
        } else if (i2 < n && tensor) {
            // W[:, i2:] += [-Err | Wpre] * [U[blk, i2:] ; P[blk, i2:]] on the tensor cores: B operand rows
            // are rows i2.. of U^T (first B contraction steps) and of P^T (the next B)
            TcGemmArgs g = tc_args(Wk + i2, ldk, (int)m, n - i2, 2 * blocksize, 1.f, 1.f, TC_FULL, TC_MASK_NONE, t.hd);
            g.b_row0 = i2; g.b_k0 = i0; g.k_split = blocksize; g.b2_k0 = i0;
            *err = launch_tc_gemm(maps, g, *t.sched, t.num_sms, s, false);
            if (*err != cudaSuccess) return GPTAQ_ERR_CUDA;
            ++*launches;
        } else if (i2 < n) {
            // W[:, i2:] += [-Err | Wpre] * [U[blk, i2:] ; P[blk, i2:]]   (lazy-batch update)
            Operand bop = make_operand(t.U + (int64_t)i0 * n + i2, 1, n);
            bop.p2 = t.P + (int64_t)i0 * n + i2;
            bop.k_split = blocksize;
            GemmProblem pt = make_problem(make_operand(EW, 2 * blocksize, 1), bop, Wk + i2, ldk,
                                          (int)m, n - i2, 2 * blocksize, 1.f, 1.f, GEMM_FULL);
            *err = launch_simt_gemm(pt, false, true, s);
            if (*err != cudaSuccess) return GPTAQ_ERR_CUDA;
            ++*launches;
        }
    }
    if (t.perm) {
        // dequantized weights back to the caller's column order
        unpermute_rows_kernel<<<(unsigned)m, 256, (size_t)n * sizeof(float), s>>>(Wk, ldk, n, t.perm);
        QLAUNCHED();
    }
    return GPTAQ_OK;
}


// ---------------------------------------------------------------------------
// Built-in scratch of gptaq_quantize_static: one array per GPU that loads the library, held
// until the process exits.  Layout: status header | dead-input flags (all zero) | [-Err | Wpre].
// In host code the array's name is only a stand-in for the symbol, not a device address; the
// address that kernels may use is looked up once per device with cudaGetSymbolAddress.
// ---------------------------------------------------------------------------
constexpr size_t STATIC_FLAGS_OFFSET = 256;
constexpr size_t STATIC_EW_OFFSET = STATIC_FLAGS_OFFSET + GPTAQ_STATIC_MAX_N;
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_EW_OFFSET + (size_t)GPTAQ_STATIC_SCRATCH_FLOATS * sizeof(float);
static_assert(STATIC_EW_OFFSET % 256 == 0, "scratch alignment");
static_assert(sizeof(StateHeader) <= STATIC_FLAGS_OFFSET, "header fits");

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

struct StaticScratch {
    bool ready;
    uint8_t *base;
    int num_sms;
};
constexpr int MAX_DEVICES = 64;
StaticScratch g_static_table[MAX_DEVICES];
std::mutex g_static_mutex;

__global__ void export_status_kernel(const StateHeader *hd, int64_t *out) {
    out[0] = hd->status;
    out[1] = hd->info;
}

// Set-up on first use, once per device, with that device current: resolves the device address
// of the scratch array and raises the shared-memory limit of the column-loop kernels.
cudaError_t static_scratch_for_current_device(StaticScratch **out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticScratch &sc = g_static_table[dev];
    if (!sc.ready) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sc.num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(column_loop_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 2 * 128 * 128 * (int)sizeof(float));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(column_loop_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 2 * 64 * 64 * (int)sizeof(float));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(column_block_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(column_block_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(column_block_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
        if (e != cudaSuccess) return e;
        sc.base = static_cast<uint8_t *>(ptr);
        sc.ready = true;
    }
    *out = &sc;
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t gptaq_state_bytes(int64_t n) {
    if (n <= 0) return 0;
    return state_layout(n).total;
}

size_t gptaq_workspace_bytes(int64_t n, int64_t m_max, int64_t max_batch_tokens, int blocksize) {
    if (n <= 0 || m_max < 0 || max_batch_tokens < 0 || !valid_block(blocksize)) return 0;
    // the fp16 operand copies of one token batch share the space of the later steps' scratch
    size_t kp = round_up((size_t)max_batch_tokens, (size_t)UBK);
    size_t xt = 2 * round_up(3 * (size_t)n * kp * 2, ALIGN) + stats_scratch_bytes(MAX_SMS_FOR_SIZING);
    return std::max(ws_layout(n, m_max, blocksize).total, xt);
}

gptaq_status_t gptaq_create(gptaq_handle_t *out, int64_t n, void *d_state, size_t state_bytes,
                            void *d_workspace, size_t workspace_bytes, gptaq_stream_t stream) {
    if (!out) return GPTAQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (n <= 0 || n > (int64_t)1 << 20 || !d_state || !d_workspace) return GPTAQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_state) % ALIGN) || (reinterpret_cast<uintptr_t>(d_workspace) % ALIGN))
        return GPTAQ_ERR_INVALID_ARG;
    Layout l = state_layout(n);
    if (state_bytes < l.total) return GPTAQ_ERR_WORKSPACE;
    if (workspace_bytes < ws_layout(n, 0, 32).total) return GPTAQ_ERR_WORKSPACE;
    gptaq_ctx *h = new (std::nothrow) gptaq_ctx();
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    h->n = n;
    h->state = static_cast<char *>(d_state);
    h->state_bytes = state_bytes;
    h->ws = static_cast<char *>(d_workspace);
    h->ws_bytes = workspace_bytes;
    h->hd = reinterpret_cast<StateHeader *>(h->state);
    h->H = reinterpret_cast<float *>(h->state + l.h_off);
    h->D = reinterpret_cast<float *>(h->state + l.d_off);
    h->dead = reinterpret_cast<uint8_t *>(h->state + l.dead_off);
    h->dead_raw = reinterpret_cast<uint8_t *>(h->state + l.dead_raw_off);
    h->perm = reinterpret_cast<int *>(h->state + l.perm_off);
    h->act_order = false;
    h->launches = 0;
    h->stats_precision = GPTAQ_STATS_FP16_SPLIT_TENSOR;
    h->tensor = tc_shape_ok(n) && encode_tiled_fn() != nullptr;
    h->f16 = h->tensor && (n % 8) == 0;
    h->terms = GPTAQ_TERM_ERR | GPTAQ_TERM_ASYM;
    h->clip_steps = 0; h->clip_min = 1.f;
    h->static_groups = false;
    h->kernel_timing = false;
    h->timing_used = 0;
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(factor_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FP_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(column_loop_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 2 * 128 * 128 * (int)sizeof(float));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(invert_diag_blocks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ID_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(stats_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)UMMA_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM);
    // the conversion of the next batch shares the SMs with the running product: both kernels ask for
    // the largest shared-memory carve-out, so that a conversion CTA fits beside a product CTA
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(stats_umma_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(convert_transpose_kernel<0>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(convert_transpose_kernel<1>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(column_loop_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 2 * 64 * 64 * (int)sizeof(float));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(column_block_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(column_block_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(column_block_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)column_block_smem(128));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(unpermute_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ACT_ORDER_MAX_N * 4);
    if (e != cudaSuccess) {
        delete h;
        return GPTAQ_ERR_CUDA;
    }
    h->gemm_stream = nullptr;
    h->relayout = false;
    h->next_buf = 0;
    h->fix_pending = false;
    h->d_upper_only = false;
    for (int i = 0; i < 2; ++i) { h->conv_done[i] = h->gemm_done[i] = nullptr; h->gemm_pending[i] = false; }
    {
        // highest priority: when a product and the conversion of the next batch become ready together, the
        // product's CTAs (one per SM, nearly all of its shared memory) are placed first and the conversion
        // fills the SMs that the product's last round of tiles leaves idle
        int prio_lo = 0, prio_hi = 0;
        e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->gemm_stream, cudaStreamNonBlocking, prio_hi);
    }
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&h->conv_done[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->gemm_done[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        gptaq_destroy(h);
        return GPTAQ_ERR_CUDA;
    }
    gptaq_status_t st = gptaq_reset(h, stream);
    if (st != GPTAQ_OK) {
        gptaq_destroy(h);
        return st;
    }
    *out = h;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_reset(gptaq_handle_t h, gptaq_stream_t stream) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    Layout l = state_layout(h->n);
    OK(join_statistics(h, static_cast<cudaStream_t>(stream)));
    CU(cudaMemsetAsync(h->state, 0, l.total, static_cast<cudaStream_t>(stream)));
    h->stage = STAGE_ACCUM;
    h->tokens = 0;
    h->d_upper_only = false;
    h->sched.base = 0;           // the counter in the header was zeroed with the rest of the state
    return GPTAQ_OK;
}

gptaq_status_t gptaq_destroy(gptaq_handle_t h) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    if (h->gemm_stream) {
        cudaStreamSynchronize(h->gemm_stream);
        cudaStreamDestroy(h->gemm_stream);
    }
    for (int i = 0; i < 2; ++i) {
        if (h->conv_done[i]) cudaEventDestroy(h->conv_done[i]);
        if (h->gemm_done[i]) cudaEventDestroy(h->gemm_done[i]);
    }
    for (auto &ev : h->timing_events) { cudaEventDestroy(ev.first); cudaEventDestroy(ev.second); }
    delete h;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_accumulate(gptaq_handle_t h, const float *d_X, const float *d_Xfp,
                                int64_t tokens, int64_t ld, gptaq_stream_t stream) {
    if (!h || tokens < 0 || tokens > INT32_MAX) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_ACCUM) return GPTAQ_ERR_BAD_STATE;
    if (tokens == 0) return GPTAQ_OK;
    if (!d_X || !d_Xfp || ld < h->n) return GPTAQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = (int)h->n;
    if (tc_eligible(h)) return accumulate_tc(h, d_X, d_Xfp, tokens, ld, s);
    OK(join_statistics(h, s));
    // H (upper tiles) += X X^T
    Operand xa = make_operand(d_X, 1, ld);
    GemmProblem ph = make_problem(xa, xa, h->H, n, n, n, (int)tokens, 1.f, 1.f, GEMM_UPPER_TILES);
    OK(gemm(h, ph, true, true, s));
    // dXX^T += (X~ - X) X^T, the difference taken in float32 at load time
    Operand da = xa;
    da.sub = d_Xfp;
    GemmProblem pd = make_problem(da, xa, h->D, n, n, n, (int)tokens, 1.f, 1.f, GEMM_FULL);
    OK(gemm(h, pd, true, true, s));
    h->tokens += tokens;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_flush(gptaq_handle_t h, gptaq_stream_t stream) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    return join_statistics(h, static_cast<cudaStream_t>(stream));
}

gptaq_status_t gptaq_accumulate_host(gptaq_handle_t h, const float *h_X, const float *h_Xfp,
                                     int64_t tokens, int64_t ld, void *d_stage, size_t stage_bytes,
                                     gptaq_stream_t stream) {
    if (!h || tokens < 0) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_ACCUM) return GPTAQ_ERR_BAD_STATE;
    if (tokens == 0) return GPTAQ_OK;
    if (!h_X || !h_Xfp || !d_stage || ld < h->n) return GPTAQ_ERR_INVALID_ARG;
    size_t one = (size_t)tokens * (size_t)h->n * sizeof(float);
    if (stage_bytes < 2 * one) return GPTAQ_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float *dx = static_cast<float *>(d_stage);
    float *dxfp = dx + (size_t)tokens * (size_t)h->n;
    size_t rowb = (size_t)h->n * sizeof(float);
    CU(cudaMemcpy2DAsync(dx, rowb, h_X, (size_t)ld * sizeof(float), rowb, (size_t)tokens,
                         cudaMemcpyHostToDevice, s));
    CU(cudaMemcpy2DAsync(dxfp, rowb, h_Xfp, (size_t)ld * sizeof(float), rowb, (size_t)tokens,
                         cudaMemcpyHostToDevice, s));
    return gptaq_accumulate(h, dx, dxfp, tokens, h->n, stream);
}

gptaq_status_t gptaq_factor(gptaq_handle_t h, float damp, gptaq_stream_t stream) {
    if (!h || !(damp >= 0.f) || !std::isfinite(damp)) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_ACCUM || h->tokens <= 0) return GPTAQ_ERR_BAD_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    OK(join_statistics(h, s));
    const int n = (int)h->n;
    const int nb = (n + NB - 1) / NB;
    WsLayout wl = ws_layout(h->n, 0, 32);
    float *T = reinterpret_cast<float *>(h->ws + wl.t_off);
    float *Rinv = reinterpret_cast<float *>(h->ws + wl.rinv_off);
    float *H = h->H;

    diag_stats_kernel<<<1, 1024, 0, s>>>(H, n, (float)(1.0 / (double)h->tokens), damp, h->hd, h->dead_raw);
    LAUNCHED();
    if (h->act_order) {
        // columns in order of decreasing diag(H): H and dXX^T are permuted on both sides, through T
        rank_desc_kernel<<<(n + 255) / 256, 256, 0, s>>>(H, n, (float)(1.0 / (double)h->tokens), h->dead_raw, h->perm, h->dead);
        LAUNCHED();
        const dim3 pg((n + 255) / 256, n);
        permute_matrix_kernel<<<pg, 256, 0, s>>>(H, T, n, h->perm, 1);
        LAUNCHED();
        CU(cudaMemcpyAsync(H, T, (size_t)n * n * sizeof(float), cudaMemcpyDeviceToDevice, s));
        permute_matrix_kernel<<<pg, 256, 0, s>>>(h->D, T, n, h->perm, 0);
        LAUNCHED();
        CU(cudaMemcpyAsync(h->D, T, (size_t)n * n * sizeof(float), cudaMemcpyDeviceToDevice, s));
    } else {
        CU(cudaMemcpyAsync(h->dead, h->dead_raw, (size_t)n, cudaMemcpyDeviceToDevice, s));
    }
    scale_damp_kernel<<<dim3((n + 63) / 64, (n + 63) / 64), 256, 0, s>>>(H, n, h->hd, h->dead);
    LAUNCHED();

    // reverse Cholesky H_d = R R^T, R upper, from the last block column upwards
    float *pan_hi = h->tensor ? reinterpret_cast<float *>(h->ws + wl.pan_off[0]) : nullptr;
    float *pan_lo = h->tensor ? reinterpret_cast<float *>(h->ws + wl.pan_off[1]) : nullptr;
    TcMaps pan_maps;
    const int pan_ld = h->f16 ? SUPER_NB : NB;
    if (h->tensor) {
        const SplitOperand pan{pan_hi, pan_lo, n, pan_ld, pan_ld, h->f16};
        if (!make_tc_maps(&pan_maps, pan, pan, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
    }
    for (int p = nb - 1; p >= 0; --p) {
        const int b0 = p * NB;
        const int s0 = h->f16 ? b0 / SUPER_NB * SUPER_NB : b0;      // first column of this panel's super-panel
        // diagonal block (factor + inverse) and the panel above it: R[0:b0, blk] = A[0:b0, blk] inv(R_pp)^T
        FactorPanelArgs fa;
        fa.H = H; fa.n = n; fa.b0 = b0; fa.Rdiag = Rinv + (size_t)p * NB * NB;
        fa.pan_hi = pan_hi; fa.pan_lo = pan_lo; fa.pan_f16 = h->f16 ? 1 : 0; fa.hd = h->hd;
        fa.pan_ld = pan_ld; fa.pan_col0 = b0 - s0;
        // rows above the block in tiles of 32, 64 or 128 rows: the smallest tile that still gives every
        // SM at most one tile spreads a short panel over more SMs (the diagonal block is refactored by
        // every CTA either way)
        int tr = 32;
        while (tr < NB && b0 / tr > h->num_sms) tr *= 2;
        fa.tile_rows = tr;
        const int fgrid = std::max(1, std::min(b0 / tr, h->num_sms));
        fa.rows_per_cta = ((b0 + fgrid - 1) / fgrid + tr - 1) / tr * tr;
        // one more CTA, without a slab, stores the diagonal factor while there is an SM left for it
        const int fextra = (b0 > 0 && fgrid < h->num_sms) ? 1 : 0;
        CU(launch_pdl(true, factor_panel_kernel, dim3(fgrid + fextra), dim3(FP_THREADS), FP_SMEM, s, fa));
        h->launches++;
        if (p == 0) break;
        if (h->f16 && b0 >= TC_MIN_N) {
            const unsigned *am = h->hd->tc_amax + AMAX_PAN;
            if (b0 > s0) {
                // inside the super-panel: A[0:b0, s0:b0] -= R[0:b0, blk] R[s0:b0, blk]^T  (upper part)
                TcGemmArgs g = tc_args(H + s0, n, b0, b0 - s0, NB, -1.f, 1.f, TC_UPPER_TILES, TC_MASK_UPPER_KEEP, h->hd);
                g.diag_off = s0; g.a_k0 = g.b_k0 = b0 - s0; g.b_row0 = s0;
                g.amax_a = g.amax_b = am;
                CU(launch_tc_gemm(pan_maps, g, h->sched, h->num_sms, s));
            } else {
                // super-panel [s0, s1) done: A[0:s0, 0:s0] -= R[0:s0, s0:s1] R[0:s0, s0:s1]^T  (upper part)
                const int s1 = std::min(s0 + SUPER_NB, nb * NB);
                TcGemmArgs g = tc_args(H, n, s0, s0, s1 - s0, -1.f, 1.f, TC_UPPER_TILES, TC_MASK_UPPER_KEEP, h->hd);
                g.amax_a = g.amax_b = am;
                CU(launch_tc_gemm(pan_maps, g, h->sched, h->num_sms, s));
            }
            h->launches++;
            continue;
        }
        // A[0:b0, 0:b0] -= R[0:b0, blk] R[0:b0, blk]^T  (upper part)
        if (h->tensor && b0 >= TC_MIN_N) {
            TcGemmArgs g = tc_args(H, n, b0, b0, NB, -1.f, 1.f, TC_UPPER_TILES, TC_MASK_UPPER_KEEP, h->hd);
            CU(launch_tc_gemm(pan_maps, g, h->sched, h->num_sms, s));
            h->launches++;
        } else {
            Operand rp = make_operand(H + b0, n, 1);
            GemmProblem ps = make_problem(rp, rp, H, n, b0, b0, std::min(NB, n - b0), -1.f, 1.f, GEMM_UPPER_TILES);
            OK(gemm(h, ps, false, false, s));
        }
    }

    // U = R^-1: inverted diagonal blocks, then off-diagonal blocks by doubling:
    // inv([[A, B], [0, C]]) = [[A^-1, -A^-1 B C^-1], [0, C^-1]]
    invert_diag_blocks_kernel<<<nb, ID_THREADS, ID_SMEM, s>>>(H, n, Rinv);
    LAUNCHED();
    float *S1h = nullptr, *S1l = nullptr, *S2h = nullptr, *S2l = nullptr;
    TcMaps inv_maps;
    if (h->tensor && !h->f16) {
        S1h = reinterpret_cast<float *>(h->ws + wl.s_off[0]); S1l = reinterpret_cast<float *>(h->ws + wl.s_off[1]);
        S2h = reinterpret_cast<float *>(h->ws + wl.s_off[2]); S2l = reinterpret_cast<float *>(h->ws + wl.s_off[3]);
        const SplitOperand A{S1h, S1l, n, n, n}, B{S2h, S2l, n, n, n};
        if (!make_tc_maps(&inv_maps, A, B, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
    }
    for (int64_t sz = NB; sz < n; sz *= 2) {
        const int np = (int)((n - sz + 2 * sz - 1) / (2 * sz));
        const int tail = (int)(n - (2 * sz * (np - 1) + sz));
        const int64_t bstride = 2 * sz * ((int64_t)n + 1);
        if (h->f16 && damp > 0.f && sz >= 2 * NB) {
            // The two products on the tensor cores with FP16-split operands.  Ranges: B holds entries of R
            // (bounded like the panels), the inverted blocks are bounded by 1 / sqrt(lambda), the
            // intermediate T records its own maximum in the first product's epilogue.
            const size_t nn = (size_t)n * n;
            __half *A1 = reinterpret_cast<__half *>(h->ws + wl.s_off[0]);     // left operands, K-major at their own coordinates
            __half *B2 = reinterpret_cast<__half *>(h->ws + wl.s_off[1]);     // transposed right operands
            unsigned *am = h->hd->tc_amax;
            const SplitOperand Aop{A1, A1 + nn, n, n, n, true}, Bop{B2, B2 + nn, n, n, n, true};
            TcMaps m16;
            if (!make_tc_maps(&m16, Aop, Bop, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
            SplitBatch sb; sb.nbatch = np; sb.src_bstride = sb.dst_bstride = bstride;
            SplitBatch sbt = sb; sbt.cols_last = tail;
            SplitBatch sbc = sb; sbc.rows_last = tail; sbc.cols_last = tail;
            CU(cudaMemsetAsync(am + AMAX_T, 0, sizeof(unsigned), s));
            CU(launch_split16(H + sz, n, A1 + sz, A1 + nn + sz, n, (int)sz, (int)sz, false, SPLIT_ALL, 1.f, am + AMAX_PAN, s, sbt));
            CU(launch_split16(H + sz * n + sz, n, B2 + sz * n + sz, B2 + nn + sz * n + sz, n, (int)sz, (int)sz, true,
                              SPLIT_UPPER, 1.f, am + AMAX_INV, s, sbc));
            TcGemmArgs g1 = tc_args(T + sz, n, (int)sz, (int)sz, (int)sz, 1.f, 0.f, TC_TRI_RIGHT, TC_MASK_NONE, h->hd);
            g1.nbatch = np; g1.c_bstride = bstride; g1.N_last = tail; g1.K_last = tail;
            g1.a_row0 = 0; g1.a_row_bs = (int)(2 * sz); g1.a_k0 = (int)sz; g1.a_k_bs = (int)(2 * sz);
            g1.b_row0 = (int)sz; g1.b_row_bs = (int)(2 * sz); g1.b_k0 = (int)sz; g1.b_k_bs = (int)(2 * sz);
            g1.amax_a = am + AMAX_PAN; g1.amax_b = am + AMAX_INV; g1.amax_out = am + AMAX_T;
            CU(launch_tc_gemm(m16, g1, h->sched, h->num_sms, s));
            CU(launch_split16(H, n, A1, A1 + nn, n, (int)sz, (int)sz, false, SPLIT_UPPER, 1.f, am + AMAX_INV, s, sb));
            CU(launch_split16(T + sz, n, B2 + sz * n, B2 + nn + sz * n, n, (int)sz, (int)sz, true, SPLIT_ALL, 1.f, am + AMAX_T, s, sbt));
            TcGemmArgs g2 = tc_args(H + sz, n, (int)sz, (int)sz, (int)sz, -1.f, 0.f, TC_TRI_LEFT, TC_MASK_NONE, h->hd);
            g2.nbatch = np; g2.c_bstride = bstride; g2.N_last = tail;
            g2.a_row0 = 0; g2.a_row_bs = (int)(2 * sz); g2.a_k0 = 0; g2.a_k_bs = (int)(2 * sz);
            g2.b_row0 = (int)sz; g2.b_row_bs = (int)(2 * sz); g2.b_k0 = 0; g2.b_k_bs = (int)(2 * sz);
            g2.amax_a = am + AMAX_INV; g2.amax_b = am + AMAX_T;
            CU(launch_tc_gemm(m16, g2, h->sched, h->num_sms, s));
            h->launches += 6;
            continue;
        }
        if (h->tensor && !h->f16 && sz >= 2 * NB) {
            // Same two products on the tensor cores, TF32-split operands (widths that are multiples of 4
            // only).  S1 holds K-major copies of the left operands at
            // their own coordinates (B, then A^-1), S2 the transposed right operands (C^-T, then T^T).
            SplitBatch sb; sb.nbatch = np; sb.src_bstride = sb.dst_bstride = bstride;
            SplitBatch sbt = sb; sbt.cols_last = tail;                 // blocks with `tail` columns
            SplitBatch sbc = sb; sbc.rows_last = tail; sbc.cols_last = tail;
            CU(launch_split(H + sz, n, S1h + sz, S1l + sz, n, (int)sz, (int)sz, false, SPLIT_ALL, 1.f, s, sbt));
            h->launches++;
            CU(launch_split(H + sz * n + sz, n, S2h + sz * n + sz, S2l + sz * n + sz, n, (int)sz, (int)sz, true,
                            SPLIT_UPPER, 1.f, s, sbc));
            h->launches++;
            TcGemmArgs g1 = tc_args(T + sz, n, (int)sz, (int)sz, (int)sz, 1.f, 0.f, TC_TRI_RIGHT, TC_MASK_NONE, h->hd);
            g1.nbatch = np; g1.c_bstride = bstride; g1.N_last = tail; g1.K_last = tail;
            g1.a_row0 = 0; g1.a_row_bs = (int)(2 * sz); g1.a_k0 = (int)sz; g1.a_k_bs = (int)(2 * sz);
            g1.b_row0 = (int)sz; g1.b_row_bs = (int)(2 * sz); g1.b_k0 = (int)sz; g1.b_k_bs = (int)(2 * sz);
            CU(launch_tc_gemm(inv_maps, g1, h->sched, h->num_sms, s));
            h->launches++;
            CU(launch_split(H, n, S1h, S1l, n, (int)sz, (int)sz, false, SPLIT_UPPER, 1.f, s, sb));
            h->launches++;
            CU(launch_split(T + sz, n, S2h + sz * n, S2l + sz * n, n, (int)sz, (int)sz, true, SPLIT_ALL, 1.f, s, sbt));
            h->launches++;
            TcGemmArgs g2 = tc_args(H + sz, n, (int)sz, (int)sz, (int)sz, -1.f, 0.f, TC_TRI_LEFT, TC_MASK_NONE, h->hd);
            g2.nbatch = np; g2.c_bstride = bstride; g2.N_last = tail;
            g2.a_row0 = 0; g2.a_row_bs = (int)(2 * sz); g2.a_k0 = 0; g2.a_k_bs = (int)(2 * sz);
            g2.b_row0 = (int)sz; g2.b_row_bs = (int)(2 * sz); g2.b_k0 = 0; g2.b_k_bs = (int)(2 * sz);
            CU(launch_tc_gemm(inv_maps, g2, h->sched, h->num_sms, s));
            h->launches++;
            continue;
        }
        // the 128-wide level, and every level of an fp16-split handle without damping (nothing bounds the
        // inverse in advance then): plain float32 products
        // T = B * C^-1
        GemmProblem p1 = make_problem(make_operand(H + sz, n, 1),
                                      make_operand(H + sz * n + sz, 1, n), T + sz, n,
                                      (int)sz, (int)sz, (int)sz, 1.f, 0.f, GEMM_TRI_RIGHT);
        p1.nbatch = np; p1.batchA = p1.batchB = p1.batchC = bstride;
        p1.batchN_last = tail; p1.batchK_last = tail;
        OK(gemm(h, p1, false, true, s));
        // B <- -A^-1 * T
        GemmProblem p2 = make_problem(make_operand(H, n, 1), make_operand(T + sz, 1, n), H + sz, n,
                                      (int)sz, (int)sz, (int)sz, -1.f, 0.f, GEMM_TRI_LEFT);
        p2.nbatch = np; p2.batchA = p2.batchB = p2.batchC = bstride;
        p2.batchN_last = tail;
        OK(gemm(h, p2, false, true, s));
    }
    if (h->tensor && !h->f16) {
        // operand copies of U for the products that follow: S1 = split(U), S2 = split(U^T)
        // (FP16-split handles make theirs in gptaq_build_P, once the range of U is known)
        CU(launch_split(H, n, S1h, S1l, n, n, n, false, SPLIT_UPPER, 1.f, s));
        h->launches++;
        CU(launch_split(H, n, S2h, S2l, n, n, n, true, SPLIT_UPPER, 1.f, s));
        h->launches++;
    }
    h->stage = STAGE_FACTORED;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_build_P(gptaq_handle_t h, float alpha, gptaq_stream_t stream) {
    if (!h || !std::isfinite(alpha)) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_FACTORED) return GPTAQ_ERR_BAD_STATE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = (int)h->n;
    WsLayout wl = ws_layout(h->n, 0, 32);
    float *O = reinterpret_cast<float *>(h->ws + wl.t_off);
    if (h->tensor && h->f16) {
        // FP16-split operands (half the bytes and twice the MMA rate of the TF32 form): every operand is
        // scaled by a power of two into the fp16 range, so its largest magnitude is recorded first (by a
        // reduction kernel for U and dXX^T, by the producing GEMM's epilogue for O and P).
        // Workspace: S[0] = U^T (kept for gptaq_quantize), S[1] = U, then P^T (kept), S[4] = dXX^T, then O.
        const size_t nn = (size_t)n * n;
        __half *UT16 = reinterpret_cast<__half *>(h->ws + wl.s_off[0]);
        __half *U16 = reinterpret_cast<__half *>(h->ws + wl.s_off[1]);
        __half *A16 = reinterpret_cast<__half *>(h->ws + wl.s_off[4]);
        unsigned *am = h->hd->tc_amax;
        const float inv_tokens = (float)(1.0 / (double)h->tokens);
        CU(cudaMemsetAsync(am + AMAX_U, 0, 4 * sizeof(unsigned), s));      // slots U, D, O, P
        CU(launch_absmax(h->H, n, n, n, SPLIT_UPPER, 1.f, am + AMAX_U, h->num_sms, s));
        // (of dXX^T only the entries above the diagonal reach O: row j of U starts at column j and M_U keeps j > i)
        CU(launch_absmax(h->D, n, n, n, SPLIT_STRICT_UPPER, inv_tokens, am + AMAX_D, h->num_sms, s));
        CU(launch_split16(h->H, n, U16, U16 + nn, n, n, n, false, SPLIT_UPPER, 1.f, am + AMAX_U, s, SplitBatch(),
                          UT16, UT16 + nn));        // U and U^T in one pass
        CU(launch_split16(h->D, n, A16, A16 + nn, n, n, n, false, SPLIT_STRICT_UPPER, inv_tokens, am + AMAX_D, s));
        h->launches += 4;
        const SplitOperand Uop{U16, U16 + nn, n, n, n, true}, UTop{UT16, UT16 + nn, n, n, n, true};
        const SplitOperand Aop{A16, A16 + nn, n, n, n, true};
        TcMaps maps;
        // O = ((dXX^T / tokens) U^T) .* M_U  (contraction over k >= column, U[a][k] = 0 below)
        if (!make_tc_maps(&maps, Aop, Uop, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
        TcGemmArgs go = tc_args(O, n, n, n, n, 1.f, 0.f, TC_O, TC_MASK_STRICT_ZERO, h->hd);
        go.amax_a = am + AMAX_D; go.amax_b = am + AMAX_U; go.amax_out = am + AMAX_O;
        CU(launch_tc_gemm(maps, go, h->sched, h->num_sms, s));
        CU(launch_split16(O, n, A16, A16 + nn, n, n, n, false, SPLIT_STRICT_UPPER, 1.f, am + AMAX_O, s));
        // P = alpha * O U  (B operand rows are rows of U^T)
        if (!make_tc_maps(&maps, Aop, UTop, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
        TcGemmArgs gp = tc_args(h->D, n, n, n, n, alpha, 0.f, TC_P, TC_MASK_STRICT_ZERO, h->hd);
        gp.amax_a = am + AMAX_O; gp.amax_b = am + AMAX_U; gp.amax_out = am + AMAX_P;
        CU(launch_tc_gemm(maps, gp, h->sched, h->num_sms, s));
        // P^T for the lazy-batch updates of gptaq_quantize, over the copy of U that is no longer needed
        CU(launch_split16(h->D, n, U16, U16 + nn, n, n, n, true, SPLIT_STRICT_UPPER, 1.f, am + AMAX_P, s));
        h->launches += 4;
        h->stage = STAGE_P;
        return GPTAQ_OK;
    }
    if (h->tensor) {
        float *S[6];
        for (int i = 0; i < 6; ++i) S[i] = reinterpret_cast<float *>(h->ws + wl.s_off[i]);
        const SplitOperand Us{S[0], S[1], n, n, n}, UTs{S[2], S[3], n, n, n}, S3{S[4], S[5], n, n, n};
        TcMaps maps;
        // S3 = split(dXX^T / tokens);  O = (S3 U^T) .* M_U  (contraction over k >= column, U[a][k] = 0 below)
        CU(launch_split(h->D, n, S[4], S[5], n, n, n, false, SPLIT_ALL, (float)(1.0 / (double)h->tokens), s));
        h->launches++;
        if (!make_tc_maps(&maps, S3, Us, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
        CU(launch_tc_gemm(maps, tc_args(O, n, n, n, n, 1.f, 0.f, TC_O, TC_MASK_STRICT_ZERO, h->hd), h->sched, h->num_sms, s));
        h->launches++;
        // S3 = split(O);  P = alpha * O U  (B operand rows are rows of U^T)
        CU(launch_split(O, n, S[4], S[5], n, n, n, false, SPLIT_STRICT_UPPER, 1.f, s));
        h->launches++;
        if (!make_tc_maps(&maps, S3, UTs, nullptr)) { h->cuda_error = "cuTensorMapEncodeTiled failed"; return GPTAQ_ERR_CUDA; }
        CU(launch_tc_gemm(maps, tc_args(h->D, n, n, n, n, alpha, 0.f, TC_P, TC_MASK_STRICT_ZERO, h->hd), h->sched, h->num_sms, s));
        h->launches++;
        // S3 = split(P^T) for the lazy-batch updates of gptaq_quantize
        CU(launch_split(h->D, n, S[4], S[5], n, n, n, true, SPLIT_STRICT_UPPER, 1.f, s));
        h->launches++;
        h->stage = STAGE_P;
        return GPTAQ_OK;
    }
    // O = (dXX^T U^T) .* M_U
    GemmProblem po = make_problem(make_operand(h->D, n, 1), make_operand(h->H, n, 1), O, n, n, n, n,
                                  1.f, 0.f, GEMM_O);
    OK(gemm(h, po, false, false, s));
    // P = (alpha / tokens) * O U
    GemmProblem pp = make_problem(make_operand(O, n, 1), make_operand(h->H, 1, n), h->D, n, n, n, n,
                                  (float)((double)alpha / (double)h->tokens), 0.f, GEMM_P);
    OK(gemm(h, pp, false, true, s));
    h->stage = STAGE_P;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_build_P_rowwise(gptaq_handle_t h, float alpha, gptaq_stream_t stream) {
    if (!h || !std::isfinite(alpha)) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_FACTORED) return GPTAQ_ERR_BAD_STATE;
    if (h->n > P_ROWWISE_MAX_N) return GPTAQ_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = (int)h->n;
    CU(cudaFuncSetAttribute(p_rowwise_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(2 * P_ROWWISE_MAX_N * sizeof(float))));
    p_rowwise_kernel<<<n, PR_THREADS, 2 * (size_t)n * sizeof(float), s>>>(h->D, h->H, n, (float)((double)alpha / (double)h->tokens));
    LAUNCHED();
    // the operand copies that gptaq_quantize reads, as gptaq_build_P leaves them
    WsLayout wl = ws_layout(h->n, 0, 32);
    if (h->tensor && h->f16) {
        const size_t nn = (size_t)n * n;
        __half *UT16 = reinterpret_cast<__half *>(h->ws + wl.s_off[0]);
        __half *PT16 = reinterpret_cast<__half *>(h->ws + wl.s_off[1]);
        unsigned *am = h->hd->tc_amax;
        CU(cudaMemsetAsync(am + AMAX_U, 0, 4 * sizeof(unsigned), s));
        CU(launch_absmax(h->H, n, n, n, SPLIT_UPPER, 1.f, am + AMAX_U, h->num_sms, s));
        CU(launch_absmax(h->D, n, n, n, SPLIT_STRICT_UPPER, 1.f, am + AMAX_P, h->num_sms, s));
        CU(launch_split16(h->H, n, UT16, UT16 + nn, n, n, n, true, SPLIT_UPPER, 1.f, am + AMAX_U, s));
        CU(launch_split16(h->D, n, PT16, PT16 + nn, n, n, n, true, SPLIT_STRICT_UPPER, 1.f, am + AMAX_P, s));
        h->launches += 4;
    } else if (h->tensor) {
        float *S4 = reinterpret_cast<float *>(h->ws + wl.s_off[4]), *S5 = reinterpret_cast<float *>(h->ws + wl.s_off[5]);
        CU(launch_split(h->D, n, S4, S5, n, n, n, true, SPLIT_STRICT_UPPER, 1.f, s));
        h->launches++;
    }
    h->stage = STAGE_P;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_quantize(gptaq_handle_t h, void *d_W, int w_dtype, int64_t m, int64_t ldw,
                              int bits, int group, int sym, int blocksize,
                              uint8_t *d_codes, float *d_scales, float *d_zeros, float *d_Wq,
                              gptaq_stream_t stream) {
    if (!h || m < 0 || m > INT32_MAX) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_P) return GPTAQ_ERR_BAD_STATE;
    gptaq_status_t st = check_quantize_args(h->n, d_W, w_dtype, m, ldw, bits, group, blocksize, d_codes,
                                            d_scales, d_zeros, d_Wq);
    if (st != GPTAQ_OK || m == 0) return st;
    if (h->act_order && (!d_Wq || d_Wq == d_W)) return GPTAQ_ERR_INVALID_ARG;
    WsLayout wl = ws_layout(h->n, m, blocksize);
    if (h->ws_bytes < wl.total) return GPTAQ_ERR_WORKSPACE;
    QuantizeTarget t;
    t.n = (int)h->n; t.U = h->H; t.P = h->D; t.dead = h->dead; t.hd = h->hd; t.sched = &h->sched;
    t.EW = reinterpret_cast<float *>(h->ws + wl.ew_off);
    t.num_sms = h->num_sms;
    t.terms = h->terms;
    t.perm = h->act_order ? h->perm : nullptr;
    t.clip_steps = h->clip_steps; t.clip_min = h->clip_min;
    t.static_groups = h->static_groups; t.dead_orig = h->dead_raw;
    t.UT_hi = t.UT_lo = t.PT_hi = t.PT_lo = nullptr; t.EW_lo = nullptr;
    // FP16-split trailing update where a block is a whole number of 64-step K-blocks; TF32-split for
    // widths that are multiples of 4 only; plain float32 products otherwise (blocks of 32 columns)
    const bool f16 = h->f16 && (blocksize % 64) == 0;
    if (f16) {
        t.UT16 = reinterpret_cast<const __half *>(h->ws + wl.s_off[0]);
        t.PT16 = reinterpret_cast<const __half *>(h->ws + wl.s_off[1]);
        t.EWS16 = reinterpret_cast<__half *>(h->ws + wl.ew_lo_off);
        t.EW16 = reinterpret_cast<__half *>(h->ws + wl.ew16_off);
        t.row_inv = reinterpret_cast<float *>(h->ws + wl.rs_off);
        t.row_inv_s = t.row_inv + m;
        t.amax_u = h->hd->tc_amax + AMAX_U; t.amax_p = h->hd->tc_amax + AMAX_P;
    } else if (h->tensor && !h->f16) {
        float *S[6];
        for (int i = 0; i < 6; ++i) S[i] = reinterpret_cast<float *>(h->ws + wl.s_off[i]);
        t.UT_hi = S[2]; t.UT_lo = S[3]; t.PT_hi = S[4]; t.PT_lo = S[5];
        t.EW_lo = reinterpret_cast<float *>(h->ws + wl.ew_lo_off);
    }
    cudaError_t e = cudaSuccess;
    st = quantize_core(t, d_W, w_dtype, m, ldw, bits, group, sym, blocksize, d_codes, d_scales, d_zeros, d_Wq,
                       static_cast<cudaStream_t>(stream), &h->launches, &e);
    if (st == GPTAQ_ERR_CUDA) h->cuda_error = cudaGetErrorString(e);
    return st;
}

size_t gptaq_quantize_stage_bytes(int64_t m, int64_t n, int group) {
    if (m < 0 || n <= 0 || group < 0) return 0;
    size_t G = group > 0 ? (size_t)((n + group - 1) / group) : 1;
    return round_up((size_t)m * n * sizeof(float), ALIGN) + round_up((size_t)m * n, ALIGN) +
           2 * round_up((size_t)m * G * sizeof(float), ALIGN);
}

gptaq_status_t gptaq_quantize_host(gptaq_handle_t h, const float *h_W, int64_t m, int64_t ldw,
                                   int bits, int group, int sym, int blocksize,
                                   uint8_t *h_codes, float *h_scales, float *h_zeros, float *h_Wq,
                                   void *d_stage, size_t stage_bytes, gptaq_stream_t stream) {
    if (!h || m < 0) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_P) return GPTAQ_ERR_BAD_STATE;
    if (m == 0) return GPTAQ_OK;
    if (!h_W || !h_codes || !h_scales || !h_zeros || !d_stage || ldw < h->n || group < 0)
        return GPTAQ_ERR_INVALID_ARG;
    if (stage_bytes < gptaq_quantize_stage_bytes(m, h->n, group)) return GPTAQ_ERR_WORKSPACE;
    const size_t n = (size_t)h->n;
    const size_t G = group > 0 ? (n + group - 1) / group : 1;
    char *base = static_cast<char *>(d_stage);
    float *dW = reinterpret_cast<float *>(base);
    uint8_t *dC = reinterpret_cast<uint8_t *>(base + round_up((size_t)m * n * sizeof(float), ALIGN));
    float *dS = reinterpret_cast<float *>(reinterpret_cast<char *>(dC) + round_up((size_t)m * n, ALIGN));
    float *dZ = reinterpret_cast<float *>(reinterpret_cast<char *>(dS) + round_up((size_t)m * G * sizeof(float), ALIGN));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpy2DAsync(dW, n * sizeof(float), h_W, (size_t)ldw * sizeof(float), n * sizeof(float),
                         (size_t)m, cudaMemcpyHostToDevice, s));
    OK(gptaq_quantize(h, dW, GPTAQ_W_FP32, m, (int64_t)n, bits, group, sym, blocksize, dC, dS, dZ, nullptr,
                      stream));
    CU(cudaMemcpyAsync(h_codes, dC, (size_t)m * n, cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(h_scales, dS, (size_t)m * G * sizeof(float), cudaMemcpyDeviceToHost, s));
    CU(cudaMemcpyAsync(h_zeros, dZ, (size_t)m * G * sizeof(float), cudaMemcpyDeviceToHost, s));
    if (h_Wq) CU(cudaMemcpyAsync(h_Wq, dW, (size_t)m * n * sizeof(float), cudaMemcpyDeviceToHost, s));
    return GPTAQ_OK;
}

gptaq_status_t gptaq_quantize_static(const float *d_U, const float *d_P, int64_t n, void *d_W, int w_dtype,
                                     int64_t m, int64_t ldw, int bits, int group, int sym, int blocksize,
                                     uint8_t *d_codes, float *d_scales, float *d_zeros, float *d_Wq,
                                     int64_t *d_status, gptaq_stream_t stream) {
    if (!d_U || !d_P || n <= 0 || m < 0 || m > INT32_MAX) return GPTAQ_ERR_INVALID_ARG;
    gptaq_status_t st = check_quantize_args(n, d_W, w_dtype, m, ldw, bits, group, blocksize, d_codes, d_scales,
                                            d_zeros, d_Wq);
    if (st != GPTAQ_OK) return st;
    // the limits of the built-in scratch come before anything touches the device
    if (n > GPTAQ_STATIC_MAX_N || (int64_t)m * 2 * blocksize > GPTAQ_STATIC_SCRATCH_FLOATS)
        return GPTAQ_ERR_WORKSPACE;
    if (m == 0) return GPTAQ_OK;
    StaticScratch *sc = nullptr;
    cudaError_t e = static_scratch_for_current_device(&sc);
    if (e != cudaSuccess) return GPTAQ_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // every call shares the array and finds the last call's contents: the status header and
    // the all-zero dead-input flags have to start from zero
    e = cudaMemsetAsync(sc->base, 0, STATIC_EW_OFFSET, s);
    if (e != cudaSuccess) return GPTAQ_ERR_CUDA;
    QuantizeTarget t;
    TcSched static_sched;        // (the header is zeroed at every call; this path launches no tensor-core GEMM)
    t.n = (int)n; t.U = d_U; t.P = d_P; t.sched = &static_sched;
    t.hd = reinterpret_cast<StateHeader *>(sc->base);
    t.dead = sc->base + STATIC_FLAGS_OFFSET;
    t.EW = reinterpret_cast<float *>(sc->base + STATIC_EW_OFFSET);
    t.num_sms = sc->num_sms;
    t.UT_hi = t.UT_lo = t.PT_hi = t.PT_lo = nullptr; t.EW_lo = nullptr;
    int64_t launches = 0;
    st = quantize_core(t, d_W, w_dtype, m, ldw, bits, group, sym, blocksize, d_codes, d_scales, d_zeros, d_Wq, s,
                       &launches, &e);
    if (st != GPTAQ_OK) return st;
    if (d_status) {
        export_status_kernel<<<1, 1, 0, s>>>(t.hd, d_status);
        if (cudaGetLastError() != cudaSuccess) return GPTAQ_ERR_CUDA;
    }
    return GPTAQ_OK;
}

gptaq_status_t gptaq_sync_status(gptaq_handle_t h, int64_t *info, gptaq_stream_t stream) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    OK(join_statistics(h, s));
    StateHeader hd;
    CU(cudaMemcpyAsync(&hd, h->hd, sizeof(hd), cudaMemcpyDeviceToHost, s));
    CU(cudaStreamSynchronize(s));
    if (info) *info = hd.info;
    return static_cast<gptaq_status_t>(hd.status);
}

float *gptaq_H(gptaq_handle_t h) { return h ? h->H : nullptr; }
float *gptaq_D(gptaq_handle_t h) { return h ? h->D : nullptr; }
const float *gptaq_U(gptaq_handle_t h) { return (h && h->stage != STAGE_ACCUM) ? h->H : nullptr; }
const float *gptaq_P(gptaq_handle_t h) { return (h && h->stage == STAGE_P) ? h->D : nullptr; }

gptaq_status_t gptaq_selftest_bounded_wait(gptaq_handle_t h, double seconds, gptaq_stream_t stream) {
    if (!h || !(seconds > 0.0) || seconds > 2.0) return GPTAQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int khz = 0;
    CU(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, h->device));
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(h->hd, (long long)(seconds * 1e3 * (double)khz));
    LAUNCHED();
    return GPTAQ_OK;
}
int64_t gptaq_tokens(gptaq_handle_t h) { return h ? h->tokens : -1; }

gptaq_status_t gptaq_set_tokens(gptaq_handle_t h, int64_t tokens) {
    if (!h || tokens < 0) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_ACCUM) return GPTAQ_ERR_BAD_STATE;
    h->tokens = tokens;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_set_stats_precision(gptaq_handle_t h, int precision) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    if (precision != GPTAQ_STATS_FP16_TENSOR && precision != GPTAQ_STATS_FP32 &&
        precision != GPTAQ_STATS_FP16_SPLIT_TENSOR && precision != GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR)
        return GPTAQ_ERR_UNSUPPORTED;
    if (h->stage != STAGE_ACCUM) return GPTAQ_ERR_BAD_STATE;
    if (precision != h->stats_precision) h->relayout = true;
    h->stats_precision = precision;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_set_act_order(gptaq_handle_t h, int enable) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    if (h->stage != STAGE_ACCUM) return GPTAQ_ERR_BAD_STATE;
    if (enable && h->n > ACT_ORDER_MAX_N) return GPTAQ_ERR_UNSUPPORTED;
    // the permutation needs the part of dXX^T below the diagonal, which earlier batches did not accumulate
    if (enable && !h->act_order && h->d_upper_only) return GPTAQ_ERR_BAD_STATE;
    h->act_order = enable != 0;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_set_static_groups(gptaq_handle_t h, int enable) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    h->static_groups = enable != 0;
    return GPTAQ_OK;
}

const int32_t *gptaq_perm(gptaq_handle_t h) { return (h && h->act_order && h->stage != STAGE_ACCUM) ? h->perm : nullptr; }

gptaq_status_t gptaq_set_clip_search(gptaq_handle_t h, int steps, float min_ratio) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    if (steps < 0 || steps > 1024) return GPTAQ_ERR_UNSUPPORTED;
    if (steps > 0 && !(min_ratio > 0.f && min_ratio < 1.f)) return GPTAQ_ERR_INVALID_ARG;
    h->clip_steps = steps;
    h->clip_min = steps > 0 ? min_ratio : 1.f;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_set_update_terms(gptaq_handle_t h, int terms) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    if (terms & ~(GPTAQ_TERM_ERR | GPTAQ_TERM_ASYM)) return GPTAQ_ERR_UNSUPPORTED;
    h->terms = terms;
    return GPTAQ_OK;
}

int gptaq_recommended_stats_precision(int64_t n, int64_t total_tokens) {
    // fp16 rounding of X perturbs U by about 5e-5 * sqrt(n/k) / ((1 - sqrt(n/k))^2 + damp):
    // below 1e-4 with margin once there are 16 tokens per input channel.
    return (n > 0 && total_tokens >= 16 * n) ? GPTAQ_STATS_FP16_TENSOR : GPTAQ_STATS_FP16_SPLIT_TENSOR;
}

int64_t gptaq_launch_count(gptaq_handle_t h) { return h ? h->launches : -1; }

gptaq_status_t gptaq_set_kernel_timing(gptaq_handle_t h, int enable) {
    if (!h) return GPTAQ_ERR_INVALID_ARG;
    h->kernel_timing = enable != 0;
    return GPTAQ_OK;
}

gptaq_status_t gptaq_stats_kernel_time(gptaq_handle_t h, double *ms_total, int64_t *launches) {
    if (!h || !ms_total || !launches) return GPTAQ_ERR_INVALID_ARG;
    double total = 0.0;
    for (size_t i = 0; i < h->timing_used; ++i) {
        CU(cudaEventSynchronize(h->timing_events[i].second));
        float ms = 0.f;
        CU(cudaEventElapsedTime(&ms, h->timing_events[i].first, h->timing_events[i].second));
        total += ms;
    }
    *ms_total = total;
    *launches = (int64_t)h->timing_used;
    h->timing_used = 0;
    return GPTAQ_OK;
}

const char *gptaq_status_string(gptaq_status_t s) {
    switch (s) {
        case GPTAQ_OK: return "ok";
        case GPTAQ_ERR_INVALID_ARG: return "invalid argument";
        case GPTAQ_ERR_BAD_STATE: return "call out of order";
        case GPTAQ_ERR_WORKSPACE: return "buffer too small";
        case GPTAQ_ERR_NOT_SPD: return "damped H is not positive definite";
        case GPTAQ_ERR_NONFINITE: return "non-finite value";
        case GPTAQ_ERR_TIMEOUT: return "bounded device wait ran out";
        case GPTAQ_ERR_UNSUPPORTED: return "unsupported argument combination";
        case GPTAQ_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

const char *gptaq_last_cuda_error(gptaq_handle_t h) { return h ? h->cuda_error.c_str() : ""; }

}  // extern "C"
