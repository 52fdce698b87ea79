// Small kernels of the GPTAQ layer solve: damping, the diagonal-block reverse
// Cholesky, the per-column quantize-and-propagate loop, and helpers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gptaq {

// Device-resident header at the start of the caller's state buffer.
struct StateHeader {
    int status;          // first device-side condition (gptaq_status_t), 0 = none
    int pad0;
    long long info;      // index that goes with it
    float lambda;        // damp * mean(diag H / tokens)
    float inv_tokens;
    unsigned amax[2][2]; // per operand buffer: bit patterns of max|X| and max|X~ - X| of the batch converted into it
    unsigned tc_amax[8]; // largest magnitudes of FP16-split operands of the float32-grade GEMMs (see tc_gemm.cuh)
    unsigned sched_counter; // tile numbers drawn by the float32-grade GEMM launches so far (never reset between launches)
    int pad1[13];
};
static_assert(sizeof(StateHeader) == 128, "header size");

constexpr int ST_NOT_SPD = 4, ST_NONFINITE = 5, ST_TIMEOUT = 6;

// Slots of StateHeader::tc_amax: factor panels (an a-priori bound), U, dXX^T / tokens, O, P, the blocks of
// the inverse factor while it is built (an a-priori bound), the intermediate product of one doubling level.
enum { AMAX_PAN = 0, AMAX_U = 1, AMAX_D = 2, AMAX_O = 3, AMAX_P = 4, AMAX_INV = 5, AMAX_T = 6 };

// Scale of an FP16-split operand: a power of two that puts the largest magnitude into [2^13, 2^14).
__host__ __device__ __forceinline__ float split_scale(float amax) {
    if (!(amax > 0.f) || !isfinite(amax)) return 1.f;
    int e;
    frexpf(amax, &e);                 // amax = f * 2^e, f in [0.5, 1)
    return ldexpf(1.f, 14 - e);
}

// Round to the nearest TF32 value (10 explicit mantissa bits), kept in a float.
__device__ __forceinline__ float tf32_rn(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may be
// scheduled while its predecessor in the stream drains; pdl_wait() returns once the predecessor has
// completed and its writes are visible (a no-op for a plain launch), pdl_launch_dependents() lets the
// successor be scheduled from here on.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void record_status(StateHeader *hd, int code, long long info) {
    if (atomicCAS(&hd->status, 0, code) == 0) hd->info = info;
}

// ---------------------------------------------------------------------------
// lambda = damp * mean_q(H_qq / tokens, dead -> 1); dead flags.  One CTA, fixed
// reduction order (deterministic).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) diag_stats_kernel(const float *H, int n, float inv_tokens,
                                                          float damp, StateHeader *hd,
                                                          uint8_t *dead) {
    __shared__ double red[1024];
    __shared__ float redmax[1024];
    double s = 0.0;
    float mx = 0.f;
    for (int q = threadIdx.x; q < n; q += 1024) {
        float d = H[(int64_t)q * n + q];
        if (!isfinite(d)) record_status(hd, ST_NONFINITE, q);
        bool dd = (d == 0.f);
        dead[q] = dd ? 1 : 0;
        const float v = dd ? 1.f : d * inv_tokens;
        s += dd ? 1.0 : (double)d * (double)inv_tokens;
        mx = fmaxf(mx, v);
    }
    red[threadIdx.x] = s;
    redmax[threadIdx.x] = mx;
    __syncthreads();
    for (int w = 512; w > 0; w >>= 1) {
        if (threadIdx.x < w) {
            red[threadIdx.x] += red[threadIdx.x + w];
            redmax[threadIdx.x] = fmaxf(redmax[threadIdx.x], redmax[threadIdx.x + w]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const float lambda = (float)((double)damp * red[0] / (double)n);
        hd->lambda = lambda;
        hd->inv_tokens = inv_tokens;
        // every entry of row i of the factor R (H_d = R R^T) is at most sqrt(H_d,ii): the range of the
        // factor panels is known before they exist
        hd->tc_amax[AMAX_PAN] = __float_as_uint(sqrtf(redmax[0] + lambda));
        // ... and H_d >= lambda I bounds every entry of R^-1 (and of the inverse of any diagonal block of R)
        // by 1 / sqrt(lambda)
        hd->tc_amax[AMAX_INV] = lambda > 0.f ? __float_as_uint(rsqrtf(lambda)) : 0u;
    }
}

// Upper triangle: H <- H * inv_tokens (+ lambda on the diagonal, dead -> 1 + lambda);
// strict lower triangle <- 0.
__global__ void __launch_bounds__(256) scale_damp_kernel(float *H, int n, const StateHeader *hd,
                                                         const uint8_t *dead) {
    int j = blockIdx.x * 64 + (threadIdx.x & 63);
    int ib = blockIdx.y * 64;
    if (j >= n) return;
    float inv = hd->inv_tokens, lam = hd->lambda;
    for (int r = threadIdx.x >> 6; r < 64; r += 4) {
        int i = ib + r;
        if (i >= n) break;
        float *p = H + (int64_t)i * n + j;
        if (j < i) *p = 0.f;
        else if (j == i) *p = (dead[i] ? 1.f : *p * inv) + lam;
        else *p = *p * inv;
    }
}

// ---------------------------------------------------------------------------
// One panel step of the reverse Cholesky  H_d = R R^T  (R upper), block column
// [b0, b0 + NB):
//   1. factor the NB x NB diagonal block from its last row/column upwards in shared memory,
//      32 columns at a time: one warp factors the 32 x 32 diagonal sub-block in registers
//      (lane = row, shuffles), the rows above it are solved against the sub-block one thread per
//      row, and the leading part receives the rank-32 update (all threads, the tiles of the upper
//      triangle numbered densely);
//   2. rows above the block:  R[0:b0, blk] = A[0:b0, blk] * R_pp^-T, 32 columns at a time: a product
//      with the inverse of the 32 x 32 diagonal sub-block (the four inverses: one warp each, lane =
//      column), then a rank-32 update of the columns to the left, all threads on both; written back in place and, if asked for, as split parts for the tensor-core rank update.
// Every CTA repeats step 1 (it is short and the other SMs would idle) and then takes a
// slab of rows of step 2, whose first tile is fetched while step 1 runs; the last CTA stores R_pp for
// invert_diag_blocks_kernel.  Rows/columns beyond n are padded with the identity.
// ---------------------------------------------------------------------------
constexpr int NB = 128;
constexpr int FP_THREADS = 512;
constexpr int FP_WARPS = FP_THREADS / 32;
constexpr int FP_LD = NB + 4;
constexpr int FP_YLD = 36;
constexpr size_t FP_SMEM = (2 * NB * FP_LD + 32 * FP_LD + 4 * 32 * FP_YLD + NB + 64) * sizeof(float);

struct FactorPanelArgs {
    float *H; int n; int b0;
    float *Rdiag;              // NB x NB (ld NB): the diagonal factor R_pp (upper, zeros below)
    float *pan_hi, *pan_lo;    // nullptr, or [n][NB]: TF32 parts of the panel rows
    int pan_f16;               // the two arrays hold __half instead: fp16 parts of split_scale(tc_amax[AMAX_PAN]) * row,
    int pan_ld, pan_col0;      //   row pitch pan_ld, this panel at columns pan_col0 .. + NB (several panels side by side)
    int rows_per_cta;          // slab of step 2, a multiple of tile_rows
    int tile_rows;             // rows of the slab processed at a time: 32, 64 or 128
    StateHeader *hd;
};

template <int K, int LEN>
struct SolveRowStep {
    static __device__ __forceinline__ void run(float (&a)[LEN], const float *Rt, int ld, const float *dinv) {
        const float x = a[K] * dinv[K];
        a[K] = x;
        const float *col = Rt + K * ld;
#pragma unroll
        for (int j4 = 0; j4 < (K + 3) / 4; ++j4) {
            const float4 r = *reinterpret_cast<const float4 *>(col + 4 * j4);
            if (4 * j4 + 0 < K) a[4 * j4 + 0] = fmaf(-x, r.x, a[4 * j4 + 0]);
            if (4 * j4 + 1 < K) a[4 * j4 + 1] = fmaf(-x, r.y, a[4 * j4 + 1]);
            if (4 * j4 + 2 < K) a[4 * j4 + 2] = fmaf(-x, r.z, a[4 * j4 + 2]);
            if (4 * j4 + 3 < K) a[4 * j4 + 3] = fmaf(-x, r.w, a[4 * j4 + 3]);
        }
        SolveRowStep<K - 1, LEN>::run(a, Rt, ld, dinv);
    }
};
template <int LEN>
struct SolveRowStep<-1, LEN> {
    static __device__ __forceinline__ void run(float (&)[LEN], const float *, int, const float *) {}
};
template <int LEN>
__device__ __forceinline__ void solve_row(float (&a)[LEN], const float *Rt, int ld, const float *dinv) {
    SolveRowStep<LEN - 1, LEN>::run(a, Rt, ld, dinv);
}

// One column step (K, then K - 1, ... 0) of the 32 x 32 reverse Cholesky held one row per lane.
// `piv` is the pivot of this step, already broadcast: the dependent chain from one pivot to the
// next runs through lane K - 1 alone (its own c), the other lanes' updates overlap with it.
// The scaled column c reaches the other lanes through shared memory (cv: two buffers of 32 floats,
// read back as broadcast float4s): K shuffles per step, one per element, cost three times as much.
// A pivot that is not a positive normal number is replaced by 1 without a branch, and off the chain
// (the estimate is taken from the pivot as it comes, the test runs beside it); the first such column
// is remembered in bad_col (-1: none) and reported after the block.
template <int K>
struct Chol32Step {
    static __device__ __forceinline__ void run(float (&d)[32], float piv, int lane, float *dinv, float *cv, int &bad_col) {
        // 1/sqrt(piv): hardware estimate plus one Newton step (to about one ulp)
        float rinv;
        asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(rinv) : "f"(piv));
        rinv = rinv * fmaf(-0.5f * piv, rinv * rinv, 1.5f);
        const bool bad = !(piv >= 1.17549435e-38f) || !(piv < INFINITY);
        bad_col = (bad && bad_col < 0) ? K : bad_col;
        piv = bad ? 1.f : piv;
        rinv = bad ? 1.f : rinv;
        const float c = lane < K ? d[K] * rinv : 0.f;
        d[K] = lane < K ? c : (lane == K ? piv * rinv : 0.f);
        if (lane == K) dinv[K] = rinv;
        float next = 0.f;
        if (K > 0) {
            next = __shfl_sync(0xffffffffu, fmaf(-c, c, d[K - 1]), K - 1);
            float *buf = cv + 32 * (K & 1);
            buf[lane] = c;
            __syncwarp();
#pragma unroll
            for (int j4 = (K - 1) / 4; j4 >= 0; --j4) {
                const float4 cj = *reinterpret_cast<const float4 *>(buf + 4 * j4);
                if (4 * j4 + 3 < K) d[4 * j4 + 3] = fmaf(-c, cj.w, d[4 * j4 + 3]);
                if (4 * j4 + 2 < K) d[4 * j4 + 2] = fmaf(-c, cj.z, d[4 * j4 + 2]);
                if (4 * j4 + 1 < K) d[4 * j4 + 1] = fmaf(-c, cj.y, d[4 * j4 + 1]);
                if (4 * j4 + 0 < K) d[4 * j4 + 0] = fmaf(-c, cj.x, d[4 * j4 + 0]);
            }
        }
        Chol32Step<K - 1>::run(d, next, lane, dinv, cv, bad_col);
    }
};
template <>
struct Chol32Step<-1> {
    static __device__ __forceinline__ void run(float (&)[32], float, int, float *, float *, int &) {}
};

// One column step (from 31 down to 0) of the inversion of a 32 x 32 upper triangular block held in
// shared memory as its transpose (Rt[k][i] = R[i][k], leading dimension FP_LD): lane = column of the
// inverse, y = that column, dinv = reciprocal diagonal of R.
template <int K>
struct InvColStep {
    static __device__ __forceinline__ void run(float (&y)[32], const float *Rt, const float *dinv) {
        const float x = y[K] * dinv[K];
        y[K] = x;
        const float *col = Rt + K * FP_LD;
#pragma unroll
        for (int j4 = 0; j4 < (K + 3) / 4; ++j4) {
            const float4 r = *reinterpret_cast<const float4 *>(col + 4 * j4);
            if (4 * j4 + 0 < K) y[4 * j4 + 0] = fmaf(-x, r.x, y[4 * j4 + 0]);
            if (4 * j4 + 1 < K) y[4 * j4 + 1] = fmaf(-x, r.y, y[4 * j4 + 1]);
            if (4 * j4 + 2 < K) y[4 * j4 + 2] = fmaf(-x, r.z, y[4 * j4 + 2]);
            if (4 * j4 + 3 < K) y[4 * j4 + 3] = fmaf(-x, r.w, y[4 * j4 + 3]);
        }
        InvColStep<K - 1>::run(y, Rt, dinv);
    }
};
template <>
struct InvColStep<-1> {
    static __device__ __forceinline__ void run(float (&)[32], const float *, const float *) {}
};

// C[0:rows, 0:o] -= X * Rt-columns:  C[r][j] -= sum_l Xt[l][r] * Rt[l][j]  with Xt (32 x rows) and Rt (32 x o)
// in shared memory, leading dimension FP_LD.  RT rows x 4 columns per thread, all threads of the CTA.
template <int RT>
__device__ __forceinline__ void slab_rank32_update(float (*C)[FP_LD], const float (*Xt)[FP_LD], const float (*Rt)[FP_LD],
                                                   int o, int tid, int rows) {
    const int tj = o / 4;
    for (int t = tid; t < (rows / RT) * tj; t += FP_THREADS) {
        const int ti = t / tj, j0 = 4 * (t - ti * tj);
        float acc[RT][4];
#pragma unroll
        for (int e = 0; e < RT; ++e)
#pragma unroll
            for (int f = 0; f < 4; ++f) acc[e][f] = 0.f;
#pragma unroll 8
        for (int l = 0; l < 32; ++l) {
            float xv[RT];
            if (RT == 2) {
                const float2 x2 = *reinterpret_cast<const float2 *>(&Xt[l][2 * ti]);
                xv[0] = x2.x; xv[RT - 1] = x2.y;
            } else {
                xv[0] = Xt[l][ti];
            }
            const float4 rv = *reinterpret_cast<const float4 *>(&Rt[l][j0]);
#pragma unroll
            for (int e = 0; e < RT; ++e) {
                acc[e][0] = fmaf(xv[e], rv.x, acc[e][0]); acc[e][1] = fmaf(xv[e], rv.y, acc[e][1]);
                acc[e][2] = fmaf(xv[e], rv.z, acc[e][2]); acc[e][3] = fmaf(xv[e], rv.w, acc[e][3]);
            }
        }
#pragma unroll
        for (int e = 0; e < RT; ++e) {
            float4 *cp = reinterpret_cast<float4 *>(&C[RT * ti + e][j0]);
            float4 v = *cp;
            v.x -= acc[e][0]; v.y -= acc[e][1]; v.z -= acc[e][2]; v.w -= acc[e][3];
            *cp = v;
        }
    }
}

__global__ void __launch_bounds__(FP_THREADS, 1) factor_panel_kernel(FactorPanelArgs a) {
    extern __shared__ __align__(16) float smem_f[];
    // S: the block as it is read, then R in the upper part and R^T in the lower part
    float (*S)[FP_LD] = reinterpret_cast<float (*)[FP_LD]>(smem_f);
    float (*At)[FP_LD] = reinterpret_cast<float (*)[FP_LD]>(smem_f + NB * FP_LD);         // step 2: a tile of panel rows
    float (*Pt)[FP_LD] = reinterpret_cast<float (*)[FP_LD]>(smem_f + 2 * NB * FP_LD);     // Pt[k][i]: 32 solved columns, transposed
    float *Yt = smem_f + 2 * NB * FP_LD + 32 * FP_LD;       // [4][32][FP_YLD]: Yt[c][l][j] = inv(R_cc)[j][l]
    float *dinv = Yt + 4 * 32 * FP_YLD;                     // [NB] 1 / R_jj
    float *cv = dinv + NB;                                  // 2 x 32: the scaled column of the running 32 x 32 step
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n, b0 = a.b0;
    const int nv = min(NB, n - b0);
    const bool vec = (n & 3) == 0 && (reinterpret_cast<uintptr_t>(a.H) & 15) == 0 && nv == NB;
    const int TR = a.tile_rows;
    const int r_begin = blockIdx.x * a.rows_per_cta;
    const int r_end = min(b0, r_begin + a.rows_per_cta);
    pdl_launch_dependents();
    pdl_wait();

    // the block, read along rows (all loads in flight before the first store); only j >= i is used
    if (vec) {
        float4 v[NB * NB / 4 / FP_THREADS];
#pragma unroll
        for (int it = 0; it < NB * NB / 4 / FP_THREADS; ++it) {
            const int idx = tid + it * FP_THREADS, i = idx >> 5, j4 = idx & 31;
            v[it] = *reinterpret_cast<const float4 *>(a.H + (int64_t)(b0 + i) * n + b0 + 4 * j4);
        }
        // the first tile of this CTA's slab follows asynchronously
        if (r_begin < r_end) {
            for (int idx = tid; idx < TR * (NB / 4); idx += FP_THREADS) {
                const int i = idx >> 5, j4 = idx & 31;
                const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&At[i][4 * j4]);
                const float *src = a.H + (int64_t)(r_begin + i) * n + b0 + 4 * j4;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
#pragma unroll
        for (int it = 0; it < NB * NB / 4 / FP_THREADS; ++it) {
            const int idx = tid + it * FP_THREADS, i = idx >> 5, j4 = idx & 31;
            *reinterpret_cast<float4 *>(&S[i][4 * j4]) = v[it];
        }
    } else {
        for (int i = warp; i < NB; i += FP_WARPS) {
            const float *src = a.H + (int64_t)(b0 + i) * n + b0;
            for (int j = lane; j < NB; j += 32) {
                float v = (i == j) ? 1.f : 0.f;
                if (i < nv && j < nv && j >= i) v = src[j];
                S[i][j] = v;
            }
        }
    }
    __syncthreads();

    // ---- step 1
    for (int sb = NB / 32 - 1; sb >= 0; --sb) {
        const int o = 32 * sb;
        if (warp == 0) {
            // 32 x 32 reverse Cholesky in registers, lane = row
            float d[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) d[j] = (j >= lane) ? S[o + lane][o + j] : S[o + j][o + lane];
            int bad_col = -1;
            Chol32Step<31>::run(d, __shfl_sync(0xffffffffu, d[31], 31), lane, dinv + o, cv, bad_col);
            if (bad_col >= 0 && lane == 0 && blockIdx.x == 0) record_status(a.hd, ST_NOT_SPD, b0 + o + bad_col);
            // R_ss to the upper part, its transpose to the lower part
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (j >= lane) { S[o + lane][o + j] = d[j]; S[o + j][o + lane] = d[j]; }
        }
        if (o == 0) break;
        __syncthreads();
        // rows above: x R_ss^T = S[i, sub], one thread per row; results go to the upper part,
        // to the lower part (transposed) and to Pt for the update
        if (tid < o) {
            const int i = tid;
            float x[32];
#pragma unroll
            for (int k = 0; k < 32; ++k) x[k] = S[i][o + k];
            solve_row<32>(x, &S[o][o], FP_LD, dinv + o);
#pragma unroll
            for (int k = 0; k < 32; ++k) { S[i][o + k] = x[k]; S[o + k][i] = x[k]; Pt[k][i] = x[k]; }
        }
        __syncthreads();
        // leading part: S[i][j] -= X[i] . X[j] for i <= j < o, 4 x 4 per thread; the tiles of the upper
        // triangle are numbered through a (q / 2) x (q + 1) rectangle so that the active threads are dense
        {
            const int q = o / 4;
            for (int t = tid; t < (q / 2) * (q + 1); t += FP_THREADS) {
                const int r = t / (q + 1), c = t - r * (q + 1);
                const int ti = c > r ? r : q - 1 - r, tj = c > r ? c - 1 : q - 1 - r + c;
                float acc[4][4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int f = 0; f < 4; ++f) acc[e][f] = 0.f;
#pragma unroll 8
                for (int k = 0; k < 32; ++k) {
                    const float4 ri = *reinterpret_cast<const float4 *>(&Pt[k][4 * ti]);
                    const float4 rj = *reinterpret_cast<const float4 *>(&Pt[k][4 * tj]);
                    const float av[4] = {ri.x, ri.y, ri.z, ri.w}, bv[4] = {rj.x, rj.y, rj.z, rj.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
#pragma unroll
                        for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(av[e], bv[f], acc[e][f]);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float4 *cp = reinterpret_cast<float4 *>(&S[4 * ti + e][4 * tj]);
                    float4 v = *cp;
                    v.x -= acc[e][0]; v.y -= acc[e][1]; v.z -= acc[e][2]; v.w -= acc[e][3];
                    *cp = v;
                }
            }
        }
        __syncthreads();
    }
    __syncthreads();

    // (the last CTA: the host adds one without a slab while there are SMs left)
    if (blockIdx.x == gridDim.x - 1)
        for (int idx = tid; idx < NB * NB; idx += FP_THREADS) {
            const int i = idx >> 7, j = idx & 127;
            a.Rdiag[idx] = j >= i ? S[i][j] : 0.f;
        }
    if (b0 == 0 || r_begin >= r_end) return;

    // the inverses of the four 32 x 32 diagonal sub-blocks (one warp each, lane = column)
    if (warp < NB / 32) {
        const int o = 32 * warp;
        float y[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) y[k] = (k == lane) ? 1.f : 0.f;
        InvColStep<31>::run(y, &S[o][o], dinv + o);
        float *dst = Yt + (warp * 32 + lane) * FP_YLD;
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4)
            *reinterpret_cast<float4 *>(dst + 4 * k4) = make_float4(y[4 * k4], y[4 * k4 + 1], y[4 * k4 + 2], y[4 * k4 + 3]);
    }

    // ---- step 2: rows [r_begin, r_end) of the panel in tiles of TR rows
    for (int r0 = r_begin; r0 < r_end; r0 += TR) {        // b0 and the slabs are multiples of TR
        if (vec) {
            if (r0 != r_begin) {
                for (int idx = tid; idx < TR * (NB / 4); idx += FP_THREADS) {
                    const int i = idx >> 5, j4 = idx & 31;
                    *reinterpret_cast<float4 *>(&At[i][4 * j4]) =
                        *reinterpret_cast<const float4 *>(a.H + (int64_t)(r0 + i) * n + b0 + 4 * j4);
                }
            } else {
                asm volatile("cp.async.wait_all;" ::: "memory");
            }
        } else {
            for (int i = warp; i < TR; i += FP_WARPS) {
                const float *src = a.H + (int64_t)(r0 + i) * n + b0;
                for (int k = lane; k < NB; k += 32) At[i][k] = k < nv ? src[k] : 0.f;
            }
        }
        __syncthreads();
        for (int sb = NB / 32 - 1; sb >= 0; --sb) {
            const int o = 32 * sb;
            // X = At[:, o : o + 32] * inv(R_ss)^T, a row and four columns per thread; to Pt (transposed)
            const float *Ys = Yt + sb * 32 * FP_YLD;
            for (int t = tid; t < TR * 8; t += FP_THREADS) {
                const int r = t >> 3, j0 = 4 * (t & 7);
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int l4 = 0; l4 < 8; ++l4) {
                    const float4 av = *reinterpret_cast<const float4 *>(&At[r][o + 4 * l4]);
                    const float al[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float4 yv = *reinterpret_cast<const float4 *>(Ys + (4 * l4 + e) * FP_YLD + j0);
                        acc[0] = fmaf(al[e], yv.x, acc[0]);
                        acc[1] = fmaf(al[e], yv.y, acc[1]);
                        acc[2] = fmaf(al[e], yv.z, acc[2]);
                        acc[3] = fmaf(al[e], yv.w, acc[3]);
                    }
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) Pt[j0 + e][r] = acc[e];
            }
            __syncthreads();
            // the solved columns back into the tile; columns to the left: At[r][j] -= sum_l X[r][l] R[j][o + l]
            for (int t = tid; t < TR * 8; t += FP_THREADS) {
                const int r = t >> 3, j0 = 4 * (t & 7);
                *reinterpret_cast<float4 *>(&At[r][o + j0]) = make_float4(Pt[j0][r], Pt[j0 + 1][r], Pt[j0 + 2][r], Pt[j0 + 3][r]);
            }
            if (o > 0) {
                const float (*Rt)[FP_LD] = reinterpret_cast<const float (*)[FP_LD]>(&S[o][0]);
                slab_rank32_update<2>(At, Pt, Rt, o, tid, TR);
            }
            __syncthreads();
        }
        // store the tile (and its TF32 parts)
#pragma unroll
        for (int it = 0; it < NB * NB / 4 / FP_THREADS; ++it) {
            const int idx = tid + it * FP_THREADS, i = idx >> 5, j4 = idx & 31;
            if (i >= TR) continue;
            const float4 v = *reinterpret_cast<const float4 *>(&At[i][4 * j4]);
            float *dst = a.H + (int64_t)(r0 + i) * n + b0 + 4 * j4;
            if (vec) {
                *reinterpret_cast<float4 *>(dst) = v;
            } else {
                if (4 * j4 + 0 < nv) dst[0] = v.x;
                if (4 * j4 + 1 < nv) dst[1] = v.y;
                if (4 * j4 + 2 < nv) dst[2] = v.z;
                if (4 * j4 + 3 < nv) dst[3] = v.w;
            }
            if (a.pan_hi && a.pan_f16) {
                const float sc = split_scale(__uint_as_float(a.hd->tc_amax[AMAX_PAN]));
                const float xs[4] = {sc * v.x, sc * v.y, sc * v.z, sc * v.w};
                __half2 hv[2], lv[2];
#pragma unroll
                for (int f = 0; f < 2; ++f) {
                    const __half h0 = __float2half_rn(xs[2 * f]), h1 = __float2half_rn(xs[2 * f + 1]);
                    hv[f] = __halves2half2(h0, h1);
                    lv[f] = __halves2half2(__float2half_rn(xs[2 * f] - __half2float(h0)),
                                           __float2half_rn(xs[2 * f + 1] - __half2float(h1)));
                }
                __half *ph = reinterpret_cast<__half *>(a.pan_hi) + (int64_t)(r0 + i) * a.pan_ld + a.pan_col0 + 4 * j4;
                __half *pl = reinterpret_cast<__half *>(a.pan_lo) + (int64_t)(r0 + i) * a.pan_ld + a.pan_col0 + 4 * j4;
                *reinterpret_cast<uint2 *>(ph) = make_uint2(*reinterpret_cast<uint32_t *>(&hv[0]), *reinterpret_cast<uint32_t *>(&hv[1]));
                *reinterpret_cast<uint2 *>(pl) = make_uint2(*reinterpret_cast<uint32_t *>(&lv[0]), *reinterpret_cast<uint32_t *>(&lv[1]));
            } else if (a.pan_hi) {
                const float xs[4] = {v.x, v.y, v.z, v.w};
                float hv[4], lv[4];
#pragma unroll
                for (int f = 0; f < 4; ++f) { hv[f] = tf32_rn(xs[f]); lv[f] = tf32_rn(xs[f] - hv[f]); }
                *reinterpret_cast<float4 *>(a.pan_hi + (int64_t)(r0 + i) * NB + 4 * j4) = make_float4(hv[0], hv[1], hv[2], hv[3]);
                *reinterpret_cast<float4 *>(a.pan_lo + (int64_t)(r0 + i) * NB + 4 * j4) = make_float4(lv[0], lv[1], lv[2], lv[3]);
            }
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------
// Inverts every NB x NB diagonal factor R_pp (one CTA each) and stores the inverse on the
// diagonal of H (strict lower part of the block zero): the starting point of U = R^-1.
// 32 x 32 diagonal sub-blocks by back substitution (one warp each, lane = column), then
// X12 = -X11 (R12 X22) for 32 -> 64 -> 128.
// ---------------------------------------------------------------------------
constexpr int ID_THREADS = 512;
constexpr int ID_LD = NB + 1;
constexpr size_t ID_SMEM = (2 * NB * ID_LD + 2 * 32 * 33) * sizeof(float);

__global__ void __launch_bounds__(ID_THREADS, 1) invert_diag_blocks_kernel(float *H, int n, const float *Rdiag) {
    extern __shared__ __align__(16) float smem_f[];
    float (*S)[ID_LD] = reinterpret_cast<float (*)[ID_LD]>(smem_f);
    float (*X)[ID_LD] = reinterpret_cast<float (*)[ID_LD]>(smem_f + NB * ID_LD);
    float (*T32)[32][33] = reinterpret_cast<float (*)[32][33]>(smem_f + 2 * NB * ID_LD);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b0 = blockIdx.x * NB;
    const float *src = Rdiag + (int64_t)blockIdx.x * NB * NB;
    for (int idx = tid; idx < NB * NB; idx += ID_THREADS) {
        S[idx >> 7][idx & 127] = src[idx];
        X[idx >> 7][idx & 127] = 0.f;
    }
    __syncthreads();
    if (warp < NB / 32) {
        const int o = 32 * warp;
        float x[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) x[i] = (i == lane) ? 1.f : 0.f;
#pragma unroll
        for (int i = 31; i >= 0; --i) {
            x[i] = x[i] / S[o + i][o + i];
#pragma unroll
            for (int i2 = 0; i2 < i; ++i2) x[i2] = fmaf(-S[o + i2][o + i], x[i], x[i2]);
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) X[o + i][o + lane] = x[i];
    }
    __syncthreads();
    // (the triangular operands carry explicit zeros, so full-length sums are exact)
    for (int idx = tid; idx < 2 * 1024; idx += ID_THREADS) {
        const int pr = idx >> 10, i = (idx >> 5) & 31, j = idx & 31;
        const int oa = 64 * pr, oc = oa + 32;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
        for (int k = 0; k < 32; k += 2) {
            s0 = fmaf(S[oa + i][oc + k], X[oc + k][oc + j], s0);
            s1 = fmaf(S[oa + i][oc + k + 1], X[oc + k + 1][oc + j], s1);
        }
        T32[pr][i][j] = s0 + s1;
    }
    __syncthreads();
    for (int idx = tid; idx < 2 * 1024; idx += ID_THREADS) {
        const int pr = idx >> 10, i = (idx >> 5) & 31, j = idx & 31;
        const int oa = 64 * pr, oc = oa + 32;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
        for (int k = 0; k < 32; k += 2) {
            s0 = fmaf(X[oa + i][oa + k], T32[pr][k][j], s0);
            s1 = fmaf(X[oa + i][oa + k + 1], T32[pr][k + 1][j], s1);
        }
        X[oa + i][oc + j] = -(s0 + s1);
    }
    __syncthreads();
    // T64 = R[0:64, 64:128] X[64:128, 64:128], parked in the (still unused) lower-left of X
    for (int idx = tid; idx < 64 * 64; idx += ID_THREADS) {
        const int i = idx >> 6, j = idx & 63;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 4
        for (int k = 0; k < 64; k += 4) {
            s0 = fmaf(S[i][64 + k], X[64 + k][64 + j], s0);
            s1 = fmaf(S[i][64 + k + 1], X[64 + k + 1][64 + j], s1);
            s2 = fmaf(S[i][64 + k + 2], X[64 + k + 2][64 + j], s2);
            s3 = fmaf(S[i][64 + k + 3], X[64 + k + 3][64 + j], s3);
        }
        X[64 + i][j] = (s0 + s1) + (s2 + s3);
    }
    __syncthreads();
    for (int idx = tid; idx < 64 * 64; idx += ID_THREADS) {
        const int i = idx >> 6, j = idx & 63;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 4
        for (int k = 0; k < 64; k += 4) {
            s0 = fmaf(X[i][k], X[64 + k][j], s0);
            s1 = fmaf(X[i][k + 1], X[64 + k + 1][j], s1);
            s2 = fmaf(X[i][k + 2], X[64 + k + 2][j], s2);
            s3 = fmaf(X[i][k + 3], X[64 + k + 3][j], s3);
        }
        X[i][64 + j] = -((s0 + s1) + (s2 + s3));
    }
    __syncthreads();
    for (int idx = tid; idx < NB * NB; idx += ID_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        if (b0 + i < n && b0 + j < n) H[(int64_t)(b0 + i) * n + (b0 + j)] = (j >= i) ? X[i][j] : 0.f;
    }
}

// ---------------------------------------------------------------------------
// quant(.)  -- min/max grid that contains zero, round half to even.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void make_grid(float lo, float hi, float amax, int bits, int sym,
                                          float &scale, float &zero) {
    if (sym) {
        float a = (amax == 0.f) ? 1.f : amax;
        scale = a / (float)((1 << (bits - 1)) - 1);
        zero = (float)(1 << (bits - 1));
    } else {
        lo = fminf(lo, 0.f);
        hi = fmaxf(hi, 0.f);
        if (hi == lo) { scale = 1.f; zero = 0.f; }
        else {
            scale = (hi - lo) / (float)((1 << bits) - 1);
            zero = rintf(-lo / scale);
        }
    }
}

// Clipping-range search of a grid by least squared rounding error (experimental setup of Section 5):
// candidate k of `steps` shrinks the min/max range by p_k = 1 - k (1 - min_ratio) / steps;
// the candidate with the least squared rounding error of the group's weights wins, the widest one on ties.
__device__ __forceinline__ float clip_ratio(int k, int steps, float min_ratio) {
    return 1.f - (float)k * ((1.f - min_ratio) / (float)steps);
}
__device__ __forceinline__ float rounding_error_sq(float w, float scale, float zero, float maxq) {
    const float cq = fminf(fmaxf(rintf(w * (1.f / scale)) + zero, 0.f), maxq);
    const float d = scale * (cq - zero) - w;
    return d * d;
}

// Per-channel grids from the original rows (dead inputs count as zero weights).
__global__ void __launch_bounds__(256) row_grid_kernel(const float *W, int64_t ldw, int m, int n,
                                                       const uint8_t *dead, int bits, int sym,
                                                       float *scales, float *zeros, int clip_steps, float clip_min) {
    int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    if (row >= m) return;
    const float *w = W + (int64_t)row * ldw;
    float lo = 0.f, hi = 0.f, am = 0.f;
    for (int c = lane; c < n; c += 32) {
        float v = dead[c] ? 0.f : w[c];
        lo = fminf(lo, v); hi = fmaxf(hi, v); am = fmaxf(am, fabsf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    }
    float s, z;
    make_grid(lo, hi, am, bits, sym, s, z);
    if (clip_steps > 0) {
        const float maxq = (float)((1 << bits) - 1);
        float best = INFINITY;
        for (int k = 0; k < clip_steps; ++k) {
            const float p = clip_ratio(k, clip_steps, clip_min);
            float sk, zk;
            make_grid(p * lo, p * hi, p * am, bits, sym, sk, zk);
            float err = 0.f;
            for (int c = lane; c < n; c += 32) err += rounding_error_sq(dead[c] ? 0.f : w[c], sk, zk, maxq);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
            if (err < best) { best = err; s = sk; z = zk; }
        }
    }
    if (lane == 0) { scales[row] = s; zeros[row] = z; }
}

// Static groups: one grid per output channel and per group of `group` consecutive columns of W in the
// caller's column order, from the original weights (dead inputs count as zero weights).  One warp per
// (row, group); W float32 or bf16.
template <typename T>
__global__ void __launch_bounds__(256) static_group_grid_kernel(const T *W, int64_t ldw, int m, int n, int group, int G,
                                                                const uint8_t *dead, int bits, int sym, float *scales,
                                                                float *zeros, int clip_steps, float clip_min) {
    const int64_t wid = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= (int64_t)m * G) return;
    const int row = (int)(wid / G), g = (int)(wid - (int64_t)row * G);
    const T *w = W + (int64_t)row * ldw;
    const int c0 = g * group, c1 = min(n, c0 + group);
    float lo = 0.f, hi = 0.f, am = 0.f;
    for (int c = c0 + lane; c < c1; c += 32) {
        const float v = dead[c] ? 0.f : (float)w[c];
        lo = fminf(lo, v); hi = fmaxf(hi, v); am = fmaxf(am, fabsf(v));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    }
    float s, z;
    make_grid(lo, hi, am, bits, sym, s, z);
    if (clip_steps > 0) {
        const float maxq = (float)((1 << bits) - 1);
        float best = INFINITY;
        for (int k = 0; k < clip_steps; ++k) {
            const float p = clip_ratio(k, clip_steps, clip_min);
            float sk, zk;
            make_grid(p * lo, p * hi, p * am, bits, sym, sk, zk);
            float err = 0.f;
            for (int c = c0 + lane; c < c1; c += 32) err += rounding_error_sq(dead[c] ? 0.f : (float)w[c], sk, zk, maxq);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
            if (err < best) { best = err; s = sk; z = zk; }
        }
    }
    if (lane == 0) { scales[(int64_t)row * G + g] = s; zeros[(int64_t)row * G + g] = z; }
}

// ---------------------------------------------------------------------------
// Column loop over one lazy-batch block [i0, i0 + bw) (Algorithm 1, inner
// loop).  One warp per weight row; the row's block lives in registers (lane
// owns columns lane, lane + 32, ...), the B x B diagonal tiles of U and P live
// in shared memory.  Outputs: codes, dequantized columns (in place in W),
// -Err and the pre-quantization columns (for the trailing update), group grids.
// ---------------------------------------------------------------------------
struct ColumnLoopArgs {
    float *W; int64_t ldw; int m, n;
    const float *U, *P;        // n x n, ld n
    const uint8_t *dead;
    int i0, bw;                // block start, valid width (<= 32 * T)
    int bits, group, sym;
    uint8_t *codes;            // m x n
    float *scales, *zeros;     // m x G
    int G;
    float *EW;                 // m x (2 * 32 * T): [-Err | Wpre]
    int ew_ld, ew_pre;         // column_block_kernel: row pitch of EW / EW_lo and the offset of Wpre in a row (2B and B
                               //   for the layout above; a block's slice of a wider [-Err | Wpre] otherwise)
    float *EW_lo;              // nullptr, or: EW receives the TF32 value of each entry and EW_lo the remainder
    // FP16 operand for the tensor-core update (column_block_kernel only; EW_lo is null then), or nullptr:
    // row i of [-Err | rho * Wpre] times a power of two s_i, as fp16 hi / lo parts, m x (2 * block) each;
    // row_inv[i] = 1 / s_i.  rho = scale of U^T / scale of P^T (from the two recorded maxima) lets the two
    // halves of the B operand keep scales of their own.
    __half *EW16_hi, *EW16_lo;
    float *row_inv;
    const unsigned *amax_u, *amax_p;
    StateHeader *hd;
    float err_scale, asym_scale;   // 1 or 0: switches of the two terms of the weight update (ablation)
    const int *perm;               // nullptr, or: working column c is original column perm[c] (codes go there)
    int clip_steps; float clip_min; // clipping-range search of the group grids (0: plain min/max)
    int static_groups;             // column_loop_kernel: scales / zeros hold ready grids per group of ORIGINAL columns
                                   //   (static_group_grid_kernel); column c uses group (perm ? perm[c] : c) / group
};

template <int T>
__global__ void __launch_bounds__(1024) column_loop_kernel(ColumnLoopArgs a) {
    constexpr int BW = 32 * T;
    extern __shared__ float smem_f[];
    float (*Us)[BW] = reinterpret_cast<float (*)[BW]>(smem_f);
    float (*Ps)[BW] = reinterpret_cast<float (*)[BW]>(smem_f + BW * BW);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nwarps = blockDim.x >> 5;
    const int n = a.n, i0 = a.i0, bw = a.bw;

    for (int e = tid; e < BW * BW; e += blockDim.x) {
        int r = e / BW, c = e % BW;
        float u = 0.f, p = 0.f;
        if (r < bw && c < bw && c >= r) {
            int64_t off = (int64_t)(i0 + r) * n + (i0 + c);
            u = a.U[off];
            p = a.P[off];
        }
        Us[r][c] = u; Ps[r][c] = p;
    }
    __syncthreads();

    const int row = blockIdx.x * nwarps + warp;
    if (row >= a.m) return;
    float *wrow = a.W + (int64_t)row * a.ldw + i0;

    float w[T], nerr[T], pre[T];
    int code[T];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        int c = lane + 32 * t;
        float v = 0.f;
        if (c < bw && !a.dead[i0 + c]) v = wrow[c];
        w[t] = v; nerr[t] = 0.f; pre[t] = 0.f; code[t] = 0;
        // reported from the value that was read: the clamp of the quantizer would absorb a NaN or Inf
        if (!isfinite(v)) record_status(a.hd, ST_NONFINITE, row);
    }

    const float maxq = (float)((1 << a.bits) - 1);
    float scale = 1.f, zero = 0.f;
    if (a.group <= 0) { scale = a.scales[row]; zero = a.zeros[row]; }

#pragma unroll
    for (int t = 0; t < T; ++t) {
        for (int jj = 0; jj < 32; ++jj) {
            const int j = t * 32 + jj;
            if (j >= bw) break;
            if (a.static_groups) {
                const int cj = a.perm ? a.perm[i0 + j] : i0 + j;
                scale = a.scales[(int64_t)row * a.G + cj / a.group];
                zero = a.zeros[(int64_t)row * a.G + cj / a.group];
            } else if (a.group > 0 && ((i0 + j) % a.group) == 0) {
                // grid of the group that starts here, from the current values
                const int gend = min(j + a.group, bw);
                float lo = 0.f, hi = 0.f, am = 0.f;
#pragma unroll
                for (int t2 = 0; t2 < T; ++t2) {
                    int c = lane + 32 * t2;
                    if (c >= j && c < gend) {
                        lo = fminf(lo, w[t2]); hi = fmaxf(hi, w[t2]); am = fmaxf(am, fabsf(w[t2]));
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
                    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
                    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
                }
                make_grid(lo, hi, am, a.bits, a.sym, scale, zero);
                if (a.clip_steps > 0) {
                    float best = INFINITY;
                    for (int k = 0; k < a.clip_steps; ++k) {
                        const float p = clip_ratio(k, a.clip_steps, a.clip_min);
                        float sk, zk;
                        make_grid(p * lo, p * hi, p * am, a.bits, a.sym, sk, zk);
                        float err = 0.f;
#pragma unroll
                        for (int t2 = 0; t2 < T; ++t2) {
                            int c = lane + 32 * t2;
                            if (c >= j && c < gend) err += rounding_error_sq(w[t2], sk, zk, maxq);
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) err += __shfl_xor_sync(0xffffffffu, err, o);
                        if (err < best) { best = err; scale = sk; zero = zk; }
                    }
                }
                if (lane == 0) {
                    int g = (i0 + j) / a.group;
                    a.scales[(int64_t)row * a.G + g] = scale;
                    a.zeros[(int64_t)row * a.G + g] = zero;
                }
            }
            const float wj = __shfl_sync(0xffffffffu, w[t], jj);
            float cq = fminf(fmaxf(rintf(wj * (1.f / scale)) + zero, 0.f), maxq);
            const float q = scale * (cq - zero);
            const float ne = a.err_scale * ((q - wj) * (1.f / Us[j][j]));   // -(w - q) / U_jj
            const float wp = a.asym_scale * wj;
            if (lane == jj) { w[t] = q; nerr[t] = ne; pre[t] = wp; code[t] = (int)cq; }
#pragma unroll
            for (int t2 = 0; t2 < T; ++t2) {
                if (t2 < t) continue;
                int c = lane + 32 * t2;
                if (c > j) w[t2] = fmaf(wp, Ps[j][c], fmaf(ne, Us[j][c], w[t2]));
            }
        }
    }

    bool bad = false;
    // fp16-split handles (row_inv set): Wpre is stored times rho = scale of U^T / scale of P^T, like
    // column_block_kernel does, so that the two halves of the update's B operand keep scales of their own
    float rho = 1.f;
    if (a.row_inv) {
        const float ap = __uint_as_float(*a.amax_p);
        rho = ap > 0.f ? split_scale(__uint_as_float(*a.amax_u)) / split_scale(ap) : 0.f;
    }
    float *ew = a.EW + (int64_t)row * (2 * BW);
    float *ewl = a.EW_lo ? a.EW_lo + (int64_t)row * (2 * BW) : nullptr;
    uint8_t *crow = a.codes + (int64_t)row * n + i0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        int c = lane + 32 * t;
        if (ewl) {
            const float eh = tf32_rn(nerr[t]), ph = tf32_rn(pre[t]);
            ew[c] = eh; ewl[c] = tf32_rn(nerr[t] - eh);
            ew[BW + c] = ph; ewl[BW + c] = tf32_rn(pre[t] - ph);
        } else {
            ew[c] = nerr[t];
            ew[BW + c] = rho * pre[t];
        }
        if (c < bw) {
            wrow[c] = w[t];
            if (a.perm) a.codes[(int64_t)row * n + a.perm[i0 + c]] = (uint8_t)code[t];
            else crow[c] = (uint8_t)code[t];
            bad |= !isfinite(w[t]);
        }
    }
    if (bad) record_status(a.hd, ST_NONFINITE, row);
}

// ---------------------------------------------------------------------------
// Column loop over one full lazy-batch block [i0, i0 + B), B in {32, 64, 128}, for grids per
// output channel or per group of a multiple of 32 columns.  One CTA owns `rows` weight rows
// (a multiple of 32); their block lives in shared memory.  The block is processed 32 columns
// at a time:
//   - LANES threads per row (4 for 32 rows per CTA, 2 for 64, 1 beyond) take the 32 columns into
//     registers, 32 / LANES consecutive columns each, and run the sequential part (quantize column
//     k, scaled error, rank-1 update of the later columns of the 32): the lane that holds column k
//     quantizes it and passes the scaled error and the pre-quantization value to the row's other
//     lanes by shuffles, every lane updates its own later columns from the rows k of U and P in
//     shared memory.  The dependent chain of a column is then the quantizer plus one update, not
//     the up to 31 updates of one thread (154 cycles per column with one thread per row);
//   - all threads then apply the 32 columns' errors and pre-quantization values to the rest
//     of the block, a (rows x 64) x (64 x rest) product out of shared memory.
// Same outputs as column_loop_kernel.
// ---------------------------------------------------------------------------
constexpr int CB_THREADS = 256;
constexpr int CB_LD = 128 + 4;

__host__ __device__ inline size_t column_block_smem(int rows) {
    // the block, two buffers of 32 rows of U and P, [-Err | Wpre] of 32 columns transposed, two sets of 32
    // reciprocal pivots, and per row: the chosen clipping candidate and the largest operand magnitude
    return ((size_t)rows * CB_LD + 2 * 2 * 32 * CB_LD + 64 * (rows + 4) + 2 * 32 + 2 * rows) * sizeof(float);
}
__host__ __device__ inline int column_block_lanes(int rows) { return rows <= 32 ? 4 : (rows <= 64 ? 2 : 1); }

// Round to nearest, ties to even, for a value that is clamped to [0, 255] afterwards: adding and
// subtracting 1.5 * 2^23 rounds exactly like rintf wherever |v| < 2^22 and leaves larger values large
// (the clamp decides those), in two additions instead of a trip through the conversion unit, which
// was 30 of the 154 cycles of a column step.
__device__ __forceinline__ float round_for_clamp(float v) {
    const float magic = 12582912.f;
    return __fsub_rn(__fadd_rn(v, magic), magic);
}

// Step K of the sequential part for one row held by LANES lanes (lane `sub` of the row holds columns
// sub * CPL .. + CPL - 1 of the 32 in x).  The arithmetic of every column is that of a single thread per
// row: the results do not depend on LANES.
template <int LANES, int K>
struct QuantStep {
    static constexpr int CPL = 32 / LANES;
    static __device__ __forceinline__ void run(float (&x)[CPL], float (&nerr)[CPL], float (&pre)[CPL], uint32_t (&code)[CPL / 4],
                                               int sub, const float *Us, const float *Ps, const float *udinv,
                                               float scale, float inv_scale, float zero, float maxq, float err_scale,
                                               float asym_scale) {
        constexpr int OWNER = K / CPL, KK = K % CPL;
        // Straight-line code for all lanes (no divergent branches, so that the loads of U and P for the next
        // steps can move ahead of this step's arithmetic): every lane quantizes its own column KK, the owner's
        // result is the one that is kept and passed on.
        const bool own = LANES == 1 || sub == OWNER;
        const float w0 = x[KK];
        // w / scale as w * (1 / scale): one rounding more (about 1e-7 of a step, far inside the tie band)
        // for a much shorter dependent chain
        const float cq = fminf(fmaxf(round_for_clamp(w0 * inv_scale) + zero, 0.f), maxq);
        const float q = scale * (cq - zero);
        float ne = err_scale * ((q - w0) * udinv[K]);           // -(w - q) / U_kk
        float w = asym_scale * w0;
        if (own) { x[KK] = q; nerr[KK] = ne; pre[KK] = w; code[KK >> 2] |= (uint32_t)cq << (8 * (KK & 3)); }
        if (LANES > 1) {
            ne = __shfl_sync(0xffffffffu, ne, OWNER, LANES);
            w = __shfl_sync(0xffffffffu, w, OWNER, LANES);
        }
        // this lane's columns beyond K
        const float *ur = Us + K * CB_LD + sub * CPL, *pr = Ps + K * CB_LD + sub * CPL;
#pragma unroll
        for (int j4 = 0; j4 < CPL / 4; ++j4) {
            // (compile-time skip of the quads that no lane needs any more)
            if ((LANES - 1) * CPL + 4 * j4 + 3 <= K) continue;
            const float4 u = *reinterpret_cast<const float4 *>(ur + 4 * j4);
            const float4 p = *reinterpret_cast<const float4 *>(pr + 4 * j4);
            const int c0 = sub * CPL + 4 * j4;
            const float y0 = fmaf(w, p.x, fmaf(ne, u.x, x[4 * j4 + 0]));
            const float y1 = fmaf(w, p.y, fmaf(ne, u.y, x[4 * j4 + 1]));
            const float y2 = fmaf(w, p.z, fmaf(ne, u.z, x[4 * j4 + 2]));
            const float y3 = fmaf(w, p.w, fmaf(ne, u.w, x[4 * j4 + 3]));
            x[4 * j4 + 0] = c0 + 0 > K ? y0 : x[4 * j4 + 0];
            x[4 * j4 + 1] = c0 + 1 > K ? y1 : x[4 * j4 + 1];
            x[4 * j4 + 2] = c0 + 2 > K ? y2 : x[4 * j4 + 2];
            x[4 * j4 + 3] = c0 + 3 > K ? y3 : x[4 * j4 + 3];
        }
        QuantStep<LANES, K + 1>::run(x, nerr, pre, code, sub, Us, Ps, udinv, scale, inv_scale, zero, maxq, err_scale, asym_scale);
    }
};
template <int LANES>
struct QuantStep<LANES, 32> {
    static constexpr int CPL = 32 / LANES;
    static __device__ __forceinline__ void run(float (&)[CPL], float (&)[CPL], float (&)[CPL], uint32_t (&)[CPL / 4], int,
                                               const float *, const float *, const float *, float, float, float, float, float, float) {}
};

template <int LANES>
__global__ void __launch_bounds__(CB_THREADS, 1) column_block_kernel(ColumnLoopArgs a, int rows, int B) {
    extern __shared__ __align__(16) float smem_f[];
    float (*Wt)[CB_LD] = reinterpret_cast<float (*)[CB_LD]>(smem_f);                       // [rows][B]
    // rows o..o+31 of U and of P (block columns), two buffers: the next 32 rows are fetched while the
    // current 32 columns are quantized
    float (*UP)[CB_LD] = reinterpret_cast<float (*)[CB_LD]>(smem_f + rows * CB_LD);        // [2 buffers][U, P][32]
    float *St = smem_f + rows * CB_LD + 2 * 2 * 32 * CB_LD;                                // [64][rows + 4]: -Err, then Wpre
    const int sld = rows + 4;
    float *udinv2 = St + 64 * sld;                                                         // [2][32]
    int *bsel = reinterpret_cast<int *>(udinv2 + 2 * 32);                                  // [rows]: chosen clipping candidate
    float *rmax_s = reinterpret_cast<float *>(bsel + rows);                                // [rows]: largest |operand| of the row
    const int tid = threadIdx.x;
    const int n = a.n, i0 = a.i0;
    const int row0 = blockIdx.x * rows;
    const int nrows = min(rows, a.m - row0);
    const int bq = B / 4;
    // sequential part: thread tid < rows * LANES holds columns sub * CPL .. of row lrow (whole warps take part,
    // rows beyond the matrix run on zeros and store nothing)
    constexpr int CPL = 32 / LANES;
    const int lrow = tid / LANES, sub = tid % LANES;
    const bool chain = tid < rows * LANES;

    // the block of W (dead inputs read as zero), along rows; four loads in flight per thread
    for (int base = 0; base < rows * bq; base += 4 * CB_THREADS) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = base + u * CB_THREADS + tid;
            const int r = idx / bq, c4 = idx - r * bq;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (idx < rows * bq && r < nrows) {
                const float *src = a.W + (int64_t)(row0 + r) * a.ldw + i0 + 4 * c4;
                if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) v[u] = *reinterpret_cast<const float4 *>(src);
                else { v[u].x = src[0]; v[u].y = src[1]; v[u].z = src[2]; v[u].w = src[3]; }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = base + u * CB_THREADS + tid;
            if (idx >= rows * bq) continue;
            const int r = idx / bq, c4 = idx - r * bq;
            const uchar4 dd = *reinterpret_cast<const uchar4 *>(a.dead + i0 + 4 * c4);
            if (dd.x) v[u].x = 0.f;
            if (dd.y) v[u].y = 0.f;
            if (dd.z) v[u].z = 0.f;
            if (dd.w) v[u].w = 0.f;
            // a non-finite weight is reported from the value that was read: its code and dequantized value
            // come out finite (the clamp absorbs NaN and Inf), so the results alone would not show it
            if (r < nrows && (!isfinite(v[u].x) || !isfinite(v[u].y) || !isfinite(v[u].z) || !isfinite(v[u].w)))
                record_status(a.hd, ST_NONFINITE, row0 + r);
            *reinterpret_cast<float4 *>(&Wt[r][4 * c4]) = v[u];
        }
    }

    const float maxq = (float)((1 << a.bits) - 1);
    float scale = 1.f, zero = 0.f;
    const bool owner = chain && lrow < nrows;
    const int row = row0 + lrow;
    if (a.group <= 0 && owner) { scale = a.scales[row]; zero = a.zeros[row]; }
    const bool f16 = a.EW16_hi != nullptr;
    float rho = 1.f, rmax = 0.f;
    if (f16) {
        const float ap = __uint_as_float(*a.amax_p);
        rho = ap > 0.f ? split_scale(__uint_as_float(*a.amax_u)) / split_scale(ap) : 0.f;
    }

    // rows [o, o + 32) of U and P of this block into buffer `buf`, by `nthr` threads starting at `t0`
    auto fetch_up = [&](int o, int buf, int t0, int nthr) {
        float (*Ub)[CB_LD] = UP + buf * 64;
        float (*Pb)[CB_LD] = Ub + 32;
        const int t = tid - t0;
        for (int idx = t; idx < 32 * bq; idx += nthr) {
            const int k = idx / bq, c4 = idx - k * bq;
            const int64_t off = (int64_t)(i0 + o + k) * n + i0 + 4 * c4;
            float4 u, p;
            if ((n & 3) == 0) {
                u = *reinterpret_cast<const float4 *>(a.U + off);
                p = *reinterpret_cast<const float4 *>(a.P + off);
            } else {
                u = make_float4(a.U[off], a.U[off + 1], a.U[off + 2], a.U[off + 3]);
                p = make_float4(a.P[off], a.P[off + 1], a.P[off + 2], a.P[off + 3]);
            }
            *reinterpret_cast<float4 *>(&Ub[k][4 * c4]) = u;
            *reinterpret_cast<float4 *>(&Pb[k][4 * c4]) = p;
        }
        if (t < 32) udinv2[buf * 32 + t] = 1.f / a.U[(int64_t)(i0 + o + t) * n + i0 + o + t];
    };
    fetch_up(0, 0, 0, CB_THREADS);

    for (int o = 0; o < B; o += 32) {
        const int buf = (o >> 5) & 1;
        float (*Us)[CB_LD] = UP + buf * 64;
        float (*Ps)[CB_LD] = Us + 32;
        const float *udinv = udinv2 + buf * 32;
        __syncthreads();        // the block is current; this buffer of U / P is loaded; St and the other buffer are free
        const bool group_start = a.group > 0 && ((i0 + o) % a.group) == 0;
        int best_k = 0;
        if (group_start && a.clip_steps > 0) {
            // clipping-range search, all threads: thread = (row, share of the candidates); the shares'
            // best (error, candidate) pairs meet in St, which is free until the columns are quantized
            const int ncg = CB_THREADS / rows;
            const int r = tid % rows, cgi = tid / rows;
            float *berr = St;
            int *bk = reinterpret_cast<int *>(St + CB_THREADS);
            if (cgi < ncg) {
                float lo = 0.f, hi = 0.f, am = 0.f;
                const int gend = min(o + a.group, B);
                for (int c = o; c < gend; ++c) {
                    const float v = Wt[r][c];
                    lo = fminf(lo, v); hi = fmaxf(hi, v); am = fmaxf(am, fabsf(v));
                }
                float best = INFINITY;
                int kb = 0;
                for (int k = cgi; k < a.clip_steps; k += ncg) {
                    const float p = clip_ratio(k, a.clip_steps, a.clip_min);
                    float sk, zk;
                    make_grid(p * lo, p * hi, p * am, a.bits, a.sym, sk, zk);
                    float err = 0.f;
                    for (int c = o; c < gend; ++c) err += rounding_error_sq(Wt[r][c], sk, zk, maxq);
                    if (err < best) { best = err; kb = k; }
                }
                berr[cgi * rows + r] = best;
                bk[cgi * rows + r] = kb;
            }
            __syncthreads();
            if (tid < rows) {
                float best = INFINITY;
                int kbest = 0;
                for (int c = 0; c < ncg; ++c) {
                    const float e = berr[c * rows + tid];
                    const int k = bk[c * rows + tid];
                    if (e < best || (e == best && k < kbest)) { best = e; kbest = k; }
                }
                bsel[tid] = kbest;
            }
            __syncthreads();
            if (chain) best_k = bsel[lrow];
        }
        if (tid >= CB_THREADS / 2 && o + 32 < B) fetch_up(o + 32, buf ^ 1, CB_THREADS / 2, CB_THREADS / 2);
        if (chain) {
            if (group_start) {
                // grid of the group that starts here, from the current values (the row's lanes share the scan)
                float lo = 0.f, hi = 0.f, am = 0.f;
                const int gend = min(o + a.group, B);
                for (int c = o + sub; c < gend; c += LANES) {
                    const float v = Wt[lrow][c];
                    lo = fminf(lo, v); hi = fmaxf(hi, v); am = fmaxf(am, fabsf(v));
                }
#pragma unroll
                for (int d = 1; d < LANES; d <<= 1) {
                    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
                    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
                    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, d));
                }
                const float p = a.clip_steps > 0 ? clip_ratio(best_k, a.clip_steps, a.clip_min) : 1.f;
                make_grid(p * lo, p * hi, p * am, a.bits, a.sym, scale, zero);
                if (owner && sub == 0) {
                    const int g = (i0 + o) / a.group;
                    a.scales[(int64_t)row * a.G + g] = scale;
                    a.zeros[(int64_t)row * a.G + g] = zero;
                }
            }
            float x[CPL], nerr[CPL], pre[CPL];
            uint32_t code[CPL / 4];
            const int c_lane = o + sub * CPL;                 // this lane's first column in the block
#pragma unroll
            for (int k4 = 0; k4 < CPL / 4; ++k4) {
                const float4 v = *reinterpret_cast<const float4 *>(&Wt[lrow][c_lane + 4 * k4]);
                x[4 * k4] = v.x; x[4 * k4 + 1] = v.y; x[4 * k4 + 2] = v.z; x[4 * k4 + 3] = v.w;
                code[k4] = 0u;
            }
            QuantStep<LANES, 0>::run(x, nerr, pre, code, sub, &Us[0][o], &Ps[0][o], udinv, scale, 1.f / scale, zero, maxq,
                                     a.err_scale, a.asym_scale);
            if (owner) {
                uint8_t *crow = a.codes + (int64_t)row * n + i0 + c_lane;
                if (a.perm) {
                    uint8_t *cbase = a.codes + (int64_t)row * n;
                    const int *pp = a.perm + i0 + c_lane;
#pragma unroll
                    for (int k = 0; k < CPL; ++k) cbase[pp[k]] = (uint8_t)(code[k >> 2] >> (8 * (k & 3)));
                } else if ((reinterpret_cast<uintptr_t>(crow) & (CPL >= 16 ? 15 : 7)) == 0) {
                    if constexpr (CPL == 32) {
                        *reinterpret_cast<uint4 *>(crow) = make_uint4(code[0], code[1], code[2], code[3]);
                        *reinterpret_cast<uint4 *>(crow + 16) = make_uint4(code[4], code[5], code[6], code[7]);
                    } else if constexpr (CPL == 16) {
                        *reinterpret_cast<uint4 *>(crow) = make_uint4(code[0], code[1], code[2], code[3]);
                    } else {
                        *reinterpret_cast<uint2 *>(crow) = make_uint2(code[0], code[1]);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < CPL; ++k) crow[k] = (uint8_t)(code[k >> 2] >> (8 * (k & 3)));
                }
            }
            float *ew = a.EW + (int64_t)row * a.ew_ld + c_lane;
            float *ewl = a.EW_lo ? a.EW_lo + (int64_t)row * a.ew_ld + c_lane : nullptr;
#pragma unroll
            for (int k4 = 0; k4 < CPL / 4; ++k4) {
                *reinterpret_cast<float4 *>(&Wt[lrow][c_lane + 4 * k4]) = make_float4(x[4 * k4], x[4 * k4 + 1], x[4 * k4 + 2], x[4 * k4 + 3]);
                float e4[4] = {nerr[4 * k4], nerr[4 * k4 + 1], nerr[4 * k4 + 2], nerr[4 * k4 + 3]};
                float p4[4] = {pre[4 * k4], pre[4 * k4 + 1], pre[4 * k4 + 2], pre[4 * k4 + 3]};
                if (f16) {
#pragma unroll
                    for (int f = 0; f < 4; ++f) {
                        p4[f] *= rho;
                        rmax = fmaxf(rmax, fmaxf(fabsf(e4[f]), fabsf(p4[f])));
                    }
                }
                if (!owner) continue;
                if (ewl) {
                    float el[4], pl[4];
#pragma unroll
                    for (int f = 0; f < 4; ++f) {
                        const float eh = tf32_rn(e4[f]), ph = tf32_rn(p4[f]);
                        el[f] = tf32_rn(e4[f] - eh); pl[f] = tf32_rn(p4[f] - ph);
                        e4[f] = eh; p4[f] = ph;
                    }
                    *reinterpret_cast<float4 *>(ewl + 4 * k4) = make_float4(el[0], el[1], el[2], el[3]);
                    *reinterpret_cast<float4 *>(ewl + a.ew_pre + 4 * k4) = make_float4(pl[0], pl[1], pl[2], pl[3]);
                }
                *reinterpret_cast<float4 *>(ew + 4 * k4) = make_float4(e4[0], e4[1], e4[2], e4[3]);
                *reinterpret_cast<float4 *>(ew + a.ew_pre + 4 * k4) = make_float4(p4[0], p4[1], p4[2], p4[3]);
            }
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                St[(sub * CPL + k) * sld + lrow] = nerr[k];
                St[(32 + sub * CPL + k) * sld + lrow] = pre[k];
            }
        }
        __syncthreads();
        // rest of the block: Wt[:, c] += sum_k (-Err)[:, k] U[o + k][c] + Wpre[:, k] P[o + k][c], c >= o + 32
        const int c_begin = o + 32;
        if (c_begin < B) {
            const int tr = rows / 4, tc = (B - c_begin) / 4;
            for (int t = tid; t < tr * tc; t += CB_THREADS) {
                const int tj = t / tr, ti = t - tj * tr;            // consecutive threads: consecutive row tiles
                const int c0 = c_begin + 4 * tj;
                float acc[4][4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
#pragma unroll
                    for (int f = 0; f < 4; ++f) acc[e][f] = 0.f;
#pragma unroll 4
                for (int k = 0; k < 64; ++k) {
                    const float4 av4 = *reinterpret_cast<const float4 *>(St + k * sld + 4 * ti);
                    const float4 bv4 = *reinterpret_cast<const float4 *>(k < 32 ? &Us[k][c0] : &Ps[k - 32][c0]);
                    const float av[4] = {av4.x, av4.y, av4.z, av4.w}, bv[4] = {bv4.x, bv4.y, bv4.z, bv4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e)
#pragma unroll
                        for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(av[e], bv[f], acc[e][f]);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float4 *cp = reinterpret_cast<float4 *>(&Wt[4 * ti + e][c0]);
                    float4 v = *cp;
                    v.x += acc[e][0]; v.y += acc[e][1]; v.z += acc[e][2]; v.w += acc[e][3];
                    *cp = v;
                }
            }
        }
    }
    if (f16 && chain) {
        // the row's largest operand magnitude, over its lanes
#pragma unroll
        for (int d = 1; d < LANES; d <<= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, d));
        if (sub == 0) rmax_s[lrow] = rmax;
    }
    __syncthreads();
    // dequantized block back to W
    for (int idx = tid; idx < nrows * bq; idx += CB_THREADS) {
        const int r = idx / bq, c4 = idx - r * bq;
        const float4 v = *reinterpret_cast<const float4 *>(&Wt[r][4 * c4]);
        const bool bad = !isfinite(v.x) || !isfinite(v.y) || !isfinite(v.z) || !isfinite(v.w);
        float *dst = a.W + (int64_t)(row0 + r) * a.ldw + i0 + 4 * c4;
        if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) *reinterpret_cast<float4 *>(dst) = v;
        else { dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w; }
        if (bad) record_status(a.hd, ST_NONFINITE, row0 + r);
    }
    if (f16) {
        // this CTA's rows of [-Err | rho * Wpre], scaled row by row into the fp16 range and split
        float *srow = St;                       // free since the last rank update
        if (tid < rows) {
            const bool live = tid < nrows;
            const float sc = live ? split_scale(rmax_s[tid]) : 1.f;
            srow[tid] = sc;
            if (live) a.row_inv[row0 + tid] = 1.f / sc;
        }
        __syncthreads();                        // (also: the rows written above are visible to the whole CTA)
        const int q = 2 * B / 4;
        for (int idx = tid; idx < nrows * q; idx += CB_THREADS) {
            const int r = idx / q, c4 = idx - r * q;
            const int64_t off = (int64_t)(row0 + r) * (2 * B) + 4 * c4;
            const int cc = 4 * c4;
            const float4 v = *reinterpret_cast<const float4 *>(a.EW + (int64_t)(row0 + r) * a.ew_ld +
                                                               (cc < B ? cc : a.ew_pre + cc - B));
            const float sc = srow[r];
            const float x[4] = {sc * v.x, sc * v.y, sc * v.z, sc * v.w};
            __half h[4], l[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) { h[e] = __float2half_rn(x[e]); l[e] = __float2half_rn(x[e] - __half2float(h[e])); }
            const __half2 h01 = __halves2half2(h[0], h[1]), h23 = __halves2half2(h[2], h[3]);
            const __half2 l01 = __halves2half2(l[0], l[1]), l23 = __halves2half2(l[2], l[3]);
            *reinterpret_cast<uint2 *>(a.EW16_hi + off) =
                make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
            *reinterpret_cast<uint2 *>(a.EW16_lo + off) =
                make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
        }
    }
}

// ---------------------------------------------------------------------------
// Row-by-row form of P (Eq. "unparallel"):  P[q, f] = scale * (D[q, f] U[f, f]^T) U[f, f],  f = q + 1 .. n - 1
// (L[f, f] of the paper is U[f, f]^T).  One CTA per row q, two passes over the trailing triangle of U:
//   v_a     = sum_{k >= a} D[q, k] U[a, k]      a in f   (a warp per a, along row a of U)
//   P[q, j] = sum_{q < a <= j} v_a U[a, j]      j in f   (a thread per j, coalesced across j)
// This is the form that Theorem 4.2 replaces by two matrix products; it is kept as the comparison of the
// latency discussion of Section 5, not as a path of the solve.  In place: row q of P overwrites row q of D.
// ---------------------------------------------------------------------------
constexpr int PR_THREADS = 1024;
__global__ void __launch_bounds__(PR_THREADS) p_rowwise_kernel(float *D, const float *U, int n, float scale) {
    extern __shared__ float pr_smem[];
    float *d = pr_smem, *v = pr_smem + n;
    const int q = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float *row = D + (int64_t)q * n;
    for (int c = tid; c < n; c += PR_THREADS) d[c] = c > q ? row[c] : 0.f;
    __syncthreads();
    for (int a = q + 1 + warp; a < n; a += PR_THREADS / 32) {
        const float *ur = U + (int64_t)a * n;
        float s = 0.f;
        for (int k = a + lane; k < n; k += 32) s = fmaf(d[k], ur[k], s);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) v[a] = s;
    }
    __syncthreads();
    for (int j = tid; j < n; j += PR_THREADS) {
        float s0 = 0.f, s1 = 0.f;
        int a = q + 1;
        for (; a + 1 <= j; a += 2) {
            s0 = fmaf(v[a], U[(int64_t)a * n + j], s0);
            s1 = fmaf(v[a + 1], U[(int64_t)(a + 1) * n + j], s1);
        }
        if (a <= j) s0 = fmaf(v[a], U[(int64_t)a * n + j], s0);
        row[j] = j > q ? scale * (s0 + s1) : 0.f;
    }
}

// ---------------------------------------------------------------------------
// act_order: columns sorted by decreasing diag(H).
// ---------------------------------------------------------------------------
// perm[rank] = q, rank = number of inputs that sort before q: larger value v (v = 1 for dead
// inputs, else H_qq / tokens), ties by smaller index (a stable descending sort).  O(n^2) compares.
__global__ void __launch_bounds__(256) rank_desc_kernel(const float *H, int n, float inv_tokens, const uint8_t *dead,
                                                        int *perm, uint8_t *dead_perm) {
    __shared__ float tile[256];
    const int q = blockIdx.x * 256 + threadIdx.x;
    const float vq = q < n ? (dead[q] ? 1.f : H[(int64_t)q * n + q] * inv_tokens) : 0.f;
    int rank = 0;
    for (int j0 = 0; j0 < n; j0 += 256) {
        const int j = j0 + threadIdx.x;
        tile[threadIdx.x] = j < n ? (dead[j] ? 1.f : H[(int64_t)j * n + j] * inv_tokens) : -1.f;
        __syncthreads();
        const int lim = min(256, n - j0);
        for (int t = 0; t < lim; ++t) {
            const float v = tile[t];
            rank += (v > vq) || (v == vq && j0 + t < q);
        }
        __syncthreads();
    }
    if (q < n) { perm[rank] = q; dead_perm[rank] = dead[q]; }
}

// dst[i][j] = src[perm[i]][perm[j]]; `symmetric_upper`: src holds a symmetric matrix in its upper
// triangle (element (a, b) is read at (min, max)) and only j >= i is written.
__global__ void __launch_bounds__(256) permute_matrix_kernel(const float *src, float *dst, int n, const int *perm,
                                                             int symmetric_upper) {
    const int j = blockIdx.x * 256 + threadIdx.x;
    const int i = blockIdx.y;
    if (j >= n) return;
    if (symmetric_upper && j < i) return;
    int a = perm[i], b = perm[j];
    if (symmetric_upper && a > b) { const int t = a; a = b; b = t; }
    dst[(int64_t)i * n + j] = src[(int64_t)a * n + b];
}

// dst[r][c] = src[r][perm[c]] as float32 (src float32 or bf16): the working copy of W in sorted order.
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const T *src, int64_t lds, float *dst, int64_t ldd, int m, int n,
                                                          const int *perm) {
    int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int64_t total = (int64_t)m * n;
    for (; idx < total; idx += (int64_t)gridDim.x * 256) {
        const int64_t r = idx / n, c = idx % n;
        dst[r * ldd + c] = (float)src[r * lds + perm[c]];
    }
}

// In place, one CTA per row: W[r][perm[c]] <- W[r][c] (back to the original column order); the
// row is staged in shared memory (n floats).
__global__ void __launch_bounds__(256) unpermute_rows_kernel(float *W, int64_t ldw, int n, const int *perm) {
    extern __shared__ float row_s[];
    float *w = W + (int64_t)blockIdx.x * ldw;
    for (int c = threadIdx.x; c < n; c += 256) row_s[c] = w[c];
    __syncthreads();
    for (int c = threadIdx.x; c < n; c += 256) w[perm[c]] = row_s[c];
}

__global__ void __launch_bounds__(256) bf16_to_f32_kernel(const __nv_bfloat16 *src, int64_t lds,
                                                          float *dst, int64_t ldd, int m, int n) {
    int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int64_t total = (int64_t)m * n;
    for (; idx < total; idx += (int64_t)gridDim.x * 256) {
        int64_t r = idx / n, c = idx % n;
        dst[r * ldd + c] = __bfloat162float(src[r * lds + c]);
    }
}

__global__ void __launch_bounds__(256) copy2d_kernel(const float *src, int64_t lds, float *dst,
                                                     int64_t ldd, int m, int n) {
    int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int64_t total = (int64_t)m * n;
    for (; idx < total; idx += (int64_t)gridDim.x * 256) {
        int64_t r = idx / n, c = idx % n;
        dst[r * ldd + c] = src[r * lds + c];
    }
}

}  // namespace gptaq
