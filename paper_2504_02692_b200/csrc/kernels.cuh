// Small kernels of the GPTAQ layer solve: damping, the diagonal-block reverse
// Cholesky, the per-column quantize-and-propagate loop, and helpers.
#pragma once
#include <cuda_bf16.h>
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
    unsigned amax[2];    // bit patterns of max|X| and max|X~ - X| of the batch being converted
    int pad1[24];
};
static_assert(sizeof(StateHeader) == 128, "header size");

constexpr int ST_NOT_SPD = 4, ST_NONFINITE = 5, ST_TIMEOUT = 6;

// Round to the nearest TF32 value (10 explicit mantissa bits), kept in a float.
__device__ __forceinline__ float tf32_rn(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

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
    double s = 0.0;
    for (int q = threadIdx.x; q < n; q += 1024) {
        float d = H[(int64_t)q * n + q];
        if (!isfinite(d)) record_status(hd, ST_NONFINITE, q);
        bool dd = (d == 0.f);
        dead[q] = dd ? 1 : 0;
        s += dd ? 1.0 : (double)d * (double)inv_tokens;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int w = 512; w > 0; w >>= 1) {
        if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        hd->lambda = (float)((double)damp * red[0] / (double)n);
        hd->inv_tokens = inv_tokens;
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
//   1. factor the NB x NB diagonal block from its last row/column upwards and invert the
//      factor, both in shared memory (32-wide sub-blocks: one warp factors and inverts a
//      32 x 32 block in registers, all warps apply it);
//   2. rows above the block:  R[0:b0, blk] = A[0:b0, blk] * inv(R_pp)^T, written back in
//      place and, if asked for, as TF32 hi/lo parts for the tensor-core rank-NB update.
// Every CTA repeats step 1 (it is short and the other SMs would idle) and then takes row
// tiles of step 2; CTA 0 stores inv(R_pp).  R_pp itself is not stored: nothing reads it.
// Rows/columns beyond n are padded with the identity.
// ---------------------------------------------------------------------------
constexpr int NB = 128;
constexpr int FP_THREADS = 1024;
constexpr int FP_LD = NB + 4;
constexpr size_t FP_SMEM = (2 * NB * FP_LD + 32 + 2 * 32 * 33) * sizeof(float);

struct FactorPanelArgs {
    float *H; int n; int b0;
    float *Rinv;               // NB x NB (ld NB): inverse of the diagonal factor
    float *pan_hi, *pan_lo;    // nullptr, or [n][NB]: TF32 parts of the panel rows
    StateHeader *hd;
};

__global__ void __launch_bounds__(FP_THREADS, 1) factor_panel_kernel(FactorPanelArgs a) {
    extern __shared__ float smem_f[];
    float (*S)[FP_LD] = reinterpret_cast<float (*)[FP_LD]>(smem_f);
    float (*X)[FP_LD] = reinterpret_cast<float (*)[FP_LD]>(smem_f + NB * FP_LD);
    float *colbuf = smem_f + 2 * NB * FP_LD;
    float (*T32)[32][33] = reinterpret_cast<float (*)[32][33]>(colbuf + 32);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = a.n, b0 = a.b0;
    const int nv = min(NB, n - b0);

    for (int i = warp; i < NB; i += 32)
        for (int j = lane; j < NB; j += 32) {
            float v;
            if (i < nv && j < nv) {
                const int lo = min(i, j), hi = max(i, j);
                v = a.H[(int64_t)(b0 + lo) * n + (b0 + hi)];
            } else {
                v = (i == j) ? 1.f : 0.f;
            }
            S[i][j] = v;
            X[i][j] = 0.f;
        }
    __syncthreads();

    for (int sb = NB / 32 - 1; sb >= 0; --sb) {
        const int o = 32 * sb;
        if (warp == 0) {
            // ---- 32 x 32 reverse Cholesky, lane = row, then its inverse, lane = column
            float d[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) d[j] = S[o + lane][o + j];
#pragma unroll
            for (int k = 31; k >= 0; --k) {
                float piv = __shfl_sync(0xffffffffu, d[k], k);
                if (!(piv > 0.f) || !isfinite(piv)) {
                    if (lane == 0 && blockIdx.x == 0) record_status(a.hd, ST_NOT_SPD, b0 + o + k);
                    piv = 1.f;
                }
                const float r = sqrtf(piv);
                const float c = lane < k ? d[k] / r : 0.f;
                d[k] = lane < k ? c : (lane == k ? r : 0.f);
                colbuf[lane] = c;
                __syncwarp();
#pragma unroll
                for (int j = 0; j < k; ++j) d[j] = fmaf(-c, colbuf[j], d[j]);
                __syncwarp();
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) S[o + lane][o + j] = j >= lane ? d[j] : 0.f;
            __syncwarp();
            float x[32];
#pragma unroll
            for (int i = 31; i >= 0; --i) {
                float sum = (i == lane) ? 1.f : 0.f;
#pragma unroll
                for (int k = i + 1; k < 32; ++k) sum = fmaf(-S[o + i][o + k], x[k], sum);
                x[i] = i <= lane ? sum / S[o + i][o + i] : 0.f;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) X[o + i][o + lane] = x[i];
        }
        __syncthreads();
        // ---- rows above: R[i, sub] = S[i, sub] * inv(R_ss)^T   (one warp per row, in place)
        for (int i = warp; i < o; i += 32) {
            float acc = 0.f;
#pragma unroll 8
            for (int k = 0; k < 32; ++k) acc = fmaf(S[i][o + k], X[o + lane][o + k], acc);
            __syncwarp();
            S[i][o + lane] = acc;
        }
        __syncthreads();
        // ---- leading part: S[i][j] -= R[i, sub] . R[j, sub]  (kept symmetric)
        for (int idx = tid; idx < o * o; idx += FP_THREADS) {
            const int i = idx / o, j = idx - i * o;
            if (j < i) continue;
            float acc = 0.f;
#pragma unroll 8
            for (int k = 0; k < 32; ++k) acc = fmaf(S[i][o + k], S[j][o + k], acc);
            const float v = S[i][j] - acc;
            S[i][j] = v;
            S[j][i] = v;
        }
        __syncthreads();
    }

    // ---- off-diagonal blocks of X = R^-1:  X12 = -X11 (R12 X22), 32 -> 64 -> 128
    for (int idx = tid; idx < 2 * 1024; idx += FP_THREADS) {
        const int pr = idx >> 10, i = (idx >> 5) & 31, j = idx & 31;
        const int oa = 64 * pr, oc = oa + 32;
        float acc = 0.f;
        for (int k = 0; k <= j; ++k) acc = fmaf(S[oa + i][oc + k], X[oc + k][oc + j], acc);
        T32[pr][i][j] = acc;
    }
    __syncthreads();
    for (int idx = tid; idx < 2 * 1024; idx += FP_THREADS) {
        const int pr = idx >> 10, i = (idx >> 5) & 31, j = idx & 31;
        const int oa = 64 * pr, oc = oa + 32;
        float acc = 0.f;
        for (int k = i; k < 32; ++k) acc = fmaf(X[oa + i][oa + k], T32[pr][k][j], acc);
        X[oa + i][oc + j] = -acc;
    }
    __syncthreads();
    // T64 = R[0:64, 64:128] X[64:128, 64:128], parked in the (still unused) lower-left of X
    for (int idx = tid; idx < 64 * 64; idx += FP_THREADS) {
        const int i = idx >> 6, j = idx & 63;
        float acc = 0.f;
        for (int k = 0; k <= j; ++k) acc = fmaf(S[i][64 + k], X[64 + k][64 + j], acc);
        X[64 + i][j] = acc;
    }
    __syncthreads();
    for (int idx = tid; idx < 64 * 64; idx += FP_THREADS) {
        const int i = idx >> 6, j = idx & 63;
        float acc = 0.f;
        for (int k = i; k < 64; ++k) acc = fmaf(X[i][k], X[64 + k][j], acc);
        X[i][64 + j] = -acc;
    }
    __syncthreads();
    for (int idx = tid; idx < 64 * 64; idx += FP_THREADS) X[64 + (idx >> 6)][idx & 63] = 0.f;
    __syncthreads();
    if (blockIdx.x == 0)
        for (int idx = tid; idx < NB * NB; idx += FP_THREADS) a.Rinv[idx] = X[idx >> 7][idx & 127];
    if (b0 == 0) return;

    // ---- X <- X^T in place, so that a thread reads four consecutive columns of inv(R_pp)^T at once
    for (int idx = tid; idx < NB * NB; idx += FP_THREADS) {
        const int i = idx >> 7, j = idx & 127;
        if (j > i) { const float u = X[i][j]; X[i][j] = X[j][i]; X[j][i] = u; }
    }
    // (the first tile's load below ends with a barrier)

    const int ntiles = b0 / NB;              // b0 is a multiple of NB
    const int ty = tid >> 5, tx = tid & 31;  // rows 4 ty .. 4 ty + 3, columns 4 tx .. 4 tx + 3
    const bool vec = (n & 3) == 0 && (reinterpret_cast<uintptr_t>(a.H) & 15) == 0 && nv == NB;
    for (int rt = blockIdx.x; rt < ntiles; rt += gridDim.x) {
        const int r0 = rt * NB;
        __syncthreads();                     // previous tile's reads of S are done
        for (int i = warp; i < NB; i += 32) {
            const float *src = a.H + (int64_t)(r0 + i) * n + b0;
            for (int k = lane; k < NB; k += 32) S[i][k] = k < nv ? src[k] : 0.f;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
            for (int f = 0; f < 4; ++f) acc[e][f] = 0.f;
#pragma unroll 4
        for (int k = 0; k < NB; ++k) {
            const float4 b = *reinterpret_cast<const float4 *>(&X[k][4 * tx]);
            float av[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) av[e] = S[4 * ty + e][k];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                acc[e][0] = fmaf(av[e], b.x, acc[e][0]); acc[e][1] = fmaf(av[e], b.y, acc[e][1]);
                acc[e][2] = fmaf(av[e], b.z, acc[e][2]); acc[e][3] = fmaf(av[e], b.w, acc[e][3]);
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int row = r0 + 4 * ty + e;
            float *dst = a.H + (int64_t)row * n + b0 + 4 * tx;
            if (vec) {
                *reinterpret_cast<float4 *>(dst) = make_float4(acc[e][0], acc[e][1], acc[e][2], acc[e][3]);
            } else {
#pragma unroll
                for (int f = 0; f < 4; ++f) if (4 * tx + f < nv) dst[f] = acc[e][f];
            }
            if (a.pan_hi) {
                float hv[4], lv[4];
#pragma unroll
                for (int f = 0; f < 4; ++f) { hv[f] = tf32_rn(acc[e][f]); lv[f] = tf32_rn(acc[e][f] - hv[f]); }
                *reinterpret_cast<float4 *>(a.pan_hi + (int64_t)row * NB + 4 * tx) = make_float4(hv[0], hv[1], hv[2], hv[3]);
                *reinterpret_cast<float4 *>(a.pan_lo + (int64_t)row * NB + 4 * tx) = make_float4(lv[0], lv[1], lv[2], lv[3]);
            }
        }
    }
}

// Copies the inverted diagonal blocks (NB x NB each) onto the diagonal of H.
__global__ void __launch_bounds__(256) place_diag_inverse_kernel(float *H, int n, const float *Rinv) {
    int b0 = blockIdx.x * NB;
    const float *src = Rinv + (int64_t)blockIdx.x * NB * NB;
    for (int e = threadIdx.x; e < NB * NB; e += 256) {
        int i = e / NB, j = e % NB;
        if (b0 + i < n && b0 + j < n) H[(int64_t)(b0 + i) * n + (b0 + j)] = src[e];
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

// Per-channel grids from the original rows (dead inputs count as zero weights).
__global__ void __launch_bounds__(256) row_grid_kernel(const float *W, int64_t ldw, int m, int n,
                                                       const uint8_t *dead, int bits, int sym,
                                                       float *scales, float *zeros) {
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
    if (lane == 0) {
        float s, z;
        make_grid(lo, hi, am, bits, sym, s, z);
        scales[row] = s; zeros[row] = z;
    }
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
    float *EW_lo;              // nullptr, or: EW receives the TF32 value of each entry and EW_lo the remainder
    StateHeader *hd;
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
    }

    const float maxq = (float)((1 << a.bits) - 1);
    float scale = 1.f, zero = 0.f;
    if (a.group <= 0) { scale = a.scales[row]; zero = a.zeros[row]; }

#pragma unroll
    for (int t = 0; t < T; ++t) {
        for (int jj = 0; jj < 32; ++jj) {
            const int j = t * 32 + jj;
            if (j >= bw) break;
            if (a.group > 0 && ((i0 + j) % a.group) == 0) {
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
                if (lane == 0) {
                    int g = (i0 + j) / a.group;
                    a.scales[(int64_t)row * a.G + g] = scale;
                    a.zeros[(int64_t)row * a.G + g] = zero;
                }
            }
            const float wj = __shfl_sync(0xffffffffu, w[t], jj);
            float cq = fminf(fmaxf(rintf(wj / scale) + zero, 0.f), maxq);
            const float q = scale * (cq - zero);
            const float ne = (q - wj) / Us[j][j];   // -(w - q) / U_jj
            if (lane == jj) { w[t] = q; nerr[t] = ne; pre[t] = wj; code[t] = (int)cq; }
#pragma unroll
            for (int t2 = 0; t2 < T; ++t2) {
                if (t2 < t) continue;
                int c = lane + 32 * t2;
                if (c > j) w[t2] = fmaf(wj, Ps[j][c], fmaf(ne, Us[j][c], w[t2]));
            }
        }
    }

    bool bad = false;
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
            ew[BW + c] = pre[t];
        }
        if (c < bw) {
            wrow[c] = w[t];
            crow[c] = (uint8_t)code[t];
            bad |= !isfinite(w[t]);
        }
    }
    if (bad) record_status(a.hd, ST_NONFINITE, row);
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
