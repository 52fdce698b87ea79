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
// Diagonal block of the reverse Cholesky  H_d = R R^T (R upper):  factor the
// NB x NB block in shared memory from its last row/column upwards, write R_pp
// back in place (lower part zero) and its inverse to Rinv (NB x NB, ld NB).
// Rows/columns beyond n are padded with the identity.
// ---------------------------------------------------------------------------
constexpr int NB = 128;
constexpr int DIAG_THREADS = 1024;
constexpr size_t DIAG_SMEM = 2 * NB * (NB + 1) * sizeof(float);

__global__ void __launch_bounds__(DIAG_THREADS) chol_diag_kernel(float *H, int n, int b0,
                                                                 float *Rinv, StateHeader *hd) {
    extern __shared__ float smem_f[];
    float (*S)[NB + 1] = reinterpret_cast<float (*)[NB + 1]>(smem_f);
    float (*X)[NB + 1] = reinterpret_cast<float (*)[NB + 1]>(smem_f + NB * (NB + 1));
    const int tid = threadIdx.x;
    const int tx = tid & 31, ty = tid >> 5;
    const int nv = min(NB, n - b0);

    for (int i = ty; i < NB; i += 32)
        for (int j = tx; j < NB; j += 32) {
            float v;
            if (i < nv && j < nv) {
                int a = min(i, j), b = max(i, j);
                v = H[(int64_t)(b0 + a) * n + (b0 + b)];
            } else {
                v = (i == j) ? 1.f : 0.f;
            }
            S[i][j] = v;
            X[i][j] = 0.f;
        }
    __syncthreads();

    for (int k = NB - 1; k >= 0; --k) {
        float piv = S[k][k];
        bool bad = !(piv > 0.f) || !isfinite(piv);
        if (bad) {
            if (tid == 0) record_status(hd, ST_NOT_SPD, b0 + k);
            piv = 1.f;
        }
        float r = sqrtf(piv);
        __syncthreads();
        if (tid < k) S[tid][k] = S[tid][k] / r;
        else if (tid == k) S[k][k] = r;
        __syncthreads();
        for (int i = ty; i < k; i += 32) {
            float rik = S[i][k];
            for (int j = tx; j < k; j += 32)
                if (j >= i) S[i][j] = fmaf(-rik, S[j][k], S[i][j]);
        }
        // the next iteration's pivot read is ordered by the sync below
        __syncthreads();
    }

    // X = R^-1 (upper): column j by back substitution, 8 lanes per column.
    {
        const int j = tid >> 3, l = tid & 7;
        for (int i = NB - 1; i >= 0; --i) {
            float part = 0.f;
            if (i < j)
                for (int s = i + 1 + l; s <= j; s += 8) part = fmaf(S[i][s], X[s][j], part);
            part += __shfl_xor_sync(0xffffffffu, part, 1);
            part += __shfl_xor_sync(0xffffffffu, part, 2);
            part += __shfl_xor_sync(0xffffffffu, part, 4);
            if (l == 0 && i <= j) X[i][j] = ((i == j ? 1.f : 0.f) - part) / S[i][i];
            __syncwarp();
        }
    }
    __syncthreads();

    for (int i = ty; i < NB; i += 32)
        for (int j = tx; j < NB; j += 32) {
            if (i < nv && j < nv) H[(int64_t)(b0 + i) * n + (b0 + j)] = (j >= i) ? S[i][j] : 0.f;
            Rinv[i * NB + j] = (j >= i) ? X[i][j] : 0.f;
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
