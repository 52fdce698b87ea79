// Generic fp32 tile GEMM on the plain FMA pipes.
//
// C(M x N) = alpha * A(M x K) * B(K x N) + beta * C, 128 x 128 x 16 tiles, 256
// threads, 8 x 8 outputs per thread, double-buffered shared memory.  Operands
// are described by strides so that one kernel serves every shape the solve
// needs: token-major Gram products (both operands K-slow), A * B^T panels,
// triangular products with per-tile K ranges, and the stacked [Err | Wpre] *
// [U ; P] trailing update.  It is the exact-fp32 reference path of the
// library: the tensor-core kernels replace it where a product is large, and it
// stays in use for ragged or small shapes.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gptaq {

// element (r, k) of an operand = p[r * rs + k * ks]   (r: row of A / column of B)
// k >= k_split reads p2[r * rs + (k - k_split) * ks] instead (stacked operand).
// If sub != nullptr the value is sub[...] - p[...] (same strides): used for X~ - X.
struct Operand {
    const float *p;
    int64_t rs, ks;
    const float *p2;
    int k_split;
    const float *sub;
};

enum GemmMode {
    GEMM_FULL = 0,
    GEMM_UPPER_TILES = 1,   // skip tiles that lie entirely below the diagonal
    GEMM_O = 2,             // C[i][a] = sum_{k >= a} ..., kept only for a > i (else 0); lower tiles skipped
    GEMM_P = 3,             // C[i][j] = sum_{i < k <= j} ..., strictly upper; lower tiles zero-filled
    GEMM_TRI_RIGHT = 4,     // B upper triangular: k <= j
    GEMM_TRI_LEFT = 5       // A upper triangular: k >= i
};

struct GemmProblem {
    Operand A, B;
    float *C;
    int64_t ldc;
    int M, N, K;
    float alpha, beta;
    int mode;
    // batching along blockIdx.z: every pointer advances by these element counts
    int64_t batchA, batchB, batchC;
    int batchM_last, batchN_last, batchK_last;  // dims of the last batch entry (ragged tail), 0 = same
    int nbatch;
};

constexpr int GBM = 128, GBN = 128, GBK = 16, GPAD = 4;

template <bool RC>   // RC: rows contiguous (rs == 1), else K contiguous (ks == 1)
__device__ __forceinline__ void gemm_load(const Operand &op, int row0, int k0, int R, int K,
                                          int tid, float (&v)[8]) {
    if (RC) {
        // thread: 4 consecutive rows at k = tid/32 and tid/32 + 8
        int r = row0 + (tid & 31) * 4;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int k = k0 + (tid >> 5) + h * 8;
            const float *base = op.p;
            int kk = k;
            if (op.p2 && k >= op.k_split) { base = op.p2; kk = k - op.k_split; }
            int64_t off = (int64_t)kk * op.ks + r;
            bool kin = k < K;
            if (kin && r + 3 < R && ((reinterpret_cast<uintptr_t>(base + off) & 15) == 0) &&
                (!op.sub || (reinterpret_cast<uintptr_t>(op.sub + off) & 15) == 0)) {
                float4 t = *reinterpret_cast<const float4 *>(base + off);
                if (op.sub) {
                    float4 s = *reinterpret_cast<const float4 *>(op.sub + off);
                    t.x = s.x - t.x; t.y = s.y - t.y; t.z = s.z - t.z; t.w = s.w - t.w;
                }
                v[h * 4 + 0] = t.x; v[h * 4 + 1] = t.y; v[h * 4 + 2] = t.z; v[h * 4 + 3] = t.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float t = 0.f;
                    if (kin && r + e < R) {
                        t = base[off + e];
                        if (op.sub) t = op.sub[off + e] - t;
                    }
                    v[h * 4 + e] = t;
                }
            }
        }
    } else {
        // thread: 4 consecutive k at row = tid/4 and tid/4 + 64
        int k = k0 + (tid & 3) * 4;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int r = row0 + (tid >> 2) + h * 64;
            const float *base = op.p;
            int kk = k;
            if (op.p2 && k >= op.k_split) { base = op.p2; kk = k - op.k_split; }
            int64_t off = (int64_t)r * op.rs + kk;
            bool rin = r < R;
            if (rin && k + 3 < K && ((reinterpret_cast<uintptr_t>(base + off) & 15) == 0) &&
                (!op.sub || (reinterpret_cast<uintptr_t>(op.sub + off) & 15) == 0)) {
                float4 t = *reinterpret_cast<const float4 *>(base + off);
                if (op.sub) {
                    float4 s = *reinterpret_cast<const float4 *>(op.sub + off);
                    t.x = s.x - t.x; t.y = s.y - t.y; t.z = s.z - t.z; t.w = s.w - t.w;
                }
                v[h * 4 + 0] = t.x; v[h * 4 + 1] = t.y; v[h * 4 + 2] = t.z; v[h * 4 + 3] = t.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float t = 0.f;
                    if (rin && k + e < K) {
                        t = base[off + e];
                        if (op.sub) t = op.sub[off + e] - t;
                    }
                    v[h * 4 + e] = t;
                }
            }
        }
    }
}

template <bool RC>
__device__ __forceinline__ void gemm_store(float (*S)[GBM + GPAD], int tid, const float (&v)[8]) {
    if (RC) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int k = (tid >> 5) + h * 8;
            *reinterpret_cast<float4 *>(&S[k][(tid & 31) * 4]) =
                make_float4(v[h * 4], v[h * 4 + 1], v[h * 4 + 2], v[h * 4 + 3]);
        }
    } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int r = (tid >> 2) + h * 64;
#pragma unroll
            for (int e = 0; e < 4; ++e) S[(tid & 3) * 4 + e][r] = v[h * 4 + e];
        }
    }
}

template <bool A_RC, bool B_RC>
__global__ void __launch_bounds__(256) simt_gemm_kernel(GemmProblem pr) {
    __shared__ __align__(16) float As[2][GBK][GBM + GPAD];
    __shared__ __align__(16) float Bs[2][GBK][GBN + GPAD];

    const int z = blockIdx.z;
    int M = pr.M, N = pr.N, K = pr.K;
    if (z == pr.nbatch - 1) {
        if (pr.batchM_last) M = pr.batchM_last;
        if (pr.batchN_last) N = pr.batchN_last;
        if (pr.batchK_last) K = pr.batchK_last;
    }
    Operand A = pr.A, B = pr.B;
    A.p += z * pr.batchA; if (A.p2) A.p2 += z * pr.batchA; if (A.sub) A.sub += z * pr.batchA;
    B.p += z * pr.batchB; if (B.p2) B.p2 += z * pr.batchB; if (B.sub) B.sub += z * pr.batchB;
    float *C = pr.C + z * pr.batchC;

    const int i0 = blockIdx.y * GBM, j0 = blockIdx.x * GBN;
    if (i0 >= M || j0 >= N) return;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int mode = pr.mode;

    bool skip = false;
    int kb = 0, ke = K;
    if (mode == GEMM_UPPER_TILES) skip = i0 >= j0 + GBN;
    else if (mode == GEMM_O) { skip = i0 >= j0 + GBN; kb = j0; }
    else if (mode == GEMM_P) { skip = i0 >= j0 + GBN; kb = i0; ke = min(K, j0 + GBN); }
    else if (mode == GEMM_TRI_RIGHT) ke = min(K, j0 + GBN);
    else if (mode == GEMM_TRI_LEFT) kb = i0;

    float acc[8][8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = 0.f;

    if (!skip && kb < ke) {
        float va[8], vb[8];
        gemm_load<A_RC>(A, i0, kb, M, ke, tid, va);
        gemm_load<B_RC>(B, j0, kb, N, ke, tid, vb);
        gemm_store<A_RC>(As[0], tid, va);
        gemm_store<B_RC>(Bs[0], tid, vb);
        __syncthreads();
        int buf = 0;
        for (int k0 = kb; k0 < ke; k0 += GBK) {
            bool more = k0 + GBK < ke;
            if (more) {
                gemm_load<A_RC>(A, i0, k0 + GBK, M, ke, tid, va);
                gemm_load<B_RC>(B, j0, k0 + GBK, N, ke, tid, vb);
            }
#pragma unroll
            for (int k = 0; k < GBK; ++k) {
                float4 a0 = *reinterpret_cast<const float4 *>(&As[buf][k][ty * 4]);
                float4 a1 = *reinterpret_cast<const float4 *>(&As[buf][k][64 + ty * 4]);
                float4 b0 = *reinterpret_cast<const float4 *>(&Bs[buf][k][tx * 4]);
                float4 b1 = *reinterpret_cast<const float4 *>(&Bs[buf][k][64 + tx * 4]);
                float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int x = 0; x < 8; ++x)
#pragma unroll
                    for (int y = 0; y < 8; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
            }
            if (more) {
                gemm_store<A_RC>(As[buf ^ 1], tid, va);
                gemm_store<B_RC>(Bs[buf ^ 1], tid, vb);
                __syncthreads();
                buf ^= 1;
            }
        }
    } else if (skip && mode != GEMM_P) {
        return;
    }

    const float alpha = pr.alpha, beta = pr.beta;
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        int i = i0 + (x < 4 ? ty * 4 + x : 64 + ty * 4 + (x - 4));
        if (i >= M) continue;
#pragma unroll
        for (int yh = 0; yh < 2; ++yh) {
            int j = j0 + yh * 64 + tx * 4;
            float *cp = C + (int64_t)i * pr.ldc + j;
            float o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float val = alpha * acc[x][yh * 4 + e];
                if ((mode == GEMM_O || mode == GEMM_P) && (j + e) <= i) val = 0.f;
                o[e] = val;
            }
            bool masked = (mode == GEMM_O || mode == GEMM_P);
            if (j + 3 < N && ((reinterpret_cast<uintptr_t>(cp) & 15) == 0)) {
                float4 t = make_float4(o[0], o[1], o[2], o[3]);
                if (beta != 0.f && !masked) {
                    float4 c = *reinterpret_cast<const float4 *>(cp);
                    t.x += beta * c.x; t.y += beta * c.y; t.z += beta * c.z; t.w += beta * c.w;
                }
                *reinterpret_cast<float4 *>(cp) = t;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (j + e < N) cp[e] = o[e] + ((beta != 0.f && !masked) ? beta * cp[e] : 0.f);
            }
        }
    }
}

struct LaunchCounter;

inline cudaError_t launch_simt_gemm(const GemmProblem &pr, bool a_rc, bool b_rc, cudaStream_t s) {
    if (pr.M <= 0 || pr.N <= 0 || pr.nbatch <= 0) return cudaSuccess;
    dim3 grid((pr.N + GBN - 1) / GBN, (pr.M + GBM - 1) / GBM, pr.nbatch);
    if (a_rc && b_rc) simt_gemm_kernel<true, true><<<grid, 256, 0, s>>>(pr);
    else if (a_rc && !b_rc) simt_gemm_kernel<true, false><<<grid, 256, 0, s>>>(pr);
    else if (!a_rc && b_rc) simt_gemm_kernel<false, true><<<grid, 256, 0, s>>>(pr);
    else simt_gemm_kernel<false, false><<<grid, 256, 0, s>>>(pr);
    return cudaGetLastError();
}

inline Operand make_operand(const float *p, int64_t rs, int64_t ks) {
    Operand o; o.p = p; o.rs = rs; o.ks = ks; o.p2 = nullptr; o.k_split = 0; o.sub = nullptr; return o;
}

inline GemmProblem make_problem(Operand A, Operand B, float *C, int64_t ldc, int M, int N, int K,
                                float alpha, float beta, int mode) {
    GemmProblem p; p.A = A; p.B = B; p.C = C; p.ldc = ldc; p.M = M; p.N = N; p.K = K;
    p.alpha = alpha; p.beta = beta; p.mode = mode; p.batchA = p.batchB = p.batchC = 0;
    p.batchM_last = p.batchN_last = p.batchK_last = 0; p.nbatch = 1; return p;
}

}  // namespace gptaq
