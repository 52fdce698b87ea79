// float32-grade tensor-core GEMM for sm_100a:  C = alpha * A * B^T + beta * C.
//
// Every operand is given as two K-major float32 arrays that hold TF32 values, hi = tf32(x)
// and lo = tf32(x - hi) (split_kernel below makes them), and the product is evaluated as
// hi*hi + hi*lo + lo*hi with tcgen05.mma.kind::tf32 and float32 accumulation in tensor
// memory: about 22 significant bits per factor, which is what the factorisation, the
// correction matrix and the propagation of quantization errors need (single TF32/fp16
// products flip integer codes).  TMA loads 128 x 32 (A) and 256 x 32 (B) tiles of both
// parts into 128-byte-swizzled shared memory; one thread issues the MMAs into one of two
// 128 x 256 accumulators; eight epilogue warps drain them.  Accumulation chains in tensor
// memory are cut every TCHUNK K-blocks and added into float32 registers with
// round-to-nearest (the tensor core truncates its accumulator).
//
// One kernel serves all shapes of the solve through a small tile description: batches of
// equally shaped problems inside one matrix (block inversion by doubling), K ranges cut to
// the non-zero part of triangular operands, a B operand that switches to a second matrix
// after k_split ([U ; P] of the lazy-batch update), and masked stores.
//
// Every wait on an mbarrier is bounded; see umma_gemm.cuh.
#pragma once
#include "umma_gemm.cuh"

namespace gptaq {

constexpr int TBM = 128, TBN = 256, TBK = 32, TSTAGES = 2;
constexpr int TA_BYTES = TBM * TBK * 4;
constexpr int TB_BYTES = TBN * TBK * 4;
constexpr int TSTAGE_BYTES = 2 * TA_BYTES + 2 * TB_BYTES;
constexpr int TCHUNK = 4;            // K-blocks (of 32) per accumulation chain in tensor memory
constexpr int TC_THREADS = 64 + 32 * UEPI_WARPS;
constexpr size_t TC_SMEM = (size_t)TSTAGES * TSTAGE_BYTES + 1024 + 256;

enum TcMode {
    TC_FULL = 0,
    TC_UPPER_TILES = 1,   // tiles entirely below the diagonal are skipped
    TC_O = 2,             // C[i][a] = sum_{k >= a} ..., lower tiles skipped
    TC_P = 3,             // C[i][j] = sum_{i <= k < j + tile} ..., lower tiles zero-filled
    TC_TRI_RIGHT = 4,     // B upper triangular: k <= j
    TC_TRI_LEFT = 5       // A upper triangular: k >= i
};
enum TcMask {
    TC_MASK_NONE = 0,
    TC_MASK_UPPER_KEEP = 1,     // elements with j < i are left untouched
    TC_MASK_STRICT_ZERO = 2     // elements with j <= i are written as 0
};

struct TcGemmArgs {
    float *C;
    long long ldc, c_bstride;
    int M, N, K;                     // one batch entry: C is M x N, K contraction steps
    int M_last, N_last, K_last;      // extents of the last batch entry (0: same)
    int nbatch;
    // tensor-map coordinates of a batch entry's first row / first k: base + z * stride
    int a_row0, a_row_bs, a_k0, a_k_bs;
    int b_row0, b_row_bs, b_k0, b_k_bs;
    int k_split;                     // > 0: contraction steps >= k_split read the second B matrix
    int b2_k0;                       //      at k coordinate b2_k0 + (k - k_split)
    float alpha, beta;
    int mode, mask;
    StateHeader *hd;
};

struct TcTile {
    bool skip, zero_fill, work;
    int z, i0, j0, Mz, Nz, kb0, kb1;   // K-block range [kb0, kb1)
};

__device__ __forceinline__ void tc_decode(const TcGemmArgs &a, int t, TcTile &ti) {
    const int TM = (a.M + TBM - 1) / TBM, TN = (a.N + TBN - 1) / TBN;
    const int per = TM * TN;
    ti.z = t / per;
    const int rem = t - ti.z * per;
    // row tile fastest: the tiles a CTA meets as it strides through the list then cover all column
    // tiles, i.e. all lengths of the triangular K ranges, evenly (column-tile-fastest order gives
    // every CTA the same few column tiles again and again: up to 2x imbalance)
    const int tn = rem / TM, tm = rem - tn * TM;
    ti.i0 = tm * TBM; ti.j0 = tn * TBN;
    const bool last = ti.z == a.nbatch - 1;
    ti.Mz = (last && a.M_last) ? a.M_last : a.M;
    ti.Nz = (last && a.N_last) ? a.N_last : a.N;
    const int Kz = (last && a.K_last) ? a.K_last : a.K;
    ti.skip = ti.i0 >= ti.Mz || ti.j0 >= ti.Nz;
    ti.zero_fill = false;
    int kb = 0, ke = Kz;
    switch (a.mode) {
        case TC_UPPER_TILES: if (ti.i0 >= ti.j0 + TBN) ti.skip = true; break;
        case TC_O: if (ti.i0 >= ti.j0 + TBN) ti.skip = true; kb = ti.j0; break;
        case TC_P:
            if (!ti.skip && ti.i0 >= ti.j0 + TBN) { ti.skip = true; ti.zero_fill = true; }
            kb = ti.i0; ke = min(Kz, ti.j0 + TBN); break;
        case TC_TRI_RIGHT: ke = min(Kz, ti.j0 + TBN); break;
        case TC_TRI_LEFT: kb = ti.i0; break;
        default: break;
    }
    ti.kb0 = kb / TBK;
    ti.kb1 = (ke + TBK - 1) / TBK;
    ti.work = !ti.skip && ti.kb0 < ti.kb1;
}

__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}

// kind::tf32 instruction descriptor: TF32 A and B (both K-major), fp32 D, M = 128, N = 256.
constexpr uint32_t UMMA_IDESC_TF32 = (1u << 4) | (2u << 7) | (2u << 10) | ((TBN >> 3) << 17) | ((TBM >> 4) << 24);

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapAhi, const __grid_constant__ CUtensorMap mapAlo,
               const __grid_constant__ CUtensorMap mapBhi, const __grid_constant__ CUtensorMap mapBlo,
               const __grid_constant__ CUtensorMap mapB2hi, const __grid_constant__ CUtensorMap mapB2lo,
               TcGemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    const uint32_t bar0 = base + TSTAGES * TSTAGE_BYTES;
    // barrier slots (8 bytes each): full[2], empty[2], tfull[2], tempty[2]; then tmem slot, abort flag
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (TSTAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * TSTAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * TSTAGES + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(aligned + TSTAGES * TSTAGE_BYTES + 8 * (2 * TSTAGES + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TSTAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), UEPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t *>(tmem_slot))), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int ntiles = a.nbatch * ((a.M + TBM - 1) / TBM) * ((a.N + TBN - 1) / TBN);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            TcTile ti;
            for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
                tc_decode(a, t, ti);
                if (!ti.work) continue;
                const int arow = a.a_row0 + ti.z * a.a_row_bs + ti.i0;
                const int brow = a.b_row0 + ti.z * a.b_row_bs + ti.j0;
                const int ak0 = a.a_k0 + ti.z * a.a_k_bs, bk0 = a.b_k0 + ti.z * a.b_k_bs;
                for (int kb = ti.kb0; kb < ti.kb1; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t s0 = base + stage * TSTAGE_BYTES;
                    const int k = kb * TBK;
                    const bool second = a.k_split > 0 && k >= a.k_split;
                    mbar_expect_tx(full_bar(stage), TSTAGE_BYTES);
                    tma_load_2d(s0, &mapAhi, ak0 + k, arow, full_bar(stage));
                    tma_load_2d(s0 + TA_BYTES, &mapAlo, ak0 + k, arow, full_bar(stage));
                    if (!second) {
                        tma_load_2d(s0 + 2 * TA_BYTES, &mapBhi, bk0 + k, brow, full_bar(stage));
                        tma_load_2d(s0 + 2 * TA_BYTES + TB_BYTES, &mapBlo, bk0 + k, brow, full_bar(stage));
                    } else {
                        const int k2 = a.b2_k0 + (k - a.k_split);
                        tma_load_2d(s0 + 2 * TA_BYTES, &mapB2hi, k2, brow, full_bar(stage));
                        tma_load_2d(s0 + 2 * TA_BYTES + TB_BYTES, &mapB2lo, k2, brow, full_bar(stage));
                    }
                    ++issued;
                    if (++stage == TSTAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // give copies that are still in flight time to land before the CTA exits
                const long long t0 = clock64();
                while (issued > 0 && clock64() - t0 < 4000000LL) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, ccount = 0;
            bool ok = true;
            TcTile ti;
            for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
                tc_decode(a, t, ti);
                if (!ti.work) continue;
                for (int kc = ti.kb0; kc < ti.kb1 && ok; kc += TCHUNK) {
                    const uint32_t buf = ccount & 1u, cphase = (ccount >> 1) & 1u;
                    if (!mbar_wait(tempty_bar(buf), cphase ^ 1u, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * TBN;
                    const int kc1 = min(kc + TCHUNK, ti.kb1);
                    for (int kb = kc; kb < kc1; ++kb) {
                        if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t s0 = base + stage * TSTAGE_BYTES;
                        const uint64_t ahi = make_kmajor_desc(s0), alo = make_kmajor_desc(s0 + TA_BYTES);
                        const uint64_t bhi = make_kmajor_desc(s0 + 2 * TA_BYTES);
                        const uint64_t blo = make_kmajor_desc(s0 + 2 * TA_BYTES + TB_BYTES);
                        // small terms first, the hi * hi term last
#pragma unroll
                        for (int k = 0; k < TBK / 8; ++k)
                            umma_tf32(d_tmem, alo + (uint64_t)(k * 2), bhi + (uint64_t)(k * 2), UMMA_IDESC_TF32,
                                      (kb != kc || k != 0) ? 1u : 0u);
#pragma unroll
                        for (int k = 0; k < TBK / 8; ++k)
                            umma_tf32(d_tmem, ahi + (uint64_t)(k * 2), blo + (uint64_t)(k * 2), UMMA_IDESC_TF32, 1u);
#pragma unroll
                        for (int k = 0; k < TBK / 8; ++k)
                            umma_tf32(d_tmem, ahi + (uint64_t)(k * 2), bhi + (uint64_t)(k * 2), UMMA_IDESC_TF32, 1u);
                        umma_commit(empty_bar(stage));
                        if (++stage == TSTAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit(tfull_bar(buf));
                    ++ccount;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        const int quarter = warp & 3;                 // TMEM lanes 32 * quarter .. + 31
        const int half = (warp - 2) >> 2;             // columns [128 * half, 128 * half + 128)
        uint32_t ccount = 0;
        bool ok = true;
        float acc[TBN / 2];
        TcTile ti;
        for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
            tc_decode(a, t, ti);
            if (ti.skip && !ti.zero_fill) continue;
#pragma unroll
            for (int i = 0; i < TBN / 2; ++i) acc[i] = 0.f;
            if (ti.work) {
                for (int kc = ti.kb0; kc < ti.kb1; kc += TCHUNK) {
                    const uint32_t buf = ccount & 1u, cphase = (ccount >> 1) & 1u;
                    if (!mbar_wait(tfull_bar(buf), cphase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + buf * TBN + half * (TBN / 2) + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
                    for (int gq = 0; gq < TBN / 2 / 32; ++gq) {
                        uint32_t v[32];
                        tmem_ld32(taddr + gq * 32, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[gq * 32 + i] += __uint_as_float(v[i]);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(buf));
                    ++ccount;
                }
                if (!ok) break;
            }
            const int row = ti.i0 + quarter * 32 + lane;           // within the batch entry
            const int col0 = ti.j0 + half * (TBN / 2);
            if (row >= ti.Mz) continue;
            float *cp = a.C + (long long)ti.z * a.c_bstride + (long long)row * a.ldc + col0;
            const float alpha = a.alpha, beta = a.beta;
            const bool vec_ok = (reinterpret_cast<uintptr_t>(cp) & 15) == 0;
#pragma unroll
            for (int q = 0; q < TBN / 2 / 4; ++q) {
                const int c = col0 + 4 * q;
                if (c >= ti.Nz) break;
                float v[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) v[e] = alpha * acc[4 * q + e];
                if (a.mask == TC_MASK_STRICT_ZERO) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (c + e <= row) v[e] = 0.f;
                }
                const bool keep_all = a.mask != TC_MASK_UPPER_KEEP || c >= row;
                if (vec_ok && c + 3 < ti.Nz && keep_all) {
                    if (beta == 1.f) {
                        // each element belongs to exactly one thread per launch: a reduction without
                        // return value is a plain, order-independent "+=" that needs no round trip
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(cp + 4 * q),
                                     "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
                    } else {
                        if (beta != 0.f) {
                            const float4 o = *reinterpret_cast<const float4 *>(cp + 4 * q);
                            v[0] = fmaf(beta, o.x, v[0]); v[1] = fmaf(beta, o.y, v[1]);
                            v[2] = fmaf(beta, o.z, v[2]); v[3] = fmaf(beta, o.w, v[3]);
                        }
                        *reinterpret_cast<float4 *>(cp + 4 * q) = make_float4(v[0], v[1], v[2], v[3]);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (c + e >= ti.Nz) continue;
                        if (a.mask == TC_MASK_UPPER_KEEP && c + e < row) continue;
                        cp[4 * q + e] = (beta != 0.f) ? fmaf(beta, cp[4 * q + e], v[e]) : v[e];
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) record_status(a.hd, ST_TIMEOUT, 1000000 + blockIdx.x);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---------------------------------------------------------------------------
// Operand preparation: dst_hi / dst_lo <- split(scale * src), optionally transposed and
// masked to the (strictly) upper triangle of the source, tile by tile through shared memory.
//   src element (r, c), r < rows, c < cols, at src[r * lds + c];
//   plain:      dst[r * ldd + c];   transposed: dst[c * ldd + r].
// Elements outside the mask are written as zero.  blockIdx.z walks batch entries.
// ---------------------------------------------------------------------------
enum SplitMask { SPLIT_ALL = 0, SPLIT_UPPER = 1, SPLIT_STRICT_UPPER = 2 };

struct SplitArgs {
    const float *src; long long lds, src_bstride;
    float *hi, *lo; long long ldd, dst_bstride;
    int rows, cols, rows_last, cols_last, nbatch;
    int transpose, mask;
    float scale;
};

__global__ void __launch_bounds__(256) split_kernel(SplitArgs a) {
    __shared__ float th[64][65], tl[64][65];
    const int z = blockIdx.z;
    const bool last = z == a.nbatch - 1;
    const int rows = (last && a.rows_last) ? a.rows_last : a.rows;
    const int cols = (last && a.cols_last) ? a.cols_last : a.cols;
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    if (r0 >= rows || c0 >= cols) return;
    const float *src = a.src + (long long)z * a.src_bstride;
    float *hi = a.hi + (long long)z * a.dst_bstride, *lo = a.lo + (long long)z * a.dst_bstride;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    for (int rr = ty; rr < 64; rr += 4) {
        const int r = r0 + rr, c = c0 + tx;
        float x = 0.f;
        if (r < rows && c < cols) {
            const bool keep = a.mask == SPLIT_ALL || (a.mask == SPLIT_UPPER ? c >= r : c > r);
            if (keep) x = a.scale * src[(long long)r * a.lds + c];
        }
        const float h = tf32_rn(x);
        const float l = tf32_rn(x - h);
        if (!a.transpose) {
            if (r < rows && c < cols) {
                hi[(long long)r * a.ldd + c] = h;
                lo[(long long)r * a.ldd + c] = l;
            }
        } else {
            th[rr][tx] = h; tl[rr][tx] = l;
        }
    }
    if (a.transpose) {
        __syncthreads();
        for (int cc = ty; cc < 64; cc += 4) {
            const int c = c0 + cc, r = r0 + tx;
            if (r < rows && c < cols) {
                hi[(long long)c * a.ldd + r] = th[tx][cc];
                lo[(long long)c * a.ldd + r] = tl[tx][cc];
            }
        }
    }
}

}  // namespace gptaq
