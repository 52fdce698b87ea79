// float32-grade tensor-core GEMM for sm_100a:  C = alpha * A * B^T + beta * C.
//
// Every operand is given as two K-major arrays, a high part and a low part of each element
// (hi = round(x), lo = round(x - hi)), and the product is evaluated as hi*hi + hi*lo + lo*hi
// on the tensor cores with float32 accumulation in tensor memory: about 22 significant bits
// per factor, which is what the factorisation, the correction matrix and the propagation of
// quantization errors need (single TF32/fp16 products flip integer codes).  TMA loads the
// 128-row (A) and 256-row (B) tiles of both parts, one 128-byte row piece per K-block, into
// 128-byte-swizzled shared memory; one thread issues the MMAs into one of two 128 x 256
// accumulators; eight epilogue warps drain them.  Accumulation chains in tensor memory are
// cut every TCHUNK K-blocks and added into float32 registers with round-to-nearest (the
// tensor core truncates its accumulator).  "C += ..." results leave through shared memory
// as bulk tensor reductions (one request per 128 x 32 box) where C qualifies for a tensor
// map; per-thread 16-byte reductions saturate the L2's reduction rate long before HBM.
//
// One kernel serves all shapes of the solve through a small tile description: batches of
// equally shaped problems inside one matrix (block inversion by doubling), K ranges cut to
// the non-zero part of triangular operands, a B operand that switches to a second matrix
// after k_split ([U ; P] of the lazy-batch update), and masked stores.
//
// The kernel exists for two operand kinds.  TF32: hi / lo are float32 arrays holding TF32 values, no
// range limits, 32 contraction steps per 128-byte row.  FP16: hi = fp16(s x), lo = fp16(s x - hi) with a
// power-of-two scale s per operand that puts the largest magnitude at 2^14 (split16_kernel; the scale
// is recomputed from the recorded maximum wherever it is needed), 64 contraction steps per row and
// tcgen05.mma.kind::f16: half the operand bytes and twice the MMA rate for the same 22 bits.
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
// staging of the "C += ..." epilogue: per column half one 128 x 32 float32 box (128-byte rows, swizzled),
// handed to the TMA unit as a bulk reduction
constexpr int TC_STG_BOX_BYTES = TBM * 32 * 4;
constexpr int TC_STG_BYTES = 2 * TC_STG_BOX_BYTES;
constexpr size_t TC_SMEM = (size_t)TSTAGES * TSTAGE_BYTES + TC_STG_BYTES + 1024 + 256;

enum TcMode {
    TC_FULL = 0,
    TC_UPPER_TILES = 1,   // tiles entirely below the diagonal (column j + diag_off = row i) are skipped
    TC_O = 2,             // C[i][a] = sum_{k >= a} ..., lower tiles skipped
    TC_P = 3,             // C[i][j] = sum_{i <= k < j + tile} ..., lower tiles zero-filled
    TC_TRI_RIGHT = 4,     // B upper triangular: k <= j
    TC_TRI_LEFT = 5       // A upper triangular: k >= i
};
enum TcMask {
    TC_MASK_NONE = 0,
    TC_MASK_UPPER_KEEP = 1,     // elements with j + diag_off < i are left untouched
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
    // FP16 operands: bit patterns of the operands' largest magnitudes (the B matrices share one scale);
    // the result is divided by the two scales.  nullptr for TF32 operands.
    const unsigned *amax_a, *amax_b;
    const float *row_inv;            // FP16 operands with one scale per row of A: 1 / scale of row i (amax_a null)
    unsigned *amax_out;              // if set: receives (atomicMax) the bit pattern of max |C| over what is stored
    int c_tma;                       // beta == 1, one batch entry: C += through bulk tensor reductions (mapC)
    int diag_off;                    // C is a block of columns of a square matrix: its column j is column j + diag_off there
    // Tile scheduler: CTA b starts with tile b; further tile numbers come from a counter in global
    // memory that is never reset: this launch owns its values sched_base .. sched_base + tiles - 1
    // (tiles - grid numbers of tiles, and every CTA draws exactly one number beyond the last tile before
    // it stops), the host advances the base by `tiles` per launch.
    unsigned *sched;
    unsigned sched_base;
};

// Host-side twin of StateHeader::sched_counter: the first tile number of the next launch.
struct TcSched { unsigned base = 0; };

struct TcTile {
    bool skip, zero_fill, work;
    int z, i0, j0, Mz, Nz, kb0, kb1;   // K-block range [kb0, kb1)
};

__device__ __forceinline__ void tc_decode(const TcGemmArgs &a, int t, TcTile &ti, int bk) {
    const int TM = (a.M + TBM - 1) / TBM, TN = (a.N + TBN - 1) / TBN;
    const int per = TM * TN;
    // tiles are handed out in the order of t: long K ranges first (column tiles ascending where the
    // range shrinks with the column, descending where it grows), so that the last tiles drawn are short
    if (a.mode == TC_P || a.mode == TC_TRI_RIGHT) t = a.nbatch * per - 1 - t;
    ti.z = t / per;
    const int rem = t - ti.z * per;
    // row tile fastest: the CTAs that run at the same time share a column panel of B
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
        case TC_UPPER_TILES: if (ti.i0 >= ti.j0 + a.diag_off + TBN) ti.skip = true; break;
        case TC_O: if (ti.i0 >= ti.j0 + TBN) ti.skip = true; kb = ti.j0; break;
        case TC_P:
            if (!ti.skip && ti.i0 >= ti.j0 + TBN) { ti.skip = true; ti.zero_fill = true; }
            kb = ti.i0; ke = min(Kz, ti.j0 + TBN); break;
        case TC_TRI_RIGHT: ke = min(Kz, ti.j0 + TBN); break;
        case TC_TRI_LEFT: kb = ti.i0; break;
        default: break;
    }
    ti.kb0 = kb / bk;
    ti.kb1 = (ke + bk - 1) / bk;
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

// C[c1 .. , c0 ..] += box in shared memory (float32 add at the memory side, one request per box)
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap *map, uint32_t src, int c0, int c1) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// true for every thread of the named barrier if `flag` is set for any of them
__device__ __forceinline__ bool named_bar_any(int id, int nthreads, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.or.pred q, %2, %3, p;\n\t"
        "selp.b32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)flag), "r"(id), "r"(nthreads) : "memory");
    return r != 0;
}

template <bool F16>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapAhi, const __grid_constant__ CUtensorMap mapAlo,
               const __grid_constant__ CUtensorMap mapBhi, const __grid_constant__ CUtensorMap mapBlo,
               const __grid_constant__ CUtensorMap mapB2hi, const __grid_constant__ CUtensorMap mapB2lo,
               const __grid_constant__ CUtensorMap mapC, TcGemmArgs a) {
    constexpr int BK = F16 ? 2 * TBK : TBK;        // contraction steps per K-block (one 128-byte row)
    constexpr int KSTEP = F16 ? 16 : 8;            // contraction steps per MMA (32 bytes)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    const uint32_t stg0 = base + TSTAGES * TSTAGE_BYTES;
    const uint32_t bar0 = stg0 + TC_STG_BYTES;
    // barrier slots (8 bytes each): full[2], empty[2], tfull[2], tempty[2]; then tmem slot, abort flag
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (TSTAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * TSTAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * TSTAGES + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(aligned + TSTAGES * TSTAGE_BYTES + TC_STG_BYTES + 8 * (2 * TSTAGES + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    // tile scheduler ring (at byte 128 of the barrier block): sfull[4], sempty[4], then the four tile numbers
    constexpr int NR = 4;
    auto sfull_bar = [&](int s) { return bar0 + 128u + 8u * s; };
    auto sempty_bar = [&](int s) { return bar0 + 128u + 8u * (NR + s); };
    volatile int *ring = reinterpret_cast<volatile int *>(aligned + TSTAGES * TSTAGE_BYTES + TC_STG_BYTES + 128 + 8 * 2 * NR);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TSTAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int s = 0; s < NR; ++s) { mbar_init(sfull_bar(s), 1); mbar_init(sempty_bar(s), 1 + UEPI_WARPS); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), UEPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t *>(tmem_slot))), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();                      // everything above is independent of the previous kernel's results
    const uint32_t tmem_base = *tmem_slot;
    const int ntiles = a.nbatch * ((a.M + TBM - 1) / TBM) * ((a.N + TBN - 1) / TBN);

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, pushed = 0;
            int issued = 0;
            bool ok = true;
            TcTile ti;
            bool first = true;
            while (ok) {
                // next tile for this CTA; -1 once the list is exhausted.  The first one needs no round trip
                // to the counter: tile number = CTA number; the counter hands out the numbers from gridDim.x on.
                const unsigned ticket = first ? blockIdx.x : gridDim.x + (atomicAdd(a.sched, 1u) - a.sched_base);
                first = false;
                const int t = ticket < (unsigned)ntiles ? (int)ticket : -1;
                if (t >= 0) {
                    tc_decode(a, t, ti, BK);
                    if (ti.skip && !ti.zero_fill) continue;          // nothing to do for any role
                }
                {   // hand the number to the MMA issuer and the epilogue warps
                    const uint32_t slot = pushed % NR, sph = (pushed / NR) & 1u;
                    if (!mbar_wait(sempty_bar(slot), sph ^ 1u, abort_flag)) { ok = false; break; }
                    ring[slot] = t;
                    mbar_arrive(sfull_bar(slot));
                    ++pushed;
                }
                if (t < 0) break;
                if (!ti.work) continue;
                const int arow = a.a_row0 + ti.z * a.a_row_bs + ti.i0;
                const int brow = a.b_row0 + ti.z * a.b_row_bs + ti.j0;
                const int ak0 = a.a_k0 + ti.z * a.a_k_bs, bk0 = a.b_k0 + ti.z * a.b_k_bs;
                for (int kb = ti.kb0; kb < ti.kb1; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t s0 = base + stage * TSTAGE_BYTES;
                    const int k = kb * BK;
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
            for (uint32_t taken = 0; ok; ++taken) {
                const uint32_t slot = taken % NR, sph = (taken / NR) & 1u;
                if (!mbar_wait(sfull_bar(slot), sph, abort_flag)) break;
                const int t = ring[slot];
                mbar_arrive(sempty_bar(slot));
                if (t < 0) break;
                tc_decode(a, t, ti, BK);
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
                        auto mma = [&](uint64_t ad, uint64_t bd, uint32_t accumulate) {
                            if (F16) umma_f16(d_tmem, ad, bd, UMMA_IDESC_F16, accumulate);
                            else umma_tf32(d_tmem, ad, bd, UMMA_IDESC_TF32, accumulate);
                        };
#pragma unroll
                        for (int k = 0; k < BK / KSTEP; ++k)
                            mma(alo + (uint64_t)(k * 2), bhi + (uint64_t)(k * 2), (kb != kc || k != 0) ? 1u : 0u);
#pragma unroll
                        for (int k = 0; k < BK / KSTEP; ++k) mma(ahi + (uint64_t)(k * 2), blo + (uint64_t)(k * 2), 1u);
#pragma unroll
                        for (int k = 0; k < BK / KSTEP; ++k) mma(ahi + (uint64_t)(k * 2), bhi + (uint64_t)(k * 2), 1u);
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
        float out_max = 0.f;
        float op_scale = 1.f;            // 1 / (scale of A * scale of B), without the per-row part
        if (F16) {
            if (a.amax_a) op_scale /= split_scale(__uint_as_float(*a.amax_a));
            if (a.amax_b) op_scale /= split_scale(__uint_as_float(*a.amax_b));
        }
        TcTile ti;
        for (uint32_t taken = 0; ok; ++taken) {
            const uint32_t slot = taken % NR, sph = (taken / NR) & 1u;
            if (!mbar_wait(sfull_bar(slot), sph, abort_flag)) break;
            const int t = ring[slot];
            __syncwarp();
            if (lane == 0) mbar_arrive(sempty_bar(slot));
            if (t < 0) break;
            tc_decode(a, t, ti, BK);
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
                if (!a.c_tma && !ok) break;
            }
            const int row = ti.i0 + quarter * 32 + lane;           // within the batch entry
            const int col0 = ti.j0 + half * (TBN / 2);
            if (a.c_tma) {
                // C += alpha * acc through shared memory and bulk tensor reductions: the four warps of a
                // column half fill one 128 x 32 box at a time (row = TMEM lane, 16-byte chunks swizzled
                // like the tensor map's 128-byte mode), one thread hands it to the TMA unit.  Rows and
                // columns beyond the matrix are clipped by the tensor map.
                if (named_bar_any(1 + half, 128, !ok)) { ok = false; break; }       // a wait gave up: all leave together
                float alpha = a.alpha;
                if (F16) alpha *= (a.row_inv && row < ti.Mz) ? op_scale * a.row_inv[row] : op_scale;
                const bool issuer = quarter == 2 && lane == 0;                       // first warp of the half
                const int r_in = quarter * 32 + lane;
                const uint32_t box = stg0 + half * TC_STG_BOX_BYTES;
#pragma unroll
                for (int g = 0; g < TBN / 2 / 32; ++g) {
                    if (col0 + 32 * g >= ti.Nz) break;
                    if (issuer) bulk_wait_read0();                                   // the box has been read out
                    named_bar_sync(1 + half, 128);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            v[e] = alpha * acc[32 * g + 4 * j + e];
                            if (a.mask == TC_MASK_UPPER_KEEP && col0 + 32 * g + 4 * j + e + a.diag_off < row) v[e] = 0.f;
                        }
                        const uint32_t dst = box + r_in * 128 + ((j ^ (r_in & 7)) << 4);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
                    }
                    fence_proxy_async_smem();
                    named_bar_sync(1 + half, 128);
                    if (issuer) {
                        tma_reduce_add_2d(&mapC, box, col0 + 32 * g, ti.i0);
                        bulk_commit();
                    }
                }
                continue;
            }
            if (row >= ti.Mz) continue;
            float *cp = a.C + (long long)ti.z * a.c_bstride + (long long)row * a.ldc + col0;
            const float beta = a.beta;
            float alpha = a.alpha;
            if (F16) alpha *= a.row_inv ? op_scale * a.row_inv[(long long)ti.z * a.M + row] : op_scale;
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
                if (a.amax_out) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) if (c + e < ti.Nz) out_max = fmaxf(out_max, fabsf(v[e]));
                }
                const bool keep_all = a.mask != TC_MASK_UPPER_KEEP || c + a.diag_off >= row;
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
                        if (a.mask == TC_MASK_UPPER_KEEP && c + e + a.diag_off < row) continue;
                        cp[4 * q + e] = (beta != 0.f) ? fmaf(beta, cp[4 * q + e], v[e]) : v[e];
                    }
                }
            }
        }
        if (a.c_tma) bulk_wait0();          // (only the issuing threads have groups outstanding)
        if (a.amax_out) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) out_max = fmaxf(out_max, __shfl_xor_sync(0xffffffffu, out_max, o));
            if (lane == 0 && out_max > 0.f) atomicMax(a.amax_out, __float_as_uint(out_max));
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

// ---------------------------------------------------------------------------
// FP16 operand preparation.  absmax_kernel (a CTA per row, strided) records max |scale * src| over the
// (masked) region as a float bit pattern (atomicMax on the bits orders non-negative floats);
// split16_kernel then writes
// hi = fp16(s x), lo = fp16(s x - hi), x = scale * src, s = split_scale(recorded maximum), with the
// same options as split_kernel.  The slot has to be zeroed before the first absmax_kernel into it;
// several matrices that share a scale are reduced into the same slot.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) absmax_kernel(const float *src, long long lds, int rows, int cols, int mask,
                                                     float scale, unsigned *slot) {
    __shared__ float red[8];
    float m = 0.f;
    const bool vec = (lds & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0;
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        const int cb = mask == SPLIT_ALL ? 0 : (mask == SPLIT_UPPER ? r : r + 1);     // first column kept
        const float *row = src + (long long)r * lds;
        if (vec) {
            for (int c4 = (cb >> 2) + threadIdx.x; 4 * c4 < cols; c4 += 256) {
                const int c = 4 * c4;
                float v[4] = {0.f, 0.f, 0.f, 0.f};
                if (c + 3 < cols) {
                    const float4 q = *reinterpret_cast<const float4 *>(row + c);
                    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
                } else {
                    for (int e = 0; c + e < cols; ++e) v[e] = row[c + e];
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) if (c + e >= cb) m = fmaxf(m, fabsf(v[e]));
            }
        } else {
            for (int c = cb + threadIdx.x; c < cols; c += 256) m = fmaxf(m, fabsf(row[c]));
        }
    }
    m *= fabsf(scale);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) m = fmaxf(m, red[w]);
        if (m > 0.f) atomicMax(slot, __float_as_uint(m));
    }
}

struct Split16Args {
    const float *src; long long lds, src_bstride;
    __half *hi, *lo; long long ldd, dst_bstride;
    int rows, cols, rows_last, cols_last, nbatch;      // blockIdx.z walks batch entries, as in split_kernel
    int transpose, mask;       // transpose 2: both forms, the plain one to (hi, lo), the transposed one to (hi_t, lo_t)
    float scale;
    const unsigned *amax;
    __half *hi_t, *lo_t;
};

__device__ __forceinline__ void split16_pack(const float (&x)[4], uint2 &hi, uint2 &lo) {
    __half h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { h[e] = __float2half_rn(x[e]); l[e] = __float2half_rn(x[e] - __half2float(h[e])); }
    const __half2 h01 = __halves2half2(h[0], h[1]), h23 = __halves2half2(h[2], h[3]);
    const __half2 l01 = __halves2half2(l[0], l[1]), l23 = __halves2half2(l[2], l[3]);
    hi = make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
    lo = make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
}

// 64 x 64 tiles; a thread handles four consecutive source columns (plain) or four consecutive source
// rows of one column (transposed), so that every store is 8 bytes.  Needs lds, ldd multiples of 4 and
// 16- / 8-byte aligned bases (the host checks); rows and cols are arbitrary.
__global__ void __launch_bounds__(256) split16_kernel(Split16Args a) {
    __shared__ float tile[64][65];
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    {
        const int z = blockIdx.z;
        const bool last = z == a.nbatch - 1;
        if (last && a.rows_last) a.rows = a.rows_last;
        if (last && a.cols_last) a.cols = a.cols_last;
        if (r0 >= a.rows || c0 >= a.cols) return;
        a.src += (long long)z * a.src_bstride;
        a.hi += (long long)z * a.dst_bstride;
        a.lo += (long long)z * a.dst_bstride;
        if (a.transpose == 2) { a.hi_t += (long long)z * a.dst_bstride; a.lo_t += (long long)z * a.dst_bstride; }
    }
    const float s = a.scale * split_scale(__uint_as_float(*a.amax));
    const int tq = threadIdx.x & 15, ty = threadIdx.x >> 4;        // 16 quads x 16 rows
    // all four loads of the thread first (a store in between would serialise them), none for quads that
    // the mask empties
    float xs[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty + 16 * i, c = c0 + 4 * tq;
#pragma unroll
        for (int e = 0; e < 4; ++e) xs[i][e] = 0.f;
        const bool any = a.mask == SPLIT_ALL || (a.mask == SPLIT_UPPER ? c + 3 >= r : c + 3 > r);
        if (r < a.rows && c < a.cols && any) {
            const float *sp = a.src + (long long)r * a.lds + c;
            if (c + 3 < a.cols) {
                const float4 q = __ldcs(reinterpret_cast<const float4 *>(sp));
                xs[i][0] = q.x; xs[i][1] = q.y; xs[i][2] = q.z; xs[i][3] = q.w;
            } else {
                for (int e = 0; c + e < a.cols; ++e) xs[i][e] = sp[e];
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int rr = ty + 16 * i;
        const int r = r0 + rr, c = c0 + 4 * tq;
        float x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool keep = a.mask == SPLIT_ALL || (a.mask == SPLIT_UPPER ? c + e >= r : c + e > r);
            x[e] = keep ? s * xs[i][e] : 0.f;
        }
        if (a.transpose != 1) {
            if (r < a.rows && c < a.cols) {
                uint2 hi, lo;
                split16_pack(x, hi, lo);
                __half *ph = a.hi + (long long)r * a.ldd + c, *pl = a.lo + (long long)r * a.ldd + c;
                if (c + 3 < a.cols) {
                    *reinterpret_cast<uint2 *>(ph) = hi;
                    *reinterpret_cast<uint2 *>(pl) = lo;
                } else {
                    const __half *hh = reinterpret_cast<const __half *>(&hi), *ll = reinterpret_cast<const __half *>(&lo);
                    for (int e = 0; c + e < a.cols; ++e) { ph[e] = hh[e]; pl[e] = ll[e]; }
                }
            }
        }
        if (a.transpose) {
#pragma unroll
            for (int e = 0; e < 4; ++e) tile[rr][4 * tq + e] = x[e];
        }
    }
    if (a.transpose) {
        __half *th = a.transpose == 2 ? a.hi_t : a.hi, *tl = a.transpose == 2 ? a.lo_t : a.lo;
        __syncthreads();
        // destination row = source column c, destination columns = source rows r0 + 4 * tq ..
        for (int cc = ty; cc < 64; cc += 16) {
            const int c = c0 + cc, r = r0 + 4 * tq;
            if (c >= a.cols || r >= a.rows) continue;
            const float x[4] = {tile[4 * tq][cc], tile[4 * tq + 1][cc], tile[4 * tq + 2][cc], tile[4 * tq + 3][cc]};
            uint2 hi, lo;
            split16_pack(x, hi, lo);
            __half *ph = th + (long long)c * a.ldd + r, *pl = tl + (long long)c * a.ldd + r;
            if (r + 3 < a.rows) {
                *reinterpret_cast<uint2 *>(ph) = hi;
                *reinterpret_cast<uint2 *>(pl) = lo;
            } else {
                const __half *hh = reinterpret_cast<const __half *>(&hi), *ll = reinterpret_cast<const __half *>(&lo);
                for (int e = 0; r + e < a.rows; ++e) { ph[e] = hh[e]; pl[e] = ll[e]; }
            }
        }
    }
}

// Rows of a float32 matrix [rows][cols] (pitch ld) as fp16 hi / lo parts with one power-of-two scale per
// row (the row's largest magnitude lands in [2^13, 2^14)); row_inv[r] = 1 / scale.  One warp per row;
// cols a multiple of 4, 16-byte aligned rows.
__global__ void __launch_bounds__(256) rowscale_split16_kernel(const float *src, long long ld, int rows, int cols,
                                                               __half *hi, __half *lo, float *row_inv) {
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float *row = src + (long long)r * ld;
    float m = 0.f;
    for (int c = 4 * lane; c < cols; c += 128) {
        const float4 q = *reinterpret_cast<const float4 *>(row + c);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(q.x), fabsf(q.y))), fmaxf(fabsf(q.z), fabsf(q.w)));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float sc = split_scale(m);
    if (lane == 0) row_inv[r] = 1.f / sc;
    for (int c = 4 * lane; c < cols; c += 128) {
        const float4 q = *reinterpret_cast<const float4 *>(row + c);
        const float x[4] = {sc * q.x, sc * q.y, sc * q.z, sc * q.w};
        uint2 h2, l2;
        split16_pack(x, h2, l2);
        *reinterpret_cast<uint2 *>(hi + (long long)r * cols + c) = h2;
        *reinterpret_cast<uint2 *>(lo + (long long)r * cols + c) = l2;
    }
}

}  // namespace gptaq
