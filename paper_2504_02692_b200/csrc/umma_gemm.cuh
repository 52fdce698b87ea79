// Tensor-core statistics kernel for sm_100a: C += A * B^T with fp16 operands in
// K-major shared-memory tiles (TMA, 128-byte swizzle), tcgen05.mma with fp32
// accumulators in tensor memory, and a read-modify-write epilogue into the fp32
// sums.  Persistent and warp-specialised; the CTAs work in pairs (clusters of
// two, the two SMs of one TPC) on 256 x 256 output tiles with
// tcgen05.mma.cta_group::2: each CTA loads its own 128 rows of the A operand
// and its own 128 of the 256 rows of the B operand into its own shared memory
// (plain TMA loads, no multicast), the tensor cores of both SMs read both halves
// of B, and each CTA's tensor memory receives its 128 rows of the tile.  Per
// K-block a CTA takes in 32 KB of operands for 128 x 256 outputs instead of the
// 48 KB of a single-CTA tile: the L2 -> SM operand traffic, which bounded the
// single-CTA form at 69 % tensor-pipe activity, drops by a third.
// In each CTA warp 0 issues the TMA loads and warps 2-9 drain the accumulators;
// warp 1 owns the TMEM allocation, and in the pair's first CTA its first lane
// issues the MMAs for both.  Two 256-column accumulators are kept in TMEM so
// that draining one overlaps the MMAs into the other.
//
// Every wait on an mbarrier is bounded by a clock limit; when it runs out the
// kernel records GPTAQ_ERR_TIMEOUT in the state header, tells the other CTA of
// the pair, lets outstanding copies land (bounded as well), and both CTAs meet
// at a cluster barrier, free their tensor memory and return.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.cuh"

namespace gptaq {

// UBM x UBN: the output tile of one CTA (float32-grade GEMM: one CTA per tile; statistics: the pair's
// tile is 2 UBM x UBN, one half of the rows per CTA).
constexpr int UBM = 128, UBN = 256, UBK = 64;
constexpr int UPM = 2 * UBM;                    // rows of a pair's tile
constexpr int USTAGES = 6;
constexpr int UA_BYTES = UBM * UBK * 2;         // this CTA's rows of A
constexpr int UB_BYTES = (UBN / 2) * UBK * 2;   // this CTA's half of the rows of B
constexpr int USTAGE_BYTES = UA_BYTES + UB_BYTES;
constexpr int UEPI_WARPS = 8;
constexpr int UMMA_THREADS = 64 + 32 * UEPI_WARPS;
constexpr size_t UMMA_SMEM = (size_t)USTAGES * USTAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds

// fp16 range management: operands are scaled by a power of two when the
// batch's absolute maximum is outside [2^-8, 2^15]; the epilogue undoes it.
__host__ __device__ __forceinline__ float pick_scale(float amax) {
    if (!(amax > 0.f) || !isfinite(amax)) return 1.f;
    if (amax <= 32768.f && amax >= 0.00390625f) return 1.f;
    int e;
    frexpf(amax, &e);                 // amax = f * 2^e, f in [0.5, 1)
    return ldexpf(1.f, 14 - e);       // scaled maximum in [2^13, 2^14)
}

// ---------------------------------------------------------------------------
// Prologue: token-major fp32 X, X~  ->  channel-major (K-major) fp16 X^T and
// (X~ - X)^T with the token dimension zero-padded to kp; the difference is
// taken in fp32 before the down-conversion.  PASS 0 converts with scale 1 and
// records the absolute maxima; PASS 1 redoes the conversion only if a maximum
// fell outside the fp16 comfort range.
// ---------------------------------------------------------------------------
struct ConvertArgs {
    const float *X, *Xfp;
    int64_t ld;
    int tokens, n, kp;
    __half *Xt, *dXt;       // [n][kp]
    __half *Xlo;            // [n][kp] or nullptr: fp16(X - float(fp16(X))), the second term of the split
    __half *dXlo;           // [n][kp] or nullptr: the same for X~ - X
    unsigned *amax;          // [2]: bit patterns of max|X|, max|X~ - X|
};

// Shared-memory staging of one 64-channel x 64-token tile as 32-bit words that
// hold two consecutive tokens of one channel.  Word (c, tp) lives at
// c * 33 + 2 * (c >> 5) + tp: conflict-free both for the transposing stores
// (lanes step 4 channels) and for the row reads (lanes step 4 words).
__device__ __forceinline__ int cvt_word(int c, int tp) { return c * 33 + 2 * (c >> 5) + tp; }
constexpr int CVT_WORDS = 64 * 33 + 4;

// One 64-token x 64-channel tile by one CTA of 256 threads.
template <int PASS>
__device__ __forceinline__ void convert_tile(const ConvertArgs &a, int t0, int c0, float scx, float scd,
                                             uint32_t *sx, uint32_t *sd, uint32_t *sl, uint32_t *sdl) {
    const bool split = a.Xlo != nullptr, splitd = a.dXlo != nullptr;
    const int tid = threadIdx.x;
    float mx = 0.f, md = 0.f;
    bool nan = false;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int idx = tid + it * 256;        // 0..511: 32 token pairs x 16 float4
        const int tp = idx >> 4, cl = (idx & 15) * 4;
        const int c = c0 + cl;
        float x[2][4], f[2][4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int t = t0 + 2 * tp + h;
#pragma unroll
            for (int e = 0; e < 4; ++e) { x[h][e] = 0.f; f[h][e] = 0.f; }
            if (t < a.tokens) {
                const float *px = a.X + (int64_t)t * a.ld + c;
                const float *pf = a.Xfp + (int64_t)t * a.ld + c;
                if (c + 3 < a.n && ((reinterpret_cast<uintptr_t>(px) | reinterpret_cast<uintptr_t>(pf)) & 15) == 0) {
                    float4 vx = __ldcs(reinterpret_cast<const float4 *>(px));
                    float4 vf = __ldcs(reinterpret_cast<const float4 *>(pf));
                    x[h][0] = vx.x; x[h][1] = vx.y; x[h][2] = vx.z; x[h][3] = vx.w;
                    f[h][0] = vf.x; f[h][1] = vf.y; f[h][2] = vf.z; f[h][3] = vf.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (c + e < a.n) { x[h][e] = px[e]; f[h][e] = pf[e]; }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __half hx[2], hd[2], hl[2], hdl[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float xv = x[h][e], d = f[h][e] - xv;
                if (PASS == 0) {
                    mx = fmaxf(mx, fabsf(xv)); md = fmaxf(md, fabsf(d));
                    nan |= (xv != xv) || (d != d);     // fmaxf drops NaNs
                }
                const float xs = xv * scx, ds = d * scd;
                hx[h] = __float2half_rn(xs);
                hd[h] = __float2half_rn(ds);
                hl[h] = __float2half_rn(xs - __half2float(hx[h]));
                hdl[h] = __float2half_rn(ds - __half2float(hd[h]));
            }
            const int w = cvt_word(cl + e, tp);
            sx[w] = (uint32_t)__half_as_ushort(hx[0]) | ((uint32_t)__half_as_ushort(hx[1]) << 16);
            sd[w] = (uint32_t)__half_as_ushort(hd[0]) | ((uint32_t)__half_as_ushort(hd[1]) << 16);
            if (split) sl[w] = (uint32_t)__half_as_ushort(hl[0]) | ((uint32_t)__half_as_ushort(hl[1]) << 16);
            if (splitd) sdl[w] = (uint32_t)__half_as_ushort(hdl[0]) | ((uint32_t)__half_as_ushort(hdl[1]) << 16);
        }
    }
    if (PASS == 0) {
        // block maximum first; the shared word is only touched when it would grow
        __shared__ unsigned bmax[2];
        if (tid == 0) { bmax[0] = 0u; bmax[1] = 0u; }
        __syncthreads();
        unsigned ux = nan ? 0x7fc00000u : __float_as_uint(mx), ud = __float_as_uint(md);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ux = max(ux, __shfl_xor_sync(0xffffffffu, ux, o));
            ud = max(ud, __shfl_xor_sync(0xffffffffu, ud, o));
        }
        if ((tid & 31) == 0) { atomicMax(&bmax[0], ux); atomicMax(&bmax[1], ud); }
        __syncthreads();
        if (tid == 0) {
            if (bmax[0] > *reinterpret_cast<volatile unsigned *>(&a.amax[0])) atomicMax(&a.amax[0], bmax[0]);
            if (bmax[1] > *reinterpret_cast<volatile unsigned *>(&a.amax[1])) atomicMax(&a.amax[1], bmax[1]);
        }
    }
    __syncthreads();
    // 64 channels x 8 chunks of 8 tokens (16 bytes) per matrix
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int idx = tid + it * 256;        // 0..511
        const int cl = idx >> 3, q = idx & 7;
        const int c = c0 + cl, t = t0 + q * 8;
        if (c < a.n && t < a.kp) {
            const int w = cvt_word(cl, q * 4);
            const int64_t off = (int64_t)c * a.kp + t;
            *reinterpret_cast<uint4 *>(a.Xt + off) = make_uint4(sx[w], sx[w + 1], sx[w + 2], sx[w + 3]);
            *reinterpret_cast<uint4 *>(a.dXt + off) = make_uint4(sd[w], sd[w + 1], sd[w + 2], sd[w + 3]);
            if (split) *reinterpret_cast<uint4 *>(a.Xlo + off) = make_uint4(sl[w], sl[w + 1], sl[w + 2], sl[w + 3]);
            if (splitd) *reinterpret_cast<uint4 *>(a.dXlo + off) = make_uint4(sdl[w], sdl[w + 1], sdl[w + 2], sdl[w + 3]);
        }
    }
}

// PASS 0: grid (kp / 64, ceil(n / 64)), one tile per CTA.  PASS 1: any 1-D grid; the CTAs leave at once
// unless a maximum was out of range (the usual case: a short grid keeps that exit cheap), else they
// walk the tiles.
template <int PASS>
__global__ void __launch_bounds__(256) convert_transpose_kernel(ConvertArgs a) {
    __shared__ uint32_t sx[CVT_WORDS];
    __shared__ uint32_t sd[CVT_WORDS];
    __shared__ uint32_t sl[CVT_WORDS];
    __shared__ uint32_t sdl[CVT_WORDS];
    if (PASS == 1) {
        const float scx = pick_scale(__uint_as_float(a.amax[0]));
        const float scd = pick_scale(__uint_as_float(a.amax[1]));
        if (scx == 1.f && scd == 1.f) return;
        const int TX = a.kp / 64, TY = (a.n + 63) / 64;
        for (int tile = blockIdx.x; tile < TX * TY; tile += gridDim.x) {
            convert_tile<1>(a, (tile % TX) * 64, (tile / TX) * 64, scx, scd, sx, sd, sl, sdl);
            __syncthreads();
        }
    } else {
        convert_tile<0>(a, blockIdx.x * 64, blockIdx.y * 64, 1.f, 1.f, sx, sd, sl, sdl);
    }
}

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the clock limit ran out or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit_cycles = WAIT_LIMIT_CYCLES) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- CTA pairs (clusters of two)
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The address, in the cluster's shared-memory window, of the location that has shared::cta address
// `addr` in the CTA with rank `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// try_wait with acquire semantics at cluster scope: what the other CTA of the pair wrote (to this CTA's
// shared memory, or through the commit of its MMAs) before it signalled the barrier is visible afterwards.
__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait of a CTA pair: as mbar_wait, and a wait that gives up also raises the other CTA's flag
// (at cluster address peer_abort), so that the pair winds down together instead of one timeout at a time.
__device__ __forceinline__ bool mbar_wait_pair(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                               uint32_t peer_abort, long long limit_cycles = WAIT_LIMIT_CYCLES) {
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_cluster(bar, parity)) return true;
        if ((it & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > limit_cycles) { *abort_flag = 1; st_cluster_u32(peer_abort, 1u); return false; }
        }
    }
}
// TMA load of one CTA of a pair: the tile lands in this CTA's shared memory, its bytes are counted by the
// mbarrier at cluster address `bar` (the pair's first CTA keeps the barriers of the operand ring).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// One MMA over both CTAs of the pair: D (256 x N, 128 rows in each CTA's tensor memory) += A (128 rows from
// each CTA's shared memory) * B^T (N / 2 rows from each CTA's shared memory); the descriptors address the
// same offsets in both CTAs.
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// Completion of the pair's MMAs issued so far, signalled to the mbarrier at this shared-memory offset in
// both CTAs (the commit's own multicast; no data moves).
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// K-major, 128-byte-swizzled operand tile: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                 // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                 // 128-byte swizzle
    return d;
}

// kind::f16 instruction descriptor: fp16 A and B (both K-major), fp32 D, M = 128, N = 256.
constexpr uint32_t UMMA_IDESC_F16 = (1u << 4) | (0u << 7) | (0u << 10) | ((UBN >> 3) << 17) | ((UBM >> 4) << 24);
// ... and for the pair: M = 256 (128 rows per CTA), N = 256.
constexpr uint32_t UMMA_IDESC_F16_PAIR = (1u << 4) | (0u << 7) | (0u << 10) | ((UBN >> 3) << 17) | ((UPM >> 4) << 24);

struct StatsGemmArgs {
    float *H, *D;            // n x n, ld n
    int n;
    int kblocks;             // kp / 64
    int nseg_h;              // 1: H = hi hi^T;  3: H = hi hi^T + hi lo^T + lo hi^T (split operands)
    int nseg_d;              // 1: dXX^T = dh xh^T;  3: dh xh^T + dh xl^T + dl xh^T
    const unsigned *amax;    // scales are recomputed from the recorded maxima
    StateHeader *hd;
    // Work items of a CTA pair: tiles [0, full_tiles) are whole 256 x 256 tiles; each of the remaining
    // `ntiles - full_tiles` tiles (the last, partial wave) is cut along K into `ksplit` items so that every
    // pair has work.  Item 0 of a cut tile adds into the sums like a whole tile; items c > 0 add their
    // partial result (128 x 256 per CTA) into scratch[(((tile - full_tiles) * (ksplit - 1) + c - 1) * 2 + rank)
    // * UBM * UBN], which the host zeroes before the first launch that uses it; the slots collect the partial
    // sums of all launches with the same cut (one addition per slot entry and launch, in stream order), and
    // stats_fixup_kernel adds them to the sums in a fixed order once, before the sums are read: the result
    // does not depend on timing.
    int ntiles, full_tiles, ksplit;
    float *scratch;
    int d_full;              // 0: only the tiles of dXX^T that reach the diagonal or lie above it (see TileIter)
};

// Tile enumeration shared by all roles, in units of the pair's 256 x 256 tiles.  Rows [0, T) belong to H
// (tiles entirely below the diagonal are not enumerated), rows [T, 2 T) to dXX^T.  Of dXX^T the matrix P
// (Theorem 4.2) uses the entries above the diagonal only -- the mask M_U keeps column j > i of row i of
// dXX^T U^T, and row j of U starts at column j -- so its tiles below the diagonal are enumerated only on
// request (dfull: act_order permutes dXX^T on both sides and needs all of it).  Order: bands of UBAND
// row tiles; inside a band column tile by column tile, first the band's tiles of H, then its tiles of dXX^T.
// The tiles that are in flight together then share about 2 x 8 row panels (X and X~ - X) and a handful
// of column panels of X through the L2, and X streams from HBM once per band instead of once per
// 1.3 row tiles (row-major order over the whole matrix: 15 GB of HBM reads per 8192-token batch at
// n = 14336).
constexpr int UBAND = 8;
struct TileIter {
    int T, r, tn, ord;            // (r, tn): the current tile; ord: its ordinal
    int band, k;                  // band of row tiles, position inside the group (band, tn)
    int dfull;                    // all tiles of dXX^T, not only those with r <= tn
    __host__ __device__ TileIter(int n, int dfull_) : T((n + UPM - 1) / UPM), r(0), tn(0), ord(0), band(0), k(0), dfull(dfull_) {}
    __host__ __device__ int band_rows() const { return min(UBAND, T - band * UBAND); }
    // row tiles r of the band whose tile (r, tn) of H is not entirely below the diagonal: r <= tn
    __host__ __device__ int h_count() const { return max(0, min(band_rows(), tn + 1 - band * UBAND)); }
    __host__ __device__ int d_count() const { return dfull ? band_rows() : h_count(); }
    __host__ __device__ static int total(int n, int dfull_) {
        const int t = (n + UPM - 1) / UPM;
        return t * (t + 1) / 2 + (dfull_ ? t * t : t * (t + 1) / 2);
    }
    // Advances to the tile with ordinal `target` >= ord; false when the list is exhausted.
    __host__ __device__ bool seek_to(int target) {
        int left = target - ord;
        while (band * UBAND < T) {
            const int hc = h_count();
            const int avail = hc + d_count() - k;
            if (left < avail) {
                k += left;
                ord = target;
                r = k < hc ? band * UBAND + k : T + band * UBAND + (k - hc);
                return true;
            }
            left -= avail;
            ord += avail;
            k = 0;
            if (++tn == T) { tn = 0; ++band; }
        }
        return false;
    }
};
static_assert(UBN == UPM, "the diagonal test of TileIter assumes square pair tiles");

// One work item of a pair: a tile and a range of its K-blocks (all segments concatenated).
struct StatsItem {
    int g0, g1;          // K-block range
    int part;            // 0: adds into H / dXX^T;  c > 0: partial result number c of a cut tile
    int cut_index;       // index of the cut tile among the cut tiles
};

__device__ __forceinline__ bool stats_item(const StatsGemmArgs &a, int w, TileIter &it, StatsItem &item) {
    const int nitems = a.full_tiles + (a.ntiles - a.full_tiles) * a.ksplit;
    if (w >= nitems) return false;
    int tile = w, part = 0, parts = 1;
    if (w >= a.full_tiles) {
        const int e = w - a.full_tiles;
        tile = a.full_tiles + e / a.ksplit;
        part = e - (e / a.ksplit) * a.ksplit;
        parts = a.ksplit;
    }
    if (!it.seek_to(tile)) return false;
    const int kb_total = (it.r >= it.T) ? a.kblocks * a.nseg_d : a.kblocks * a.nseg_h;
    item.g0 = (int)((long long)kb_total * part / parts);
    item.g1 = (int)((long long)kb_total * (part + 1) / parts);
    item.part = part;
    item.cut_index = tile - a.full_tiles;
    return true;
}

// Accumulation chains in tensor memory are kept short: the tensor core truncates
// its fp32 accumulator once per MMA, which biases a long sum of like-signed
// products (the diagonal of H) by about 2^-24 per step.  Every UCHUNK K-blocks
// the partial sum is therefore added, with round-to-nearest, into fp32 registers
// of the epilogue warps; HBM is touched once per tile.
constexpr int UCHUNK = 8;           // K-blocks (of 64) per TMEM accumulation chain

// Launched as clusters of two CTAs (grid = 2 x number of pairs).  Tensor maps: X^T, (X~ - X)^T and their
// low parts, [n][kp] fp16, boxes of 64 tokens x 128 channels; they serve as A and as B operand alike.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(UMMA_THREADS, 1)
stats_umma_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapD,
                  const __grid_constant__ CUtensorMap mapL, const __grid_constant__ CUtensorMap mapDL,
                  StatsGemmArgs a) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the swizzled tiles (the same offsets in both CTAs of the pair: the MMA's
    // shared-memory descriptors are applied to both)
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    const uint32_t bar0 = base + USTAGES * USTAGE_BYTES;
    // barrier slots (8 bytes each): full[USTAGES], empty[USTAGES], tfull[2], tempty[2]; then tmem slot, abort flag.
    //   full    first CTA only: its own arrive.expect_tx + the bytes of both CTAs' loads
    //   empty   each CTA its own: one arrival per use, from the commit of the MMAs that read the stage
    //   tfull   each CTA its own: one arrival, from the commit of an accumulation chain
    //   tempty  first CTA only: the epilogue warps of both CTAs
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (USTAGES + s); };
    auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * USTAGES + b); };
    auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * USTAGES + 2 + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(aligned + USTAGES * USTAGE_BYTES + 8 * (2 * USTAGES + 4));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();              // 0: issues the MMAs, keeps full / tempty
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const uint32_t peer_abort = map_to_cta(smem_u32(const_cast<int *>(abort_flag)), rank ^ 1u);
    if (threadIdx.x == 0) {
        for (int s = 0; s < USTAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * UEPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // one warp of each CTA, the same warp in both: the allocation spans the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(const_cast<uint32_t *>(tmem_slot))), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();              // the other CTA's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int KB = a.kblocks;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (each CTA its own halves)
        if (lane == 0) {
            TileIter it(a.n, a.d_full);
            StatsItem item;
            uint32_t stage = 0, phase = 0;
            int issued = 0;
            bool ok = true;
            for (int w = pair; ok && stats_item(a, w, it, item); w += npairs) {
                const bool isD = it.r >= it.T;
                const int row0 = (isD ? it.r - it.T : it.r) * UPM + (int)rank * UBM;      // this CTA's rows of the tile
                const int col0 = it.tn * UBN + (int)rank * (UBN / 2);                     // this CTA's half of the columns' operand
                for (int g = item.g0; g < item.g1; ++g) {
                    const int seg = g / KB, kb = g - seg * KB;
                    const CUtensorMap *mapA = isD ? (seg == 2 ? &mapDL : &mapD) : (seg == 2 ? &mapL : &mapX);
                    const CUtensorMap *mapB = (seg == 1) ? &mapL : &mapX;
                    if (!mbar_wait_pair(empty_bar(stage), phase ^ 1u, abort_flag, peer_abort)) { ok = false; break; }
                    const uint32_t sa = base + stage * USTAGE_BYTES, sb = sa + UA_BYTES;
                    const uint32_t fb = map_to_cta(full_bar(stage), 0u);
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * USTAGE_BYTES);
                    tma_load_2d_pair(sa, mapA, kb * UBK, row0, fb);
                    tma_load_2d_pair(sb, mapB, kb * UBK, col0, fb);
                    ++issued;
                    if (++stage == USTAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // give copies that are still in flight time to land before the CTA exits
                const long long t0 = clock64();
                while (issued > 0 && clock64() - t0 < 4000000LL) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (first CTA of the pair)
        if (lane == 0 && rank == 0) {
            TileIter it(a.n, a.d_full);
            StatsItem item;
            uint32_t stage = 0, phase = 0, ccount = 0;     // ccount: chunks issued so far
            bool ok = true;
            for (int w = pair; ok && stats_item(a, w, it, item); w += npairs) {
                for (int kb0 = item.g0; kb0 < item.g1 && ok; kb0 += UCHUNK) {
                    const uint32_t buf = ccount & 1u, cphase = (ccount >> 1) & 1u;
                    if (!mbar_wait_pair(tempty_bar(buf), cphase ^ 1u, abort_flag, peer_abort)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * UBN;
                    const int kb1 = min(kb0 + UCHUNK, item.g1);
                    for (int kb = kb0; kb < kb1; ++kb) {
                        if (!mbar_wait_pair(full_bar(stage), phase, abort_flag, peer_abort)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sa = base + stage * USTAGE_BYTES, sb = sa + UA_BYTES;
                        const uint64_t ad = make_kmajor_desc(sa), bd = make_kmajor_desc(sb);
#pragma unroll
                        for (int k = 0; k < UBK / 16; ++k)
                            umma_f16_pair(d_tmem, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), UMMA_IDESC_F16_PAIR,
                                          (kb != kb0 || k != 0) ? 1u : 0u);
                        umma_commit_pair(empty_bar(stage));
                        if (++stage == USTAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit_pair(tfull_bar(buf));
                    ++ccount;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9): this CTA's 128 rows
        const int quarter = warp & 3;                 // TMEM lanes 32 * quarter .. + 31
        const int half = (warp - 2) >> 2;             // columns [128 * half, 128 * half + 128)
        TileIter it(a.n, a.d_full);
        StatsItem item;
        uint32_t ccount = 0;
        bool ok = true;
        const float sx = pick_scale(__uint_as_float(a.amax[0]));
        const float sd = pick_scale(__uint_as_float(a.amax[1]));
        float acc[UBN / 2];
        for (int w = pair; ok && stats_item(a, w, it, item); w += npairs) {
            const bool isD = it.r >= it.T;
#pragma unroll
            for (int i = 0; i < UBN / 2; ++i) acc[i] = 0.f;
            for (int kb0 = item.g0; kb0 < item.g1; kb0 += UCHUNK) {
                const uint32_t buf = ccount & 1u, cphase = (ccount >> 1) & 1u;
                if (!mbar_wait_pair(tfull_bar(buf), cphase, abort_flag, peer_abort)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + buf * UBN + half * (UBN / 2) + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
                for (int gq = 0; gq < UBN / 2 / 32; ++gq) {
                    uint32_t v[32];
                    tmem_ld32(taddr + gq * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[gq * 32 + i] += __uint_as_float(v[i]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(buf), 0u));
                ++ccount;
            }
            if (!ok) break;
            const float inv = 1.f / (sx * (isD ? sd : sx));
            if (item.part > 0) {
                // partial result of a cut tile: added into its slot, all 128 x 256 entries
                float *sp = a.scratch + (((int64_t)item.cut_index * (a.ksplit - 1) + item.part - 1) * 2 + (int)rank) * (UBM * UBN) +
                            (quarter * 32 + lane) * UBN + half * (UBN / 2);
#pragma unroll
                for (int q = 0; q < UBN / 2 / 4; ++q)
                    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(sp + 4 * q),
                                 "f"(acc[4 * q + 0] * inv), "f"(acc[4 * q + 1] * inv),
                                 "f"(acc[4 * q + 2] * inv), "f"(acc[4 * q + 3] * inv) : "memory");
                continue;
            }
            const int row = (isD ? it.r - it.T : it.r) * UPM + (int)rank * UBM + quarter * 32 + lane;
            const int col0 = it.tn * UBN + half * (UBN / 2);
            float *C = isD ? a.D : a.H;
            if (row < a.n) {
                float *cp = C + (int64_t)row * a.n + col0;
                if (col0 + UBN / 2 <= a.n && (reinterpret_cast<uintptr_t>(cp) & 15) == 0) {
                    // each element belongs to exactly one CTA per launch: a reduction without
                    // return value is a plain, order-independent "+=" that needs no round trip
#pragma unroll
                    for (int q = 0; q < UBN / 2 / 4; ++q)
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(cp + 4 * q),
                                     "f"(acc[4 * q + 0] * inv), "f"(acc[4 * q + 1] * inv),
                                     "f"(acc[4 * q + 2] * inv), "f"(acc[4 * q + 3] * inv) : "memory");
                } else {
#pragma unroll
                    for (int q = 0; q < UBN / 2; ++q)
                        if (col0 + q < a.n) cp[q] = fmaf(acc[q], inv, cp[q]);
                }
            }
        }
    }

    // Both CTAs leave together: neither frees tensor memory, nor lets its shared memory go, while the
    // other may still signal its barriers or its MMAs read its operands.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (*abort_flag && threadIdx.x == 0) record_status(a.hd, ST_TIMEOUT, blockIdx.x);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Exercises the bounded wait on its own: one warp waits for a barrier phase that nothing will ever
// complete, gives up after `limit_cycles` and records GPTAQ_ERR_TIMEOUT like the GEMM kernels do.
__global__ void bounded_wait_selftest_kernel(StateHeader *hd, long long limit_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_cycles);
    __syncthreads();
    if (!ok && threadIdx.x == 0) record_status(hd, ST_TIMEOUT, 2000000);
}

// Adds the collected partial sums of the cut tiles (see StatsGemmArgs) into H / dXX^T, partial 1 first, then
// 2, ...: FIXUP_SLABS CTAs per cut tile, after the last stats_umma_kernel that used these slots.
constexpr int FIXUP_SLABS = 32;     // CTAs per cut tile, UPM / FIXUP_SLABS rows each
__global__ void __launch_bounds__(256) stats_fixup_kernel(StatsGemmArgs a) {
    TileIter it(a.n, a.d_full);
    if (!it.seek_to(a.full_tiles + blockIdx.x)) return;
    const bool isD = it.r >= it.T;
    const int row0 = (isD ? it.r - it.T : it.r) * UPM, col0 = it.tn * UBN;
    float *C = isD ? a.D : a.H;
    // slot of partial c, CTA rank r: ((blockIdx.x * (ksplit - 1) + c) * 2 + r) * UBM * UBN
    const float *sp = a.scratch + (int64_t)blockIdx.x * (a.ksplit - 1) * 2 * (UBM * UBN);
    constexpr int ROWS = UPM / FIXUP_SLABS;
    const bool vec = (a.n & 3) == 0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0;
#pragma unroll
    for (int it4 = 0; it4 < ROWS * UBN / 4 / 256; ++it4) {
        const int e4 = threadIdx.x + it4 * 256;
        const int i = blockIdx.y * ROWS + e4 / (UBN / 4), j = (e4 % (UBN / 4)) * 4;
        if (row0 + i >= a.n || col0 + j >= a.n) continue;
        float *cp = C + (int64_t)(row0 + i) * a.n + col0 + j;
        const float *pp = sp + (int64_t)(i / UBM) * (UBM * UBN) + (i % UBM) * UBN + j;
        const int64_t pstride = 2 * (int64_t)(UBM * UBN);
        if (vec && col0 + j + 3 < a.n) {
            float4 v = *reinterpret_cast<const float4 *>(cp);
            for (int c = 0; c < a.ksplit - 1; ++c) {
                const float4 p = *reinterpret_cast<const float4 *>(pp + c * pstride);
                v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            }
            *reinterpret_cast<float4 *>(cp) = v;
        } else {
            for (int f = 0; f < 4 && col0 + j + f < a.n; ++f) {
                float v = cp[f];
                for (int c = 0; c < a.ksplit - 1; ++c) v += pp[c * pstride + f];
                cp[f] = v;
            }
        }
    }
}

}  // namespace gptaq
