// A persistent tcgen05 GEMM skeleton for sm_100a: C[M][N] = sum_k A[M][K] * B[N][K], both operands K-major in
// memory, fed by TMA through a ring of mbarrier-guarded stages, accumulated in tensor memory (two buffers, so the
// epilogue of one tile runs under the main loop of the next).  Two instantiations of the arithmetic:
//   TC_TF32  fp32 operands read as TF32, fp32 accumulator (the backward products of Algorithm 1),
//   TC_I8    signed 8-bit operands, int32 accumulator (the unpacked-codes comparison of the forward product).
// Included by the translation units that launch it; everything is in an anonymous namespace.
#pragma once
#include <cuda.h>
#include "qnn_internal.cuh"
#include "mbit_math.cuh"

namespace {

enum TcKind { TC_TF32 = 0, TC_I8 = 1 };

// ------------------------------------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Every wait is bounded: after `limit` failed polls (WAIT_LIMIT unless the caller of the kernel says otherwise) the
// waiter raises the abort flag of its CTA and the global error word, and every role of the CTA leaves its loop at
// its next look at the flag.
constexpr uint32_t WAIT_LIMIT = 1u << 24;

// *err: 0 = no error; else 1 + the id of the wait that gave up first (one device word for the whole library).
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag, unsigned id,
                                          unsigned int *err, uint32_t limit) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(err, 0u, 1u + id);
    return false;
}

// After an abort: lets the copies still in flight land before the CTA's shared memory goes away.  `it` = stage uses
// issued so far; the last min(it, stages) of them may still be under way, each signals full[use % stages].
__device__ __forceinline__ void drain_copies_in_flight(uint64_t *full, long long it, int stages, uint32_t limit) {
    for (long long j = it > stages ? it - stages : 0; j < it; ++j)
        for (uint32_t w = 0; w < limit && !mbar_try_wait(&full[j % stages], (uint32_t)(j / stages) & 1u); ++w) {}
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z, int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t ncols) {   // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {   // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x BN x (32 bytes of K) step issued by a single thread.
template <int KIND>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    if (KIND == TC_TF32)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// 32 consecutive accumulator columns of this thread's row (lane of tensor memory = row of the tile).
__device__ __forceinline__ void tmem_load_32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile written by TMA with the 128-byte swizzle: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, both operands K-major, M = 128, N = BN: accumulator format at bit 4 (1 = fp32, 2 = int32),
// A and B formats at bits 7 and 10 (kind::tf32: 2 = TF32; kind::i8: 1 = signed 8-bit), N/8 at bit 17, M/16 at bit 24.
template <int BN, int KIND>
__host__ __device__ constexpr uint32_t idesc_kmajor() {
    return (KIND == TC_TF32 ? ((1u << 4) | (2u << 7) | (2u << 10)) : ((2u << 4) | (1u << 7) | (1u << 10))) |
           ((uint32_t)(BN >> 3) << 17) | ((128u >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------ the GEMM kernel

constexpr int BM = 128;                 // rows of C per CTA = lanes of tensor memory
constexpr int BK_BYTES = 128;           // bytes of K per stage row = one swizzle span (32 fp32 or 128 int8 elements)
constexpr int MMA_K_BYTES = 32;         // bytes of K one instruction consumes (8 TF32 or 32 int8 elements)
constexpr int EPI_WARPS = 8;            // two warps per quarter of the tensor-memory lanes, alternating 32-column chunks
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;   // warp 0: TMA producer, warp 1: MMA issuer + tensor-memory owner

// Data gradient of a convolution as an implicit GEMM (no patch matrix in memory): result pixel (n, h, w) sums, over the
// taps (r, s) that reach it and over the output features co, g[n][(h + pad - r)/st][(w + pad - s)/st][co] * qw[co][r][s][c].
// Pixels are taken one stride class (h mod st, w mod st) at a time, because all pixels of a class are reached by the
// same taps; the 128 rows of a tile are bn images x bh x bw pixels of the class (powers of two), so that the A operand of
// one (tap, block of 32 features) is ONE 4-D box of g, shifted by the tap; the tensor map fills what lies outside g with
// zeros, which is exactly the contribution of a tap that reaches no output.  B is the tap's weight codes [c][co].
struct ConvGather {
    int enabled;
    int st, pad, R, S;
    int H, W;                           // result (= layer input) image
    int log_bw, log_bh, log_bn;         // tile = 2^log_bn images x 2^log_bh x 2^log_bw pixels of a class
    int tiles_w, tiles_h, tiles_nb;     // tiles per class along w, h and the batch
    int coblocks;                       // blocks of 32 output features (the contraction within a tap)
    int n_images;
};

// Weight gradient of a convolution as an implicit GEMM: GW[co][(r, s), c] = sum over output pixels (n, ho, wo) of
// g[n][ho][wo][co] * qa[n][ho*st - pad + r][wo*st - pad + s][c].  The contraction runs over pixels, so both operands are
// read pixel-contiguous: A from the transposed gradient gt[co][n][ho][j] and B from copies of the transposed activation
// codes in which the stride and the shift along w are baked in: with r - pad = rho + st*q (0 <= rho < st), input row
// ho*st - pad + r = (ho + q)*st + rho, so copy (s, rho) holds, for a' = 0 .. Hq - 1 and j = 0 .. Wq - 1,
//   qas[s*st + rho][c][n][a'][j] = qa[n][(a' + qmin)*st + rho][j*st - pad + s][c]      (zero outside the image),
// qmin = floor(-pad / st), Hq = Ho + floor((R - 1 - pad) / st) - qmin.  Rows of both operands hold Wq >= Wo columns (Wo
// rounded up to 4, the extra columns of gt zero), and (row, column) is ONE index p = row*Wq + j: a block of the
// contraction is 32 consecutive p of one image, and tap (r, s) is copy (s, rho) read at p + (q - qmin)*Wq -- a multiple
// of 4 elements, as the 16-byte rule for the start of a TMA box along its innermost dimension demands (which is why
// the shift along w lives in the copies while the shift along h is free).  For stride 1 there are S copies of the
// padded image.  A tile of the result = 128 output features x up to BN channels of ONE tap.
struct ConvWeightGather {
    int enabled;
    int C, S, st, pad, qmin;
    int tiles_c;                        // channel tiles per tap
    int Wq;                             // columns per stored row
    int kb_per_image;                   // blocks of the contraction per image: ceil(Ho*Wq / 32)
};

struct GemmParams {
    int M, N, K;                        // C[M][N] = alpha * sum_k A[M][K] * B[N][K]
    float alpha;
    float *C;                           // fp32 result (TC_I8: optional, float(acc) * alpha)
    long long ldc;
    int *acc;                           // TC_I8 only, optional: the int32 accumulators [M][N], leading dimension ldc
    unsigned int *err;                  // device word that records a wait that gave up
    const float *x;                     // optional [M][N] (leading dimension ldx): fuse Eq. 12 with `bits` planes and range r
    long long ldx;
    int bits;
    float r;
    MbitPlaneConsts enc;                // constants of Eq. 12 for `bits` planes
    int tiles_n, tiles;
    int whole_items, items;             // work items: tiles [0, whole_items) whole, the rest split into two halves along N
    // Split contraction (ksplit > 1; for products with few output tiles and a long K): work item w = tile * ksplit + s
    // contracts K blocks [s * kb_per_split, (s + 1) * kb_per_split) and writes alpha times its partial product to
    // C + s * split_stride (dense partial buffers); sum_partials_kernel then adds the ksplit buffers in index order.
    int ksplit, kb_per_split;
    long long split_stride;
    unsigned int wait_limit;            // polls after which a wait on an arrival gives up (0 = WAIT_LIMIT)
    ConvGather conv;                    // enabled: A is gathered from the gradient image, rows of C are pixels (see above)
    ConvWeightGather wconv;             // enabled: the contraction runs over the pixels of a convolution (see above)
};

// floor(a / b) and whether b divides a, for b > 0 and any sign of a
__device__ __forceinline__ bool exact_div(int a, int b, int &q) {
    q = a >= 0 ? a / b : -((-a + b - 1) / b);
    return q * b == a;
}

// One tile of the convolution's data gradient: stride class, first image / class row / class column, channel tile.
struct ConvTile {
    int ph, pw, n0, a0, b0, c0;
    int nkb;                            // K blocks: (taps of the class) x coblocks
};
template <int BN>
__device__ __forceinline__ ConvTile conv_tile(int tile, const GemmParams &p) {
    const ConvGather &c = p.conv;
    ConvTile t;
    const int ct = tile % p.tiles_n;
    int mt = tile / p.tiles_n;
    t.c0 = ct * BN;
    const int wb = mt % c.tiles_w; mt /= c.tiles_w;
    const int hb = mt % c.tiles_h; mt /= c.tiles_h;
    const int nb = mt % c.tiles_nb; mt /= c.tiles_nb;
    t.pw = mt % c.st;
    t.ph = mt / c.st;
    t.b0 = wb << c.log_bw; t.a0 = hb << c.log_bh; t.n0 = nb << c.log_bn;
    int th = 0, tw = 0, q;
    for (int r = 0; r < c.R; ++r) th += exact_div(t.ph + c.pad - r, c.st, q) ? 1 : 0;
    for (int s = 0; s < c.S; ++s) tw += exact_div(t.pw + c.pad - s, c.st, q) ? 1 : 0;
    t.nkb = th * tw * c.coblocks;
    return t;
}
// Offset (in rows of C / x) of tile row `row`, or -1 when the row lies outside the image or the batch.
__device__ __forceinline__ long long conv_row(const ConvTile &t, int row, const GemmParams &p) {
    const ConvGather &c = p.conv;
    const int dw = row & ((1 << c.log_bw) - 1);
    const int dh = (row >> c.log_bw) & ((1 << c.log_bh) - 1);
    const int dn = row >> (c.log_bw + c.log_bh);
    const int n = t.n0 + dn, h = (t.a0 + dh) * c.st + t.ph, w = (t.b0 + dw) * c.st + t.pw;
    if (n >= c.n_images || h >= c.H || w >= c.W) return -1;
    return ((long long)n * c.H + h) * c.W + w;
}

// One column of a 32 x 32 chunk (this lane's), rows_here rows: C = Eq. 12 applied to the staged products and x.
// Four rows are in flight at a time; the element arithmetic has no branch, so their instructions interleave.
template <int BITS>
__device__ __forceinline__ void epilogue_encoder(float *cptr, long long ldc, const float *xptr, long long ldx,
                                                 const float *stage_col, int rows_here, float r, const MbitPlaneConsts &c) {
    int rr = 0;
#pragma unroll 1
    for (; rr + 4 <= rows_here; rr += 4) {
        float xv[4], o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) xv[e] = __ldcs(xptr + (long long)(rr + e) * ldx);
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = mbit_backward_shared<BITS>(xv[e], r, stage_col[(rr + e) * 33], c);
#pragma unroll
        for (int e = 0; e < 4; ++e) cptr[(long long)(rr + e) * ldc] = o[e];
    }
    for (; rr < rows_here; ++rr)
        cptr[(long long)rr * ldc] = mbit_backward_shared<BITS>(__ldcs(xptr + (long long)rr * ldx), r, stage_col[rr * 33], c);
}

// Convolution data gradient: one column (this lane's) of a 32 x 32 chunk whose rows are tile rows row0 .. row0 + 31;
// BITS > 0 applies Eq. 12 with x read at the same pixel.
template <int BITS>
__device__ __forceinline__ void conv_epilogue_rows(const ConvTile &t, int row0, const GemmParams &p, int col, const float *stage_col) {
#pragma unroll 4
    for (int rr = 0; rr < 32; ++rr) {
        const long long pix = conv_row(t, row0 + rr, p);
        if (pix < 0) continue;
        float v = t.nkb ? stage_col[rr * 33] : 0.0f;      // a stride class that no tap reaches: nothing was accumulated
        if constexpr (BITS > 0) v = mbit_backward_shared<BITS>(__ldcs(p.x + pix * p.ldx + col), p.r, v, p.enc);
        p.C[pix * p.ldc + col] = v;
    }
}

// Work item w of a launch: whole tiles first; the tiles of a ragged last round (fewer than half as many as there are
// CTAs) are split into two halves along N so that the round takes about half a tile's time instead of a whole one.
struct WorkItem {
    int m0, n0, width;
    int kb0, kb1, split;                // K blocks [kb0, kb1) of this item; index of its partial buffer
    int n_end;                          // columns of C from here on are not this tile's
};
template <int BN>
__device__ __forceinline__ WorkItem work_item(int w, const GemmParams &p, int nkb) {
    int tile = w, off = 0, width = BN;
    if (p.ksplit > 1) {
        // items that contract the same range of K blocks are neighbours (they run at the same time and read the same
        // slices of both operands through L2)
        const int sp = w / p.tiles;
        tile = w - sp * p.tiles;
        const int kb0 = sp * p.kb_per_split;
        const int nt = tile % p.tiles_n;
        if (p.wconv.enabled) {                                      // column tile nt = (tap, channel tile)
            const int tap = nt / p.wconv.tiles_c, c0 = (nt - tap * p.wconv.tiles_c) * BN;
            return {(tile / p.tiles_n) * BM, tap * p.wconv.C + c0, BN, kb0, min(nkb, kb0 + p.kb_per_split), sp,
                    tap * p.wconv.C + min(p.wconv.C, c0 + BN)};
        }
        return {(tile / p.tiles_n) * BM, nt * BN, BN, kb0, min(nkb, kb0 + p.kb_per_split), sp, p.N};
    }
    if (p.wconv.enabled) {
        const int nt = tile % p.tiles_n;
        const int tap = nt / p.wconv.tiles_c, c0 = (nt - tap * p.wconv.tiles_c) * BN;
        return {(tile / p.tiles_n) * BM, tap * p.wconv.C + c0, BN, 0, nkb, 0, tap * p.wconv.C + min(p.wconv.C, c0 + BN)};
    }
    if (w >= p.whole_items) {
        const int r = w - p.whole_items;
        tile = p.whole_items + (r >> 1);
        off = (r & 1) * (BN / 2);
        width = BN / 2;
    }
    return {(tile / p.tiles_n) * BM, (tile % p.tiles_n) * BN + off, width, 0, nkb, 0, p.N};
}

template <int BN, int STAGES>
struct GemmSmem {
    static constexpr int A_BYTES = BM * BK_BYTES;
    static constexpr int B_BYTES = BN * BK_BYTES;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int EPI_OFFSET = STAGES * STAGE_BYTES;                       // per epilogue warp a 32 x 33 fp32 tile
    static constexpr int BAR_OFFSET = EPI_OFFSET + EPI_WARPS * 32 * 33 * 4;
    static constexpr int TOTAL = BAR_OFFSET + (2 * STAGES + 4) * 8 + 16 + 1024;   // + slack for the 1024-byte alignment
};

// Persistent: CTA b works on tiles b, b + gridDim.x, ...  The accumulator is double-buffered in tensor memory
// (2 x BN columns), so the epilogue of one tile runs under the main loop of the next.
template <int BN, int STAGES, int KIND>
__global__ void __launch_bounds__(GEMM_THREADS, 1) tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                 const __grid_constant__ CUtensorMap map_b,
                                                                 const __grid_constant__ CUtensorMap map_b_half,
                                                                 const GemmParams p) {
    using L = GemmSmem<BN, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L::BAR_OFFSET);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;          // [2]: the MMAs of a tile have retired
    uint64_t *acc_empty = acc_full + 2;           // [2]: the epilogue has read the buffer out
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int BK = BK_BYTES / (KIND == TC_TF32 ? 4 : 1);   // elements of K per stage
    const int nkb = (p.K + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], EPI_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(tmem_slot, 2 * BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    int committed = 0;                  // MMA issuer: tiles whose accumulator has been committed to acc_full

    if (warp == 0) {
        if (lane == 0) {
            long long it = 0;                                 // stage uses so far, over all tiles
            int s = 0;                                        // ring position it % STAGES and parity of it / STAGES, kept
            uint32_t ph = 0;                                  // incrementally (this one thread's instructions are the pace)
            auto advance = [&]() {
                ++it;
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            };
            for (int w = blockIdx.x; w < p.items && !*abort_flag; w += gridDim.x) {
                if (KIND == TC_TF32 && p.conv.enabled) {
                    // implicit gather: per tap of the tile's stride class and block of 32 output features, one 4-D box
                    // of the gradient image shifted by the tap (zero outside it) and the tap's weight codes
                    const ConvTile t = conv_tile<BN>(w, p);
                    for (int r = 0; r < p.conv.R && !*abort_flag; ++r) {
                        int dr, ds;
                        if (!exact_div(t.ph + p.conv.pad - r, p.conv.st, dr)) continue;
                        for (int sx = 0; sx < p.conv.S && !*abort_flag; ++sx) {
                            if (!exact_div(t.pw + p.conv.pad - sx, p.conv.st, ds)) continue;
                            const int tap = r * p.conv.S + sx, wx = t.b0 + ds, hy = t.a0 + dr;
                            for (int cb = 0; cb < p.conv.coblocks; ++cb) {
                                if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag, 0, p.err, p.wait_limit)) break;
                                mbar_expect_tx(&full[s], L::STAGE_BYTES);
                                tma_load_4d(smem + s * L::STAGE_BYTES, &map_a, &full[s], cb * BK, wx, hy, t.n0);
                                tma_load_3d(smem + s * L::STAGE_BYTES + L::A_BYTES, &map_b, &full[s], cb * BK, t.c0, tap);
                                advance();
                            }
                        }
                    }
                    continue;
                }
                const WorkItem wi = work_item<BN>(w, p, nkb);
                if (KIND == TC_TF32 && p.wconv.enabled) {
                    // block kb of the contraction = (image n, block pb of its pixels), walked incrementally
                    const ConvWeightGather &c = p.wconv;
                    const int tap = wi.n0 / c.C, cbase = wi.n0 - tap * c.C;
                    const int r = tap / c.S, sx = tap - r * c.S;
                    int q;                                                        // r - pad = rho + st*q
                    exact_div(r - c.pad, c.st, q);
                    const int rho = r - c.pad - q * c.st;
                    const int shift = (q - c.qmin) * c.Wq, copy = sx * c.st + rho;
                    int n = wi.kb0 / c.kb_per_image, pb = wi.kb0 - n * c.kb_per_image;
                    for (int kb = wi.kb0; kb < wi.kb1; ++kb) {
                        if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag, 0, p.err, p.wait_limit)) break;
                        mbar_expect_tx(&full[s], L::STAGE_BYTES);
                        tma_load_3d(smem + s * L::STAGE_BYTES, &map_a, &full[s], pb * BK, n, wi.m0);
                        tma_load_4d(smem + s * L::STAGE_BYTES + L::A_BYTES, &map_b, &full[s], pb * BK + shift, n, cbase, copy);
                        advance();
                        if (++pb == c.kb_per_image) { pb = 0; ++n; }
                    }
                    continue;
                }
                const bool whole = wi.width == BN;
                for (int kb = wi.kb0; kb < wi.kb1; ++kb) {
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag, 0, p.err, p.wait_limit)) break;
                    mbar_expect_tx(&full[s], whole ? L::STAGE_BYTES : L::A_BYTES + L::B_BYTES / 2);
                    tma_load_2d(smem + s * L::STAGE_BYTES, &map_a, &full[s], kb * BK, wi.m0);
                    tma_load_2d(smem + s * L::STAGE_BYTES + L::A_BYTES, whole ? &map_b : &map_b_half, &full[s], kb * BK, wi.n0);
                    advance();
                }
            }
            if (*abort_flag) drain_copies_in_flight(full, it, STAGES, p.wait_limit);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int s = 0;                                        // ring position and phase, as in the producer
            uint32_t ph = 0;
            int local = 0;
            for (int w = blockIdx.x; w < p.items && !*abort_flag; w += gridDim.x, ++local) {
                WorkItem wi;
                if (KIND == TC_TF32 && p.conv.enabled) wi = WorkItem{0, 0, BN, 0, conv_tile<BN>(w, p).nkb, 0, p.N};
                else wi = work_item<BN>(w, p, nkb);
                const uint32_t idesc = wi.width == BN ? idesc_kmajor<BN, KIND>() : idesc_kmajor<BN / 2, KIND>();
                const int buf = local & 1;
                if (!mbar_wait(&acc_empty[buf], ((uint32_t)(local >> 1) & 1u) ^ 1u, abort_flag, 3, p.err, p.wait_limit)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = wi.kb0; kb < wi.kb1; ++kb) {
                    if (!mbar_wait(&full[s], ph, abort_flag, 1, p.err, p.wait_limit)) break;
                    tc_fence_after();
                    const uint64_t a_desc = smem_desc_k_sw128(smem_u32(smem + s * L::STAGE_BYTES));
                    const uint64_t b_desc = smem_desc_k_sw128(smem_u32(smem + s * L::STAGE_BYTES + L::A_BYTES));
#pragma unroll
                    for (int j = 0; j < BK_BYTES / MMA_K_BYTES; ++j)   // 32 bytes along K per step = 2 descriptor address units
                        tc_mma<KIND>(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, ((kb - wi.kb0) | j) != 0 ? 1u : 0u);
                    tc_commit(&empty[s]);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                tc_commit(&acc_full[buf]);
                committed = local + 1;
            }
        }
    } else {
        const int q = warp & 3;                            // a warp reaches the 32 lanes [32*(warp%4), +32) only
        const int half = (warp - 2) >> 2;                  // which of the two warps of this quarter
        int local = 0;
        for (int w = blockIdx.x; w < p.items; w += gridDim.x, ++local) {
            const bool conv = KIND == TC_TF32 && p.conv.enabled;
            ConvTile ct = {};
            WorkItem wi;
            if (conv) {
                ct = conv_tile<BN>(w, p);
                wi = WorkItem{0, ct.c0, BN, 0, ct.nkb, 0, p.N};
            } else {
                wi = work_item<BN>(w, p, nkb);
            }
            const int m0 = wi.m0, n0 = wi.n0;
            const int buf = local & 1;
            // every lane polls (each needs the barrier's acquire), but the warp must reach the warp-wide
            // tensor-memory load together or not at all: one lane giving up makes all of them leave
            if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[buf], (uint32_t)(local >> 1) & 1u, abort_flag, 2, p.err, p.wait_limit)))
                break;
            tc_fence_after();
            // Each 32 x 32 chunk goes through the warp's shared tile: tensor memory hands a thread one row, memory
            // wants a warp on one row, so that every access to C and x is a whole 128-byte line.
            float *stage = reinterpret_cast<float *>(smem + L::EPI_OFFSET) + (warp - 2) * (32 * 33);
#pragma unroll 1
            for (int c0 = half * 32; c0 < wi.width; c0 += 64) {
                if (n0 + c0 >= wi.n_end) break;            // uniform over the warp
                uint32_t v[32];
                tmem_load_32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
                const int col = n0 + c0 + lane;
                const int rows_here = min(32, p.M - (m0 + q * 32));
                if (KIND == TC_I8) {
                    int *istage = reinterpret_cast<int *>(stage);
#pragma unroll
                    for (int i = 0; i < 32; ++i) istage[lane * 33 + i] = (int)v[i];
                    __syncwarp();
                    if (col < wi.n_end) {
                        const long long off = (long long)(m0 + q * 32) * p.ldc + col;
#pragma unroll 8
                        for (int rr = 0; rr < rows_here; ++rr) {
                            const int a = istage[rr * 33 + lane];
                            if (p.acc) p.acc[off + (long long)rr * p.ldc] = a;
                            if (p.C) p.C[off + (long long)rr * p.ldc] = __fmul_rn((float)a, p.alpha);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) stage[lane * 33 + i] = __fmul_rn(__uint_as_float(v[i]), p.alpha);
                    __syncwarp();
                    if (conv) {
                        // rows of the tile are pixels of a stride class: each row has its own place in the result
                        if (col < wi.n_end) {
                            switch (p.x ? p.bits : 0) {
                                case 0: conv_epilogue_rows<0>(ct, q * 32, p, col, stage + lane); break;
                                case 1: conv_epilogue_rows<1>(ct, q * 32, p, col, stage + lane); break;
                                case 2: conv_epilogue_rows<2>(ct, q * 32, p, col, stage + lane); break;
                                case 3: conv_epilogue_rows<3>(ct, q * 32, p, col, stage + lane); break;
                                case 4: conv_epilogue_rows<4>(ct, q * 32, p, col, stage + lane); break;
                                case 5: conv_epilogue_rows<5>(ct, q * 32, p, col, stage + lane); break;
                                case 6: conv_epilogue_rows<6>(ct, q * 32, p, col, stage + lane); break;
                                case 7: conv_epilogue_rows<7>(ct, q * 32, p, col, stage + lane); break;
                                default: conv_epilogue_rows<8>(ct, q * 32, p, col, stage + lane); break;
                            }
                        }
                    } else if (col < wi.n_end) {
                        float *cptr = p.C + (long long)wi.split * p.split_stride + (long long)(m0 + q * 32) * p.ldc + col;
                        if (p.x) {
                            const float *xptr = p.x + (long long)(m0 + q * 32) * p.ldx + col;
                            switch (p.bits) {
                                case 1: epilogue_encoder<1>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 2: epilogue_encoder<2>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 3: epilogue_encoder<3>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 4: epilogue_encoder<4>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 5: epilogue_encoder<5>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 6: epilogue_encoder<6>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                case 7: epilogue_encoder<7>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                                default: epilogue_encoder<8>(cptr, p.ldc, xptr, p.ldx, stage + lane, rows_here, p.r, p.enc); break;
                            }
                        } else {
#pragma unroll 8
                            for (int rr = 0; rr < rows_here; ++rr) cptr[(long long)rr * p.ldc] = stage[rr * 33 + lane];
                        }
                    }
                }
                __syncwarp();
            }
            // the buffer is free once every epilogue warp has read its part out
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&acc_empty[buf])) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // every MMA that was issued has retired once the last committed tile's barrier has completed its phase
        // (a tile that an abort cut short is committed too, with whatever was issued for it, so this covers it)
        if (lane == 0 && committed > 0) {
            const int last = committed - 1;
            for (uint32_t w = 0; w < p.wait_limit && !mbar_try_wait(&acc_full[last & 1], (uint32_t)(last >> 1) & 1u); ++w) {}
        }
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
    }
}


// ------------------------------------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(ptr);
    }();
    return fn;
}

// Tensor map of a row-major matrix [rows][cols] of 4-byte (TC_TF32) or 1-byte (TC_I8) elements with leading
// dimension ld (elements), box = 128 bytes of a row x box_rows rows, 128-byte swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap *map, const void *base, long long rows, long long cols, long long ld, int box_rows, int kind) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const int esz = kind == TC_TF32 ? 4 : 1;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
    cuuint32_t box[2] = {(cuuint32_t)(BK_BYTES / esz), (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, kind == TC_TF32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
              const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of an fp32 tensor of `rank` dimensions (innermost first): dims in elements, strides of dimensions 1.. in
// elements, box = 32 elements (128 bytes) x box[1..], 128-byte swizzle, zero fill outside the tensor.
bool make_map_nd(CUtensorMap *map, const void *base, int rank, const long long *dims, const long long *strides_elems,
                 const int *box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || rank < 2 || rank > 5) return false;
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; ++i) {
        d[i] = (cuuint64_t)dims[i];
        b[i] = (cuuint32_t)box[i];
        es[i] = 1;
        if (i > 0) st[i - 1] = (cuuint64_t)strides_elems[i - 1] * 4u;
    }
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<void *>(base), d, st, b, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

long long pad32(long long v) { return (v + 31) / 32 * 32; }

template <int BN, int STAGES, int KIND>
int launch_gemm(const CUtensorMap &map_a, const CUtensorMap &map_b, const CUtensorMap &map_b_half, GemmParams p, int sms,
                cudaStream_t st) {
    using L = GemmSmem<BN, STAGES>;
    // the attribute belongs to the (function, device) pair: set it on every launch, for whichever device is current
    if (cudaFuncSetAttribute(tc_gemm_kernel<BN, STAGES, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL) !=
        cudaSuccess)
        return QNN_E_CUDA;
    if (p.wait_limit == 0) p.wait_limit = WAIT_LIMIT;
    const long long tiles_m = (p.M + BM - 1) / BM;
    const long long tiles_n = p.wconv.enabled ? p.tiles_n : (p.N + BN - 1) / BN;   // (taps x channel tiles, set by the caller)
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return QNN_E_ARG;
    p.tiles_n = (int)tiles_n;
    p.tiles = (int)(tiles_m * tiles_n);
    int grid = p.tiles < sms ? p.tiles : sms;
    if (p.ksplit > 1) {
        if ((long long)p.tiles * p.ksplit > 0x7FFFFFFFll) return QNN_E_ARG;
        p.whole_items = p.items = p.tiles * p.ksplit;
        grid = p.items < sms ? p.items : sms;
    } else {
        p.ksplit = 1;
        const int rem = p.tiles % grid;
        const bool split = !p.conv.enabled && !p.wconv.enabled && rem > 0 && 2 * rem <= grid;
        p.whole_items = split ? p.tiles - rem : p.tiles;
        p.items = split ? p.tiles + rem : p.tiles;
    }
    tc_gemm_kernel<BN, STAGES, KIND><<<grid, GEMM_THREADS, L::TOTAL, st>>>(map_a, map_b, map_b_half, p);
    return qnn_launch_status();
}

// SM count of the current device (asked every time: a process may use several devices).
int sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return 0;
    return sms;
}

// C[M][N] = alpha * A[M][K] * B[N][K]^T.  lda / ldb in elements; rows must be 16-byte multiples.  128 x 256 tiles when
// they give every SM a tile (they read each A tile from shared memory half as often per flop as 128 x 128 ones, which
// a single CTA per SM cannot feed fast enough), 128 x 128 tiles otherwise.
template <int KIND>
int run_gemm(const void *A, long long lda, const void *B, long long ldb, GemmParams p, cudaStream_t st) {
    const int esz = KIND == TC_TF32 ? 4 : 1;
    if (p.M <= 0 || p.N <= 0 || p.K <= 0 || !p.err) return QNN_E_ARG;
    if (!qnn_aligned(A, 16) || !qnn_aligned(B, 16) || (lda * esz) % 16 || (ldb * esz) % 16) return QNN_E_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return QNN_E_CUDA;
    // a split contraction is planned for 128 x 128 tiles (gemm_ksplit) and keeps them
    const bool wide = p.ksplit <= 1 && ((long long)(p.M + BM - 1) / BM) * ((p.N + 255) / 256) >= sms;
    CUtensorMap map_a, map_b, map_b_half;
    if (!make_map(&map_a, A, p.M, p.K, lda, BM, KIND) || !make_map(&map_b, B, p.N, p.K, ldb, wide ? 256 : 128, KIND) ||
        !make_map(&map_b_half, B, p.N, p.K, ldb, wide ? 128 : 64, KIND))
        return QNN_E_CUDA;
    return wide ? launch_gemm<256, 4, KIND>(map_a, map_b, map_b_half, p, sms, st)
                : launch_gemm<128, 6, KIND>(map_a, map_b, map_b_half, p, sms, st);
}

int ceil_log2(long long v) {
    int l = 0;
    while ((1ll << l) < v) ++l;
    return l;
}

// Data gradient of a convolution (see ConvGather): result[n][h][w][c] = alpha * sum over taps and co of
// g[n][(h + pad - r)/st][(w + pad - s)/st][co] * wq[r*S + s][c][co], optionally through Eq. 12 (p.x, p.bits, p.r, p.enc).
//   g    fp32 [N][Ho][Wo][ldg] (ldg >= Cout, a multiple of 4), 16-byte aligned
//   wq   fp32 [R*S][C][ldw]    (ldw >= Cout, a multiple of 4), 16-byte aligned: the weight codes, tap-major
// p carries alpha, C (the result, ldc), x / ldx / bits / r / enc and err; the rest is filled in here.
int run_conv_data_gradient(const float *g, long long ldg, const float *wq, long long ldw, int N, int H, int W, int C, int Cout,
                           int R, int S, int stride, int pad, int Ho, int Wo, GemmParams p, cudaStream_t st) {
    if (!p.err || !qnn_aligned(g, 16) || !qnn_aligned(wq, 16) || ldg % 4 || ldw % 4) return QNN_E_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return QNN_E_CUDA;
    // tile = 2^bn images x 2^bh x 2^bw pixels of one stride class (128 rows): the shape that wastes the fewest rows,
    // among equals the one with the longest runs along w, then h (measured: the shape itself does not change the time)
    const long long Wa = (W + stride - 1) / stride, Ha = (H + stride - 1) / stride;
    int best_bw = 0, best_bh = 0;
    double best = -1.0;
    for (int lw = 7; lw >= 0; --lw)
        for (int lh = 7 - lw; lh >= 0; --lh) {
            const int ln = 7 - lw - lh;
            const double e = (double)Wa / (double)(((Wa + (1 << lw) - 1) >> lw) << lw) *
                             (double)Ha / (double)(((Ha + (1 << lh) - 1) >> lh) << lh) *
                             (double)N / (double)((((long long)N + (1 << ln) - 1) >> ln) << ln);
            if (e > best + 1e-9) { best = e; best_bw = lw; best_bh = lh; }
        }
    ConvGather &c = p.conv;
    c.enabled = 1; c.st = stride; c.pad = pad; c.R = R; c.S = S; c.H = H; c.W = W; c.n_images = N;
    c.log_bw = best_bw; c.log_bh = best_bh; c.log_bn = 7 - best_bw - best_bh;
    c.tiles_w = (int)((Wa + (1 << c.log_bw) - 1) >> c.log_bw);
    c.tiles_h = (int)((Ha + (1 << c.log_bh) - 1) >> c.log_bh);
    c.tiles_nb = (int)(((long long)N + (1 << c.log_bn) - 1) >> c.log_bn);
    c.coblocks = (Cout + 31) / 32;
    const long long mtiles = (long long)stride * stride * c.tiles_nb * c.tiles_h * c.tiles_w;
    if (mtiles * BM > 0x7FFFFFFFll) return QNN_E_RANGE;
    p.M = (int)(mtiles * BM); p.N = C; p.K = 0;
    p.ksplit = 1;
    // tile width: the narrowest of 64 / 128 / 256 channels that covers C (256 only when that still gives every SM a
    // tile); columns beyond C would be multiplied for nothing
    const int bn = C <= 64 ? 64 : ((C <= 128 || mtiles * ((C + 255) / 256) < sms) ? 128 : 256);
    const long long gdims[4] = {Cout, Wo, Ho, N}, gstr[3] = {ldg, (long long)Wo * ldg, (long long)Ho * Wo * ldg};
    const int gbox[4] = {32, 1 << c.log_bw, 1 << c.log_bh, 1 << c.log_bn};
    const long long wdims[3] = {Cout, C, (long long)R * S}, wstr[2] = {ldw, (long long)C * ldw};
    const int wbox[3] = {32, bn, 1};
    CUtensorMap map_a, map_b;
    if (!make_map_nd(&map_a, g, 4, gdims, gstr, gbox) || !make_map_nd(&map_b, wq, 3, wdims, wstr, wbox)) return QNN_E_CUDA;
    return bn == 256 ? launch_gemm<256, 4, TC_TF32>(map_a, map_b, map_b, p, sms, st)
         : bn == 128 ? launch_gemm<128, 6, TC_TF32>(map_a, map_b, map_b, p, sms, st)
                     : launch_gemm<64, 8, TC_TF32>(map_a, map_b, map_b, p, sms, st);
}

// Weight gradient of a convolution (see ConvWeightGather): gw[co][(r*S + s)*C + c] = alpha * sum over output pixels of
// gt[co][n][ho][j] * (copy (s, rho(r)) of the codes read (q(r) - qmin) rows further down).
//   gt   fp32 [Cout][N][Ho][Wq], qas fp32 [S*stride][C][N][Hq][Wq] (conv_wgrad_plan), padding columns zero; 16-byte aligned
//   split_ws: partial products when the contraction is split over the CTAs (conv_wgrad_split_workspace bytes)
struct ConvWgradPlan {
    int Wq, Hq, qmin, kb_per_image, bn, tiles_c, ksplit, kb_per_split;
    long long nkb;
};
int floor_div(int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }

ConvWgradPlan conv_wgrad_plan(int N, int C, int Cout, int R, int S, int stride, int pad, int Ho, int Wo) {
    ConvWgradPlan pl;
    pl.Wq = (Wo + 3) / 4 * 4;
    pl.qmin = floor_div(-pad, stride);
    pl.Hq = Ho + floor_div(R - 1 - pad, stride) - pl.qmin;
    pl.kb_per_image = (int)(((long long)Ho * pl.Wq + 31) / 32);
    pl.nkb = (long long)N * pl.kb_per_image;
    pl.bn = C <= 64 ? 64 : (C <= 128 ? 128 : 256);
    pl.tiles_c = (C + pl.bn - 1) / pl.bn;
    // at most about two work items per SM (sized for 148 SMs so that workspace queries and calls agree), at least
    // four blocks each; among those the fewest parts whose rounds are within 3 % of the best filled (every part
    // writes, and the sum re-reads, one partial result)
    const long long tiles = (((long long)Cout + BM - 1) / BM) * R * S * pl.tiles_c;
    long long most = (2 * 148) / tiles;
    if (most > pl.nkb / 4) most = pl.nkb / 4;
    if (most > 64) most = 64;
    auto fill = [&](long long parts) {
        const long long items = tiles * parts;
        return (double)items / (double)((items + 147) / 148 * 148);
    };
    double best = 0.0;
    for (long long parts = 1; parts <= most; ++parts) best = fill(parts) > best ? fill(parts) : best;
    long long want = 1;
    while (want < most && fill(want) < best - 0.03) ++want;
    if (want < 2) {
        pl.ksplit = 1; pl.kb_per_split = (int)pl.nkb;
    } else {
        const long long per = (pl.nkb + want - 1) / want;
        pl.kb_per_split = (int)per;
        pl.ksplit = (int)((pl.nkb + per - 1) / per);
    }
    return pl;
}
size_t conv_wgrad_split_workspace(int N, int C, int Cout, int R, int S, int stride, int pad, int Ho, int Wo) {
    const ConvWgradPlan pl = conv_wgrad_plan(N, C, Cout, R, S, stride, pad, Ho, Wo);
    return pl.ksplit > 1 ? (size_t)pl.ksplit * (size_t)Cout * (size_t)R * S * C * sizeof(float) : 0;
}

// C[i][j] = sum over s (in increasing order: a fixed summation order) of part[s][i][j]; dense partial buffers [M][N].
__global__ void __launch_bounds__(256) sum_partials_kernel(const float *__restrict__ part, int ksplit, long long stride,
                                                          long long M, long long N, float *__restrict__ C, long long ldc) {
    const long long total = M * N;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
        float sum = part[i];
        for (int sp = 1; sp < ksplit; ++sp) sum = __fadd_rn(sum, part[(long long)sp * stride + i]);
        C[(i / N) * ldc + i % N] = sum;
    }
}

// How many ways to split the contraction of an M x N x K TF32 product so that about two work items per SM exist
// (sized for 148 SMs, independent of the device so that workspace queries and calls agree): 1 when the output
// already has that many 128 x 128 tiles or K is short.  Every split gets at least four 32-element K blocks.
int gemm_ksplit(long long M, long long N, long long K, int *kb_per_split) {
    const long long tiles = ((M + BM - 1) / BM) * ((N + 127) / 128);
    const long long nkb = (K + 31) / 32;
    long long want = (2 * 148) / tiles;
    if (want > nkb / 4) want = nkb / 4;
    if (want > 64) want = 64;
    if (want < 2) { *kb_per_split = (int)nkb; return 1; }
    const long long per = (nkb + want - 1) / want;
    *kb_per_split = (int)per;
    return (int)((nkb + per - 1) / per);                  // every split non-empty
}
size_t gemm_split_workspace(long long M, long long N, long long K) {
    int per;
    const int ks = gemm_ksplit(M, N, K, &per);
    return ks > 1 ? (size_t)ks * (size_t)M * (size_t)N * sizeof(float) : 0;
}

// run_gemm<TC_TF32> with the contraction split over CTAs when the output has few tiles; split_ws holds the partial
// products (gemm_split_workspace bytes, 16-byte aligned).  No fused encoder epilogue in this form.  A split product
// always runs on 128 x 128 tiles (run_gemm looks at ksplit), whatever the number of row tiles.
int run_gemm_tf32_split(const void *A, long long lda, const void *B, long long ldb, GemmParams p, void *split_ws,
                        cudaStream_t st) {
    int per;
    const int ks = gemm_ksplit(p.M, p.N, p.K, &per);
    if (ks <= 1 || p.x) return run_gemm<TC_TF32>(A, lda, B, ldb, p, st);
    float *C = p.C;
    const long long ldc = p.ldc;
    p.ksplit = ks; p.kb_per_split = per;
    p.C = static_cast<float *>(split_ws); p.ldc = p.N; p.split_stride = (long long)p.M * p.N;
    const int rc = run_gemm<TC_TF32>(A, lda, B, ldb, p, st);
    if (rc != QNN_OK) return rc;
    const long long total = (long long)p.M * p.N;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    sum_partials_kernel<<<blocks, 256, 0, st>>>(p.C, ks, p.split_stride, p.M, p.N, C, ldc);
    return qnn_launch_status();
}

int run_conv_weight_gradient(const float *gt, const float *qas, int N, int C, int Cout, int R, int S, int stride, int pad,
                             int Ho, int Wo, GemmParams p, void *split_ws, cudaStream_t st) {
    if (!p.err || !qnn_aligned(gt, 16) || !qnn_aligned(qas, 16)) return QNN_E_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return QNN_E_CUDA;
    const ConvWgradPlan pl = conv_wgrad_plan(N, C, Cout, R, S, stride, pad, Ho, Wo);
    if (pl.nkb * 32 > 0x7FFFFFFFll) return QNN_E_RANGE;
    const long long Kg = (long long)R * S * C;
    ConvWeightGather &c = p.wconv;
    c.enabled = 1; c.C = C; c.S = S; c.st = stride; c.pad = pad; c.qmin = pl.qmin;
    c.tiles_c = pl.tiles_c; c.Wq = pl.Wq; c.kb_per_image = pl.kb_per_image;
    p.M = Cout; p.N = (int)Kg; p.K = (int)(pl.nkb * 32);
    p.tiles_n = R * S * pl.tiles_c;
    float *C_out = p.C;
    const long long ldc = p.ldc;
    p.ksplit = pl.ksplit; p.kb_per_split = pl.kb_per_split;
    if (pl.ksplit > 1) { p.C = static_cast<float *>(split_ws); p.ldc = Kg; p.split_stride = (long long)Cout * Kg; }
    const long long pa = (long long)Ho * pl.Wq, pb = (long long)pl.Hq * pl.Wq;       // pixels per image in gt / in a copy
    const long long adims[3] = {pa, N, Cout}, astr[2] = {pa, pa * N};
    const int abox[3] = {32, 1, BM};
    const long long bdims[4] = {pb, N, C, (long long)S * stride}, bstr[3] = {pb, pb * N, pb * N * C};
    const int bbox[4] = {32, 1, pl.bn, 1};
    CUtensorMap map_a, map_b;
    if (!make_map_nd(&map_a, gt, 3, adims, astr, abox) || !make_map_nd(&map_b, qas, 4, bdims, bstr, bbox)) return QNN_E_CUDA;
    const int rc = pl.bn == 256 ? launch_gemm<256, 4, TC_TF32>(map_a, map_b, map_b, p, sms, st)
                 : pl.bn == 128 ? launch_gemm<128, 6, TC_TF32>(map_a, map_b, map_b, p, sms, st)
                                : launch_gemm<64, 8, TC_TF32>(map_a, map_b, map_b, p, sms, st);
    if (rc != QNN_OK || pl.ksplit <= 1) return rc;
    const long long total = (long long)Cout * Kg;
    const int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    sum_partials_kernel<<<blocks, 256, 0, st>>>(static_cast<const float *>(split_ws), pl.ksplit, p.split_stride, Cout, Kg, C_out, ldc);
    return qnn_launch_status();
}

}  // namespace
