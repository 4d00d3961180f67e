// Backward products of a fully-connected layer (Algorithm 1, backward propagation).
//
// With g_hat = alpha * g the two products are dense real-by-integer contractions,
//   G [r][k] = sum_n g_hat[r][n] * qw[n][k]      (g_{a^m} = 2^(m-1) * G,  since sum_j 2^(j-1) W^j = qw)
//   GW[n][k] = sum_r g_hat[r][n] * qa[r][k]      (g_{W^j} = 2^(j-1) * GW, since sum_m 2^(m-1) a^m = qa)
// and run on the tensor cores: one TF32 GEMM C = alpha * A * B^T with both operands K-major in shared memory
// (tcgen05.mma, kind::tf32, accumulator in tensor memory), fed by TMA through a ring of mbarrier-guarded stages.
// The integer codes (|q| <= 255) are exact in TF32; the gradient keeps 11 significant bits per element.
// Bound: tensor pipe (2*M*N*K flop per call).
#include <cuda.h>
#include "qnn_internal.cuh"
#include "mbit_math.cuh"

namespace {

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

// Every wait is bounded: after WAIT_LIMIT failed polls the waiter raises the abort flag of its CTA and the global
// error word, and every role of the CTA leaves its loop at the next poll.
constexpr uint32_t WAIT_LIMIT = 1u << 24;

__device__ unsigned int g_tc_error;   // 0 = no error; else 1 + the id of the wait that gave up first

__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag, unsigned id) {
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023u) == 1023u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(&g_tc_error, 0u, 1u + id);
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
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

// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x BN x 8 TF32 step issued by a single thread.
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// 32 consecutive accumulator columns of this thread's row (lane of tensor memory = row of the tile).
__device__ __forceinline__ void tmem_load_32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
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
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor of a K-major tile written by TMA with the 128-byte swizzle: rows of 128 bytes,
// groups of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulator, TF32 A and B, both K-major, M = 128, N = BN.
template <int BN>
__host__ __device__ constexpr uint32_t idesc_tf32() {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((128u >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------ the GEMM kernel

constexpr int BM = 128;                 // rows of C per CTA = lanes of tensor memory
constexpr int BK = 32;                  // fp32 elements per stage row = 128 bytes = one swizzle span
constexpr int UMMA_K = 8;               // K of one TF32 instruction (32 bytes)
constexpr int EPI_WARPS = 8;            // two warps per quarter of the tensor-memory lanes, alternating 32-column chunks
constexpr int GEMM_THREADS = 64 + 32 * EPI_WARPS;   // warp 0: TMA producer, warp 1: MMA issuer + tensor-memory owner

struct GemmParams {
    int M, N, K;                        // C[M][N] = alpha * sum_k A[M][K] * B[N][K]
    float alpha;
    float *C;
    long long ldc;
    const float *x;                     // optional [M][N] (leading dimension ldx): fuse Eq. 12 with `bits` planes and range r
    long long ldx;
    int bits;
    float r;
    MbitPlaneConsts enc;                // constants of Eq. 12 for `bits` planes
    int tiles_n, tiles;
};

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

template <int BN, int STAGES>
struct GemmSmem {
    static constexpr int A_BYTES = BM * BK * 4;
    static constexpr int B_BYTES = BN * BK * 4;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int EPI_OFFSET = STAGES * STAGE_BYTES;                       // per epilogue warp a 32 x 33 fp32 tile
    static constexpr int BAR_OFFSET = EPI_OFFSET + EPI_WARPS * 32 * 33 * 4;
    static constexpr int TOTAL = BAR_OFFSET + (2 * STAGES + 4) * 8 + 16 + 1024;   // + slack for the 1024-byte alignment
};

// Persistent: CTA b works on tiles b, b + gridDim.x, ...  The accumulator is double-buffered in tensor memory
// (2 x BN columns), so the epilogue of one tile runs under the main loop of the next.
template <int BN, int STAGES>
__global__ void __launch_bounds__(GEMM_THREADS, 1) tf32_gemm_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                   const __grid_constant__ CUtensorMap map_b,
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

    if (warp == 0) {
        if (lane == 0) {
            long long it = 0;                                 // stage uses so far, over all tiles
            for (int tile = blockIdx.x; tile < p.tiles && !*abort_flag; tile += gridDim.x) {
                const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = (int)(it % STAGES);
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag, 0)) break;
                    mbar_expect_tx(&full[s], L::STAGE_BYTES);
                    tma_load_2d(smem + s * L::STAGE_BYTES, &map_a, &full[s], kb * BK, m0);
                    tma_load_2d(smem + s * L::STAGE_BYTES + L::A_BYTES, &map_b, &full[s], kb * BK, n0);
                }
            }
            if (*abort_flag) {   // let the copies still in flight land before the CTA's shared memory goes away
                for (long long j = it > STAGES ? it - STAGES : 0; j < it; ++j)
                    for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_try_wait(&full[j % STAGES], (uint32_t)(j / STAGES) & 1u); ++w) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_tf32<BN>();
            long long it = 0;
            int local = 0;
            for (int tile = blockIdx.x; tile < p.tiles && !*abort_flag; tile += gridDim.x, ++local) {
                const int buf = local & 1;
                if (!mbar_wait(&acc_empty[buf], ((uint32_t)(local >> 1) & 1u) ^ 1u, abort_flag, 3)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = (int)(it % STAGES);
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                    if (!mbar_wait(&full[s], ph, abort_flag, 1)) break;
                    tc_fence_after();
                    const uint64_t a_desc = smem_desc_k_sw128(smem_u32(smem + s * L::STAGE_BYTES));
                    const uint64_t b_desc = smem_desc_k_sw128(smem_u32(smem + s * L::STAGE_BYTES + L::A_BYTES));
#pragma unroll
                    for (int j = 0; j < BK / UMMA_K; ++j)   // 32 bytes along K per step = 2 descriptor address units
                        tc_mma_tf32(d_tmem, a_desc + 2 * j, b_desc + 2 * j, idesc, (kb | j) != 0 ? 1u : 0u);
                    tc_commit(&empty[s]);
                }
                tc_commit(&acc_full[buf]);
            }
        }
    } else {
        const int q = warp & 3;                            // a warp reaches the 32 lanes [32*(warp%4), +32) only
        const int half = (warp - 2) >> 2;                  // which of the two warps of this quarter
        int local = 0;
        for (int tile = blockIdx.x; tile < p.tiles; tile += gridDim.x, ++local) {
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
            const int buf = local & 1;
            if (!mbar_wait(&acc_full[buf], (uint32_t)(local >> 1) & 1u, abort_flag, 2)) break;
            tc_fence_after();
            // Each 32 x 32 chunk goes through the warp's shared tile: tensor memory hands a thread one row, memory
            // wants a warp on one row, so that every access to C and x is a whole 128-byte line.
            float *stage = reinterpret_cast<float *>(smem + L::EPI_OFFSET) + (warp - 2) * (32 * 33);
#pragma unroll 1
            for (int c0 = half * 32; c0 < BN; c0 += 64) {
                if (n0 + c0 >= p.N) break;                 // uniform over the warp
                float v[32];
                tmem_load_32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c0), v);
#pragma unroll
                for (int i = 0; i < 32; ++i) stage[lane * 33 + i] = __fmul_rn(v[i], p.alpha);
                __syncwarp();
                const int col = n0 + c0 + lane;
                const int rows_here = min(32, p.M - (m0 + q * 32));
                if (col < p.N) {
                    float *cptr = p.C + (long long)(m0 + q * 32) * p.ldc + col;
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
        const int mine = p.tiles > (int)blockIdx.x ? (p.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
        if (mine > 0) {
            const int last = mine - 1;
            for (uint32_t w = 0; w < WAIT_LIMIT && !mbar_try_wait(&acc_full[last & 1], (uint32_t)(last >> 1) & 1u); ++w) {}
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
    }
}

// ------------------------------------------------------------------------------------------------ staging kernels

// Bit planes [rows][bits][kw] -> odd codes q = 2t - (2^bits - 1) as fp32.  TRANSPOSE = false: out[row][col], a
// block covers 32 rows x 256 columns (warp w owns plane word w of eight).  TRANSPOSE = true: out[col][row], a block
// covers 256 rows x 32 columns (one plane word per row), so that each output row receives 1 KiB in one piece.
// The 32 threads of a warp run along the contiguous index of the output: every store instruction writes one line.
template <bool TRANSPOSE, int BITS>
__global__ void __launch_bounds__(256) unpack_codes_kernel(const uint32_t *__restrict__ planes, long long rows, long long k,
                                                          long long kw, float *__restrict__ out, long long ld) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float amax = (float)((1 << BITS) - 1);
    if (TRANSPOSE) {
        const long long row = (long long)blockIdx.y * 256 + threadIdx.x, wcol = blockIdx.x;
        if (row >= rows) return;
        uint32_t w[BITS];
#pragma unroll
        for (int b = 0; b < BITS; ++b) w[b] = __ldg(planes + (row * BITS + b) * kw + wcol);
        const int ncol = (int)min(32ll, k - wcol * 32);
        float *o = out + wcol * 32 * ld + row;
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
            int t = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) t |= (int)((w[b] >> c) & 1u) << b;
            if (c < ncol) o[c * ld] = (float)(2 * t) - amax;   // default cache policy: the GEMM reads it next, from L2
        }
    } else {
        const long long r0 = (long long)blockIdx.y * 32, wcol = (long long)blockIdx.x * 8 + ty;
        const long long col = wcol * 32 + tx;
        if (wcol * 32 >= k) return;
#pragma unroll 4
        for (int i = 0; i < 32; ++i) {
            const long long row = r0 + i;
            if (row >= rows) break;
            int t = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) t |= (int)((__ldg(planes + (row * BITS + b) * kw + wcol) >> tx) & 1u) << b;
            if (col < k) out[row * ld + col] = (float)(2 * t) - amax;
        }
    }
}

// out[c][r] = in[r][c] through a 32 x 33 shared tile (both sides coalesced).
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float *__restrict__ in, long long rows, long long cols,
                                                           long long ld_in, float *__restrict__ out, long long ld_out) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const long long r0 = (long long)blockIdx.y * 32, c0 = (long long)blockIdx.x * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long r = r0 + ty + 8 * i, c = c0 + tx;
        tile[ty + 8 * i][tx] = (r < rows && c < cols) ? in[r * ld_in + c] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long c = c0 + ty + 8 * i, r = r0 + tx;
        if (c < cols && r < rows) out[c * ld_out + r] = tile[tx][ty + 8 * i];
    }
}

// Row-padded copy for a gradient whose rows are not 16-byte multiples (TMA needs them to be).
__global__ void __launch_bounds__(256) copy_rows_kernel(const float *__restrict__ in, long long rows, long long cols,
                                                       float *__restrict__ out, long long ld_out) {
    const long long total = rows * cols;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
        out[(i / cols) * ld_out + i % cols] = in[i];
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

// Tensor map of a row-major fp32 matrix [rows][cols] with leading dimension ld, box = 32 columns x box_rows rows,
// 128-byte swizzle, zero fill outside the matrix.
bool make_map(CUtensorMap *map, const float *base, long long rows, long long cols, long long ld, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

long long pad32(long long v) { return (v + 31) / 32 * 32; }

template <int BN, int STAGES>
int launch_gemm(const CUtensorMap &map_a, const CUtensorMap &map_b, GemmParams p, int sms, cudaStream_t st) {
    using L = GemmSmem<BN, STAGES>;
    static bool attr_set = false;   // per process; set again on the next call if it failed
    if (!attr_set) {
        if (cudaFuncSetAttribute(tf32_gemm_kernel<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL) !=
            cudaSuccess)
            return QNN_E_CUDA;
        attr_set = true;
    }
    const long long tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return QNN_E_ARG;
    p.tiles_n = (int)tiles_n;
    p.tiles = (int)(tiles_m * tiles_n);
    const int grid = p.tiles < sms ? p.tiles : sms;
    tf32_gemm_kernel<BN, STAGES><<<grid, GEMM_THREADS, L::TOTAL, st>>>(map_a, map_b, p);
    return qnn_launch_status();
}

int sm_count() {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            sms = 0;
    }
    return sms;
}

// C[M][N] = alpha * A[M][K] * B[N][K]^T (optionally times the encoder derivative at x).  128 x 256 tiles when they
// give every SM a tile (they read each A tile from shared memory half as often per flop as 128 x 128 ones, which a
// single CTA per SM cannot feed fast enough), 128 x 128 tiles otherwise.
int run_gemm(const float *A, long long lda, const float *B, long long ldb, GemmParams p, cudaStream_t st) {
    if (p.M <= 0 || p.N <= 0 || p.K <= 0) return QNN_E_ARG;
    if (!qnn_aligned(A, 16) || !qnn_aligned(B, 16) || lda % 4 || ldb % 4) return QNN_E_ALIGN;
    const int sms = sm_count();
    if (sms <= 0) return QNN_E_CUDA;
    const bool wide = ((long long)(p.M + BM - 1) / BM) * ((p.N + 255) / 256) >= sms;
    CUtensorMap map_a, map_b;
    if (!make_map(&map_a, A, p.M, p.K, lda, BM) || !make_map(&map_b, B, p.N, p.K, ldb, wide ? 256 : 128)) return QNN_E_CUDA;
    return wide ? launch_gemm<256, 4>(map_a, map_b, p, sms, st) : launch_gemm<128, 6>(map_a, map_b, p, sms, st);
}

template <bool TRANSPOSE>
void launch_unpack(const uint32_t *planes, long long rows, long long k, int bits, long long kw, float *out, long long ld,
                   cudaStream_t st) {
    const dim3 grid = TRANSPOSE ? dim3((unsigned)qnn_ceil_div(k, 32), (unsigned)qnn_ceil_div(rows, 256))
                                : dim3((unsigned)qnn_ceil_div(k, 256), (unsigned)qnn_ceil_div(rows, 32));
#define UNPACK_CASE(B) case B: unpack_codes_kernel<TRANSPOSE, B><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    switch (bits) {
        UNPACK_CASE(1) UNPACK_CASE(2) UNPACK_CASE(3) UNPACK_CASE(4) UNPACK_CASE(5) UNPACK_CASE(6) UNPACK_CASE(7)
        default: unpack_codes_kernel<TRANSPOSE, 8><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    }
#undef UNPACK_CASE
}

int unpack_codes(const uint32_t *planes, long long rows, long long k, int bits, bool transpose, float *out, long long ld,
                 cudaStream_t st) {
    const long long kw = qnn_row_words_i(k);
    if (transpose) launch_unpack<true>(planes, rows, k, bits, kw, out, ld, st);
    else launch_unpack<false>(planes, rows, k, bits, kw, out, ld, st);
    return qnn_launch_status();
}

}  // namespace

// ------------------------------------------------------------------------------------------------ C ABI

static const size_t DIM_LIMIT = (size_t)65535 * 32;   // every dimension may become the y extent of a staging grid

static bool backward_dims_ok(size_t m, size_t n, size_t k) {
    return m >= 1 && n >= 1 && k >= 1 && m <= DIM_LIMIT && n <= DIM_LIMIT && k <= DIM_LIMIT;
}

extern "C" int qnn_unpack_codes_f32(const uint32_t *planes, size_t rows, size_t k, int bits, int transpose, float *out,
                                    size_t ld, void *stream) {
    if (!planes || !out || rows < 1 || k < 1 || rows > DIM_LIMIT || k > DIM_LIMIT || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (ld < (transpose ? rows : k)) return QNN_E_ARG;
    if (!qnn_aligned(planes, 16) || !qnn_aligned(out, 4)) return QNN_E_ALIGN;
    return unpack_codes(planes, (long long)rows, (long long)k, bits, transpose != 0, out, (long long)ld,
                        static_cast<cudaStream_t>(stream));
}

extern "C" size_t qnn_bgemm_backward_data_workspace(size_t m, size_t n, size_t k) {
    if (!backward_dims_ok(m, n, k)) return 0;
    const size_t ldn = (size_t)pad32((long long)n);
    return (k + (n % 4 ? m : 0)) * ldn * sizeof(float);
}

extern "C" int qnn_bgemm_backward_data(const float *g, const uint32_t *w_planes, size_t m, size_t n, size_t k, int wb,
                                       float alpha, const float *x, int ab, float r, float *out, void *workspace,
                                       size_t workspace_bytes, void *stream) {
    if (!g || !w_planes || !out || !workspace || !backward_dims_ok(m, n, k) || !qnn_bits_ok(wb)) return QNN_E_ARG;
    if (x && !qnn_bits_ok(ab)) return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (x && (!(r >= 1e-30f) || !(r <= 1e30f))) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bgemm_backward_data_workspace(m, n, k)) return QNN_E_ARG;
    if (!qnn_aligned(g, 16) || !qnn_aligned(w_planes, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(out, 4) ||
        (x && !qnn_aligned(x, 4)))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ldn = pad32((long long)n);
    float *wqt = static_cast<float *>(workspace);                       // [k][ldn]: wqt[kk][nn] = qw[nn][kk]
    int rc = unpack_codes(w_planes, (long long)n, (long long)k, wb, true, wqt, ldn, st);
    if (rc != QNN_OK) return rc;
    const float *a = g;
    long long lda = (long long)n;
    if (n % 4) {                                                        // rows of g are not 16-byte multiples
        float *gp = wqt + (size_t)k * ldn;
        copy_rows_kernel<<<148 * 8, 256, 0, st>>>(g, (long long)m, (long long)n, gp, ldn);
        if ((rc = qnn_launch_status()) != QNN_OK) return rc;
        a = gp;
        lda = ldn;
    }
    GemmParams p{};
    p.M = (int)m; p.N = (int)k; p.K = (int)n;
    p.alpha = alpha;
    p.C = out; p.ldc = (long long)k;
    p.x = x; p.ldx = (long long)k; p.bits = ab; p.r = r;
    if (x) p.enc = mbit_plane_consts(ab);
    return run_gemm(a, lda, wqt, ldn, p, st);
}

extern "C" size_t qnn_bgemm_backward_weights_workspace(size_t m, size_t n, size_t k) {
    if (!backward_dims_ok(m, n, k)) return 0;
    return (n + k) * (size_t)pad32((long long)m) * sizeof(float);
}

extern "C" int qnn_bgemm_backward_weights(const float *g, const uint32_t *a_planes, size_t m, size_t n, size_t k, int ab,
                                          float alpha, float *gw, void *workspace, size_t workspace_bytes, void *stream) {
    if (!g || !a_planes || !gw || !workspace || !backward_dims_ok(m, n, k) || !qnn_bits_ok(ab)) return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bgemm_backward_weights_workspace(m, n, k)) return QNN_E_ARG;
    if (!qnn_aligned(g, 4) || !qnn_aligned(a_planes, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(gw, 4))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ldm = pad32((long long)m);
    float *gt = static_cast<float *>(workspace);                        // [n][ldm]: gt[nn][rr] = g[rr][nn]
    float *aqt = gt + (size_t)n * ldm;                                  // [k][ldm]: aqt[kk][rr] = qa[rr][kk]
    const dim3 grid((unsigned)qnn_ceil_div((long long)n, 32), (unsigned)qnn_ceil_div((long long)m, 32));
    transpose_f32_kernel<<<grid, 256, 0, st>>>(g, (long long)m, (long long)n, (long long)n, gt, ldm);
    int rc = qnn_launch_status();
    if (rc != QNN_OK) return rc;
    if ((rc = unpack_codes(a_planes, (long long)m, (long long)k, ab, true, aqt, ldm, st)) != QNN_OK) return rc;
    GemmParams p{};
    p.M = (int)n; p.N = (int)k; p.K = (int)m;
    p.alpha = alpha;
    p.C = gw; p.ldc = (long long)k;
    return run_gemm(gt, ldm, aqt, ldm, p, st);
}

extern "C" int qnn_tensor_path_status(unsigned int *status) {
    if (!status) return QNN_E_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return QNN_E_CUDA;
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(v)) != cudaSuccess) return QNN_E_CUDA;
    if (v && cudaMemcpyToSymbol(g_tc_error, &zero, sizeof(zero)) != cudaSuccess) return QNN_E_CUDA;
    *status = v;
    return v ? QNN_E_DEVICE : QNN_OK;
}
