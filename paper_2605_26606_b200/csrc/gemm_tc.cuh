// bf16 GEMM on the 5th-generation tensor cores:  C[M, N] = A[M, K] * W[N, K]^T, float accumulation in TMEM.
//
// One persistent CTA per SM walks output tiles of 128 x BN.  Warp 0 feeds shared memory with TMA
// (128-byte swizzled K-major boxes of 64 bf16), warp 1 issues tcgen05.mma (UMMA 128 x BN x 16) into one
// of two TMEM accumulators, warps 2..5 drain the other accumulator with tcgen05.ld and run the fused
// epilogue, so the epilogue of tile i overlaps the main loop of tile i+1.  Tiles are ordered M-fastest:
// CTAs running together share the same weight tile, which therefore leaves HBM once.
//
// K may be cut into `splits` slices handled by different CTAs (small batches: otherwise a handful of CTAs would
// stream the whole weight matrix); every slice leaves its own partial sum and the consuming kernel adds them in
// slice order, so results are deterministic.  With DUAL the activations arrive as a bf16 value plus its bf16
// rounding remainder and both are multiplied with the same weight tile.
//
// All waits on mbarriers are bounded; a wait that runs out raises DEV_ERR_WAIT_TIMEOUT in the caller's
// error flag, every role leaves its loop, and the CTA frees its TMEM before it returns.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include <cstring>
#include <type_traits>

#include "common.cuh"

namespace pc {
namespace tc {

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr uint32_t WAIT_LIMIT = 1u << 24;

// dual: the A operand comes as two bf16 matrices (high part and rounding remainder) that are both multiplied with the
// same weight tile, which removes the bf16 rounding of the activations from the product at the cost of a second MMA.
__host__ __device__ constexpr int stage_bytes(int bn, bool dual) { return ((dual ? 2 : 1) * BM + bn) * BK * 2; }
__host__ __device__ constexpr int num_stages(int bn, bool dual) {
    int s = (200 * 1024) / stage_bytes(bn, dual);
    return s > 8 ? 8 : s;
}
__host__ __device__ constexpr int smem_bytes(int bn, bool dual) {
    return num_stages(bn, dual) * stage_bytes(bn, dual) + 1024 /*align*/ + 256 /*barriers*/;
}

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when it gave up (or when another role already raised the abort flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit = WAIT_LIMIT) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    const uint32_t zero = 0;    // no output lane is disabled
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(zero)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
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

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled
// (8-row groups 1024 bytes apart): start address, leading offset (unused for swizzled K-major, 1),
// stride offset 1024 B, descriptor version 1, layout type SWIZZLE_128B.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: D = F32, A and B both BF16 (format 1) or both IEEE half (format 0), both K-major,
// N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool half_operands) {
    return (1u << 4) | (half_operands ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------
// Epilogues: called once per (row, 32 consecutive columns); n_valid columns are inside N.
// ---------------------------------------------------------------------------------------------
struct EpiStoreF32 {
    static constexpr bool kWholeTile = false;            // C = acc (+ bias)
    float* C; int ldc; const float* bias;
    __device__ __forceinline__ void set_rows(int) {}
    __device__ __forceinline__ void operator()(int row, int col0, const float* v, int n_valid, int /*split*/) const {
        float* dst = C + (size_t)row * ldc + col0;
        if (n_valid == 32 && (ldc & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                float4 o = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                if (bias) { o.x += bias[col0 + i]; o.y += bias[col0 + i + 1]; o.z += bias[col0 + i + 2]; o.w += bias[col0 + i + 3]; }
                *reinterpret_cast<float4*>(dst + i) = o;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < n_valid) dst[i] = v[i] + (bias ? bias[col0 + i] : 0.f);
        }
    }
};
struct EpiPartial {
    static constexpr bool kWholeTile = false;             // P[split][row][col] = acc   (raw K-slice sums; the consumer adds the slices in order)
    float* P; int ld; size_t split_stride;
    __device__ __forceinline__ void set_rows(int m) { split_stride = (size_t)m * ld; }     // slices packed by the row bound
    __device__ __forceinline__ void operator()(int row, int col0, const float* v, int n_valid, int split) const {
        float* dst = P + (size_t)split * split_stride + (size_t)row * ld + col0;
        if (n_valid == 32 && (ld & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < n_valid) dst[i] = v[i];
        }
    }
};
struct EpiResidual {
    static constexpr bool kWholeTile = true;             // H += acc
    float* H; int ldc;
    __device__ __forceinline__ void set_rows(int) {}
    // Whole tile of the thread's row: the residual values of the next 32 columns are requested before the current 32
    // are added and stored (a thread owns a row, so one chunk's round trip at a time would dominate a one-tile CTA).
    template <int BN>
    __device__ __forceinline__ void tile(uint32_t taddr, int row, bool live, int n0, int N) const;
    __device__ __forceinline__ void operator()(int row, int col0, const float* v, int n_valid, int /*split*/) const {
        float* dst = H + (size_t)row * ldc + col0;
        if (n_valid == 32 && (ldc & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                float4 o = *reinterpret_cast<float4*>(dst + i);
                o.x += v[i]; o.y += v[i + 1]; o.z += v[i + 2]; o.w += v[i + 3];
                *reinterpret_cast<float4*>(dst + i) = o;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < n_valid) dst[i] += v[i];
        }
    }
};
template <int BN>
__device__ __forceinline__ void EpiResidual::tile(uint32_t taddr, int row, bool live, int n0, int N) const {
    const int n_cols = min(BN, N - n0);
    float* hrow = H + (size_t)(live ? row : 0) * ldc + n0;
    if ((ldc & 3) != 0 || (n_cols & 31) != 0) {              // ragged or unaligned: one chunk at a time
#pragma unroll 1
        for (int c = 0; c < n_cols; c += 32) {
            float v[32];
            tmem_ld32(taddr + c, v);
            if (live) (*this)(row, n0 + c, v, min(32, n_cols - c), 0);
        }
        return;
    }
    float4 cur[8], nxt[8];
    if (live) {
#pragma unroll
        for (int i = 0; i < 8; ++i) cur[i] = reinterpret_cast<const float4*>(hrow)[i];
    }
#pragma unroll 1
    for (int c = 0; c < n_cols; c += 32) {
        if (live && c + 32 < n_cols) {
#pragma unroll
            for (int i = 0; i < 8; ++i) nxt[i] = reinterpret_cast<const float4*>(hrow + c + 32)[i];
        }
        float v[32];
        tmem_ld32(taddr + c, v);
        if (live) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 o = cur[i];
                o.x += v[4 * i]; o.y += v[4 * i + 1]; o.z += v[4 * i + 2]; o.w += v[4 * i + 3];
                reinterpret_cast<float4*>(hrow + c)[i] = o;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) cur[i] = nxt[i];
        }
    }
}
struct EpiSwiGLU {
    static constexpr bool kWholeTile = false;              // columns (2j, 2j+1) = (gate_j, up_j) -> out[row, j] = silu(gate) * up, bf16 (or IEEE half)
    __nv_bfloat16* out; int ld; int half_out; int32_t* err;
    __device__ __forceinline__ void set_rows(int) {}
    __device__ __forceinline__ void operator()(int row, int col0, const float* v, int n_valid, int /*split*/) const {
        __nv_bfloat16* dst = out + (size_t)row * ld + (col0 >> 1);
        if (n_valid == 32 && (ld & 7) == 0) {
            uint32_t w[8];
            int bad = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float g0 = v[4 * i], u0 = v[4 * i + 1], g1 = v[4 * i + 2], u1 = v[4 * i + 3];
                const float y0 = g0 / (1.f + expf(-g0)) * u0, y1 = g1 / (1.f + expf(-g1)) * u1;
                if (half_out) {
                    bad |= half_bad(y0) | half_bad(y1);
                    const __half2 p = __floats2half2_rn(half_clamp(y0), half_clamp(y1));
                    w[i] = *reinterpret_cast<const uint32_t*>(&p);
                } else {
                    const __nv_bfloat162 p = __floats2bfloat162_rn(y0, y1);
                    w[i] = *reinterpret_cast<const uint32_t*>(&p);
                }
            }
            *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(dst + 8) = make_uint4(w[4], w[5], w[6], w[7]);
            if (bad) set_error(err, DEV_ERR_HALF_RANGE);
        } else {
#pragma unroll
            for (int i = 0; i < 32; i += 2)
                if (i + 1 < n_valid) {
                    const float y = v[i] / (1.f + expf(-v[i])) * v[i + 1];
                    if (half_out) reinterpret_cast<__half*>(dst)[i >> 1] = __float2half_rn(half_guard(y, err));
                    else dst[i >> 1] = __float2bfloat16_rn(y);
                }
        }
    }
};

// ---------------------------------------------------------------------------------------------
// Kernel
// ---------------------------------------------------------------------------------------------
// Epilogue warps of a kernel instance: four (one per 32-lane quarter of the accumulator) unless the epilogue asks for eight
// (Epi::kEpiWarps = 8: two warps per quarter, each walking half of the tile's columns -- for epilogues whose arithmetic,
// not their memory traffic, is what has to hide behind the next tile's main loop).
template <class E, class = void> struct EpiWarps { static constexpr int value = 4; };
template <class E> struct EpiWarps<E, std::void_t<decltype(E::kEpiWarps)>> { static constexpr int value = E::kEpiWarps; };
template <class E> constexpr int block_threads() { return 64 + 32 * EpiWarps<E>::value; }

template <int BN, bool DUAL, class Epi>
__global__ void __launch_bounds__(block_threads<Epi>(), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_a_lo,
               const __grid_constant__ CUtensorMap map_w, const StepDesc* __restrict__ sd, int M, int N, int K, int splits, Epi epi,
               int32_t* err, int half_operands) {
    // M is the row bound the grid, the tile order and the layout of partial sums were sized for; a captured step
    // may hold fewer live rows (same number of row tiles: the bound is the live count rounded up to a tile), which
    // only the epilogue needs to know, so the loads and MMAs never wait for the step descriptor.
    epi.set_rows(M);
    constexpr int STAGES = num_stages(BN, DUAL);
    constexpr int A1_BYTES = BM * BK * 2;                    // one A tile
    constexpr int A_BYTES = (DUAL ? 2 : 1) * A1_BYTES, B_BYTES = BN * BK * 2;
    constexpr uint32_t TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;
    extern __shared__ uint8_t smem_raw[];
    // tiles must start on a 1024-byte boundary for the 128-byte swizzle pattern
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * (A_BYTES + B_BYTES));
    // bars: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES, tfull0 = empty0 + 8 * STAGES, tempty0 = tfull0 + 16;
    const uint32_t tiles_u32 = smem_u32(tiles);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, EpiWarps<Epi>::value); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The kernel after this one may start its own set-up now.  This kernel, if it was launched as a programmatic dependent,
    // may be running beside the one before it: everything but the weight stream waits for that kernel here.
    grid_dep_launch_dependents();
    if (threadIdx.x != 0) grid_dep_wait();

    // work item t = ((n_tile * splits) + split) * tiles_m + m_tile; split s covers k-blocks [s*KB/splits, (s+1)*KB/splits)
    const int tiles_m = (M + BM - 1) / BM, tiles_n = (N + BN - 1) / BN, n_tiles = tiles_m * tiles_n * splits;
    const int k_blocks_total = K / BK;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer ----------------
            // The weight tiles of the first k-blocks are requested first, their activation tiles right after.
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            struct Cursor { int t, kb, kb1, m0, n0; };
            auto seek = [&](Cursor& c) {
                if (c.t >= n_tiles) return;
                const int sp = (c.t / tiles_m) % splits;
                c.m0 = (c.t % tiles_m) * BM; c.n0 = (c.t / (tiles_m * splits)) * BN;
                c.kb = sp * k_blocks_total / splits; c.kb1 = (sp + 1) * k_blocks_total / splits;
            };
            auto advance = [&](Cursor& c) { if (++c.kb == c.kb1) { c.t += gridDim.x; seek(c); } };
            Cursor cb{(int)blockIdx.x, 0, 0, 0, 0};
            seek(cb);
            {
                Cursor ca = cb;
                int ahead = 0;
                uint32_t stage_b = 0;
                while (cb.t < n_tiles && ahead < STAGES) {          // the ring is empty: no wait needed
                    mbar_arrive_expect_tx(full0 + 8 * stage_b, A_BYTES + B_BYTES);
                    tma_load_2d(tiles_u32 + stage_b * (A_BYTES + B_BYTES) + A_BYTES, &map_w, full0 + 8 * stage_b, cb.kb * BK, cb.n0);
                    ++ahead; ++stage_b;
                    advance(cb);
                }
                grid_dep_wait();          // the activations are the previous kernel's output; the weights above are not
                for (; ahead > 0; --ahead) {
                    const uint32_t sa = tiles_u32 + stage * (A_BYTES + B_BYTES);
                    tma_load_2d(sa, &map_a, full0 + 8 * stage, ca.kb * BK, ca.m0);
                    if (DUAL) tma_load_2d(sa + A1_BYTES, &map_a_lo, full0 + 8 * stage, ca.kb * BK, ca.m0);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    advance(ca);
                }
            }
            while (cb.t < n_tiles) {
                if (!mbar_wait(empty0 + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                const uint32_t sa = tiles_u32 + stage * (A_BYTES + B_BYTES), sb = sa + A_BYTES;
                mbar_arrive_expect_tx(full0 + 8 * stage, A_BYTES + B_BYTES);
                tma_load_2d(sa, &map_a, full0 + 8 * stage, cb.kb * BK, cb.m0);
                if (DUAL) tma_load_2d(sa + A1_BYTES, &map_a_lo, full0 + 8 * stage, cb.kb * BK, cb.m0);
                tma_load_2d(sb, &map_w, full0 + 8 * stage, cb.kb * BK, cb.n0);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                advance(cb);
            }
            if (!ok) { *abort_flag = 1; set_error(err, DEV_ERR_WAIT_TIMEOUT); }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = make_idesc(BM, BN, half_operands != 0);
            uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                const int sp = (t / tiles_m) % splits;
                const int k_blocks = (sp + 1) * k_blocks_total / splits - sp * k_blocks_total / splits;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = tiles_u32 + stage * (A_BYTES + B_BYTES), sb = sa + A_BYTES;
                    const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sb);
#pragma unroll
                    for (int kk = 0; kk < BK / UMMA_K; ++kk) {
                        // advancing 16 bf16 = 32 bytes inside the swizzle row: +2 in the (address >> 4) field
                        umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
                    }
                    if (DUAL) {
                        const uint64_t dl = make_smem_desc(sa + A1_BYTES);
#pragma unroll
                        for (int kk = 0; kk < BK / UMMA_K; ++kk) umma_bf16(d_tmem, dl + 2 * kk, db + 2 * kk, idesc, 1u);
                    }
                    umma_commit(empty0 + 8 * stage);          // frees the stage once these MMAs have read it
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(tfull0 + 8 * acc);                 // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (!ok) { *abort_flag = 1; set_error(err, DEV_ERR_WAIT_TIMEOUT); }
        }
    } else {
        // ---------------- epilogue warps: TMEM -> registers -> global ----------------
        const int quarter = warp & 3;                  // a warp may only read its own 32 TMEM lanes
        const int m_live = sd != nullptr ? min(M, sd->n_rows) : M;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
            const int m0 = (t % tiles_m) * BM, sp = (t / tiles_m) % splits, n0 = (t / (tiles_m * splits)) * BN;
            if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int row = m0 + quarter * 32 + lane;
            if constexpr (EpiWarps<Epi>::value == 8) {
                // two warps per quarter: warps 2..5 take the first half of the tile's columns, warps 6..9 the second
                epi.template tile_part<BN>(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN, row, row < m_live, n0, N, (warp - 2) >> 2);
            } else if constexpr (Epi::kWholeTile) {
                // the epilogue walks the accumulator tile itself (more than one pass over its columns)
                epi.template tile<BN>(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN, row, row < m_live, n0, N);
            } else {
#pragma unroll 1
                for (int c = 0; c < BN; c += 32) {
                    if (n0 + c >= N) break;                 // warp-uniform
                    float v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * BN + c, v);
                    if (row < m_live) epi(row, n0 + c, v, min(32, N - (n0 + c)), sp);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok && lane == 0) { *abort_flag = 1; set_error(err, DEV_ERR_WAIT_TIMEOUT); }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// Self-test of the bounded wait: one thread waits, with a short limit, on an mbarrier that nothing will ever arrive at
// (no copy is in flight), and reports the timeout in the error flag the way the production kernels do.
__global__ void wait_timeout_selftest_kernel(uint32_t limit, int32_t* err) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(smem_u32(&bar), 0, &abort_flag, limit)) set_error(err, DEV_ERR_WAIT_TIMEOUT);
    }
}

// Must run once per kernel instance before its first launch (raises the dynamic shared memory limit).
template <int BN, bool DUAL, class Epi>
inline cudaError_t configure() {
    return cudaFuncSetAttribute(gemm_tc_kernel<BN, DUAL, Epi>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(BN, DUAL));
}

// Host launcher.  map_w must have been encoded with box_rows = BN; map_a_lo is ignored unless DUAL.
template <int BN, bool DUAL, class Epi>
inline cudaError_t launch(cudaStream_t st, const CUtensorMap& map_a, const CUtensorMap& map_a_lo, const CUtensorMap& map_w,
                          const StepDesc* sd, int M, int N, int K, int splits, Epi epi, int32_t* err, int num_sms, bool half_operands = false,
                          bool programmatic = false) {
    auto kern = gemm_tc_kernel<BN, DUAL, Epi>;
    const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN) * splits;
    if (tiles == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(tiles < num_sms ? tiles : num_sms)); cfg.blockDim = dim3(block_threads<Epi>());
    cfg.dynamicSmemBytes = smem_bytes(BN, DUAL); cfg.stream = st;
    // programmatic: this launch may begin (set-up, first weight tiles) before the previous kernel of the stream has ended
    cudaLaunchAttribute attr[1];
    if (programmatic) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, kern, map_a, map_a_lo, map_w, sd, M, N, K, splits, epi, err, half_operands ? 1 : 0);
}

}  // namespace tc
}  // namespace pc
