// Shared-prefix decode attention for bf16 models, on tensor cores, with K/V tiles staged by TMA.
//
// The K/V arenas are viewed as 2-D tensors of 16-bit elements (IEEE half) [planes * n_slots, head_dim]; a tile of TP consecutive
// slots is fetched as head_dim/64 boxes of [TP rows x 64 columns] with the 128-byte swizzle, which makes
// the ldmatrix reads below bank-conflict free.
//
//   attn_group_kernel   one CTA per (64 query rows of a group, KV head).  The query rows are all live
//                       rollouts of the group times the query heads sharing the KV head, so the group's
//                       prompt K/V is read once per 64 query rows instead of once per rollout
//                       (S = Q K^T and O = P V as m16n8k16 MMAs, online softmax in registers).  Every
//                       query row carries its own number of visible prompt slots, which also makes this
//                       the causal prefill kernel.  Decode: leaves (m, l, unnormalised O) per query row
//                       in scratch.  Prefill: writes the normalised output.
//   attn_suffix_kernel  one warp per (rollout, KV head) streams the rollout's own suffix K/V through a
//                       3-stage TMA ring at full HBM rate.  Positions sit on the MMA M axis (S^T = K Q^T,
//                       O^T = V^T P^T), so the 6-8 query heads fill the N = 8 axis and no MMA work is
//                       padded; P is transposed between the two MMAs with movmatrix.  It leaves its
//                       (m, l, unnormalised O) record next to the prefix records.
//   attn_merge_kernel   combines the prefix records and the suffix record of every (row, head) by their
//                       log-sum-exp and writes the bf16 attention output.
//
// Scores are kept in the log2 domain (scaled by log2(e) / sqrt(head_dim)) so that exp2f is the only
// transcendental.  Waits on mbarriers are bounded (see gemm_tc.cuh).
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "kernels_basic.cuh"

namespace pc {
namespace am {

using tc::mbar_arrive;
using tc::mbar_arrive_expect_tx;
using tc::mbar_init;
using tc::mbar_wait;
using tc::smem_u32;
using tc::tma_load_2d;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Both attention products take IEEE half operands: q, K and V are stored as half (see qkv_post_kernel), P is rounded to half
__device__ __forceinline__ void mma_f16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    const __half2 p = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}
// The same for values that leave the kernel as a GEMM operand: out-of-range values are saturated and reported.
__device__ __forceinline__ uint32_t pack_f16_guard(float lo, float hi, int32_t* err) {
    return pack_f16(half_guard(lo, err), half_guard(hi, err));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}
// exp2 that maps -inf to 0 without producing NaN when both operands are -inf
__device__ __forceinline__ float exp2_safe(float x, float m) { return m == -INFINITY ? 0.f : exp2f(x - m); }

// Byte offset of (row r, dim d) (d a multiple of 8) in a swizzled tile of ROWS rows: boxes of 64 dims,
// rows of 128 bytes, 16-byte chunk index XORed with (r mod 8).
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int r, int d) {
    return (uint32_t)((d >> 6) * (ROWS * 128) + r * 128 + ((((d & 63) >> 3) ^ (r & 7)) << 4));
}

// Prefix part of the attention, per (row, query head): running max (log2 domain), sum, unnormalised output.
// When a group has few query rows its prompt is cut into n_parts ranges handled by different CTAs; every range
// leaves its own record and the suffix kernel merges all of them.
struct PrefixPartial {
    float* m;               // [n_parts][stride]
    float* l;               // [n_parts][stride]
    float* o;               // [n_parts][stride * head_dim]
    int n_parts;
    size_t stride;          // rows capacity * Hq
    int n_kv_heads;
    int n_suffix_warps;     // warps of the suffix kernel's grid: how suffixes are cut into ranges is planned for this many
};
constexpr int MAX_PREFIX_PARTS = 8;
constexpr int MAX_SUFFIX_CHUNKS = 8;
constexpr int MAX_RECORDS = MAX_PREFIX_PARTS + MAX_SUFFIX_CHUNKS;

// ---------------------------------------------------------------------------------------------
// Group (shared-prefix / causal-prefill) kernel
// ---------------------------------------------------------------------------------------------
constexpr int G_THREADS = 128;      // 4 warps x 16 query rows; two such CTAs share an SM
constexpr int G_QROWS = 64;
constexpr int G_TK = 64;            // KV positions per stage
constexpr int G_STAGES = 3;
template <int HD> constexpr int group_smem_bytes() { return G_STAGES * 2 * G_TK * HD * 2 + 1024 + 128; }

template <int HD, bool FINAL>
__global__ void __launch_bounds__(G_THREADS, 2)
attn_group_kernel(const __grid_constant__ CUtensorMap kv_map, const StepDesc* __restrict__ sd, int64_t n_slots, int Hq, int Hkv,
                  int layer, const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ group_row_start, RowGeom g,
                  float scale_log2, PrefixPartial part, __nv_bfloat16* __restrict__ out, __nv_bfloat16* __restrict__ out_lo,
                  int32_t* err) {
    constexpr int KS = HD / 16;          // k-steps of Q K^T
    constexpr int NT = G_TK / 8;         // position n-tiles per stage
    constexpr int DT = HD / 8;           // dim n-tiles of the output
    constexpr int TILE_BYTES = G_TK * HD * 2;
    const int grp = blockIdx.z, kvh = blockIdx.y;
    // Decode steps launch this kernel as a programmatic dependent of the QKV post-processing: the step descriptor, the row
    // geometry and the prompt K/V were all written before that kernel started, so the first K/V tiles are requested while
    // it still runs; q is read after grid_dep_wait().  Every CTA waits on every path (a grid that ended before the kernel
    // it depends on would let the next kernel start too early).  The prefill form reads K/V of this very pass: it waits first.
    if (FINAL) grid_dep_wait();
    if (grp >= sd->n_groups) { grid_dep_wait(); return; }
    // group_row_start holds this pass's groups from entry 0 on (decode: the copy prep_decode_rows leaves in the workspace)
    const int row0 = group_row_start[grp], n_rows = group_row_start[grp + 1] - row0;
    const int n_rep = Hq / Hkv;
    const int n_parts = FINAL ? 1 : part.n_parts;
    const int q_tiles = gridDim.x / n_parts;
    const int my_part = blockIdx.x / q_tiles;
    const int q0 = (blockIdx.x - my_part * q_tiles) * G_QROWS;
    if (q0 >= n_rows * n_rep) { grid_dep_wait(); return; }

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + G_STAGES * 2 * TILE_BYTES);
    __shared__ int s_abort;
    __shared__ int s_maxlen;
    const uint32_t tiles_u32 = smem_u32(tiles), full0 = smem_u32(bars), empty0 = full0 + 8 * G_STAGES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, G_THREADS / 32); }
        s_abort = 0;
        s_maxlen = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // Decode: the rows of a group share their prompt, so the visible prompt length is known from the group's first
    // row and the first K/V tiles are requested before anything else is loaded.  Prefill: every row sees its own
    // prefix; the longest one of the tile is found below.
    const int64_t kv_start = g.p_start[row0];
    const int64_t krow0 = (((int64_t)layer * 2 + 0) * Hkv + kvh) * n_slots + kv_start;
    const int64_t vrow0 = (((int64_t)layer * 2 + 1) * Hkv + kvh) * n_slots + kv_start;
    auto issue = [&](int tile, int stage) {
        const uint32_t kb = tiles_u32 + stage * 2 * TILE_BYTES, vb = kb + TILE_BYTES;
        mbar_arrive_expect_tx(full0 + 8 * stage, 2 * TILE_BYTES);
#pragma unroll
        for (int b = 0; b < HD / 64; ++b) {
            tma_load_2d(kb + b * (G_TK * 128), &kv_map, full0 + 8 * stage, b * 64, (int)(krow0 + (int64_t)tile * G_TK));
            tma_load_2d(vb + b * (G_TK * 128), &kv_map, full0 + 8 * stage, b * 64, (int)(vrow0 + (int64_t)tile * G_TK));
        }
    };
    int max_len = 0, tile0 = 0, n_tiles = 0;
    auto set_range = [&](int len) {
        max_len = len;
        const int n_tiles_all = (max_len + G_TK - 1) / G_TK;
        const int tiles_per_part = (n_tiles_all + n_parts - 1) / n_parts;
        tile0 = my_part * tiles_per_part;                                // this CTA covers tiles [tile0, tile0 + n_tiles)
        n_tiles = max(0, min(n_tiles_all, tile0 + tiles_per_part) - tile0);
    };
    if (!FINAL) {
        set_range(g.p_len[row0]);
        if (threadIdx.x == 0)
            for (int t = 0; t < G_STAGES && t < n_tiles; ++t) issue(tile0 + t, t);
        grid_dep_wait();
    }

    // this thread's two query rows: qr = q0 + warp*16 + lane/4 (+8); query row qr = (rollout row qr / n_rep, head qr % n_rep)
    int lim[2], grow[2], head[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int qr = q0 + warp * 16 + (lane >> 2) + 8 * i;
        const bool valid = qr < n_rows * n_rep;
        grow[i] = valid ? row0 + qr / n_rep : -1;
        head[i] = kvh * n_rep + (valid ? qr % n_rep : 0);
        lim[i] = valid ? g.p_len[grow[i]] : 0;
        if (!FINAL) lim[i] = min(lim[i], max_len);
    }
    if (FINAL) {
        int mx = max(lim[0], lim[1]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) atomicMax(&s_maxlen, mx);
    }
    // Q fragments (A operand), straight from global memory
    uint32_t qa[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            uint32_t lo = 0, hi = 0;
            if (grow[i] >= 0) {
                const __nv_bfloat16* p = q + ((size_t)grow[i] * Hq + head[i]) * HD + ks * 16 + (lane & 3) * 2;
                lo = *reinterpret_cast<const uint32_t*>(p);
                hi = *reinterpret_cast<const uint32_t*>(p + 8);
            }
            qa[ks][i] = lo;          // a0 (row), a1 (row + 8)
            qa[ks][2 + i] = hi;      // a2, a3: dims + 8
        }
    }
    if (FINAL) {
        __syncthreads();
        set_range(s_maxlen);
        if (threadIdx.x == 0)
            for (int t = 0; t < G_STAGES && t < n_tiles; ++t) issue(tile0 + t, t);
    }

    float o[DT][4];
#pragma unroll
    for (int t = 0; t < DT; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
    bool ok = true;

    for (int lt = 0; lt < n_tiles; ++lt) {
        const int tile = tile0 + lt;
        const int stage = lt % G_STAGES;
        const uint32_t phase = (uint32_t)(lt / G_STAGES) & 1u;
        if (!mbar_wait(full0 + 8 * stage, phase, &s_abort)) { ok = false; break; }
        const uint32_t kb = tiles_u32 + stage * 2 * TILE_BYTES, vb = kb + TILE_BYTES;
        // S = Q K^T for 64 positions
        float s[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                const int mat = lane >> 3;
                const int r = np * 16 + (lane & 7) + ((mat >> 1) << 3), d = ks * 16 + ((mat & 1) << 3);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kb + tile_off<G_TK>(r, d), b0, b1, b2, b3);
                mma_f16(s[2 * np], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                mma_f16(s[2 * np + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
            }
        }
        // mask, online softmax (rows lane/4 and lane/4 + 8; a row lives in the four lanes of a quad)
        const int pos0 = tile * G_TK + (lane & 3) * 2;
        float bmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int pos = pos0 + nt * 8 + (c & 1);
                const float v = pos < lim[c >> 1] ? s[nt][c] * scale_log2 : -INFINITY;
                s[nt][c] = v;
                bmax[c >> 1] = fmaxf(bmax[c >> 1], v);
            }
        }
        float corr[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            bmax[i] = fmaxf(bmax[i], __shfl_xor_sync(0xffffffffu, bmax[i], 1));
            bmax[i] = fmaxf(bmax[i], __shfl_xor_sync(0xffffffffu, bmax[i], 2));
            const float mnew = fmaxf(mrow[i], bmax[i]);
            corr[i] = exp2_safe(mrow[i], mnew);
            mrow[i] = mnew;
            lrow[i] *= corr[i];
        }
#pragma unroll
        for (int t = 0; t < DT; ++t) { o[t][0] *= corr[0]; o[t][1] *= corr[0]; o[t][2] *= corr[1]; o[t][3] *= corr[1]; }
        uint32_t pa[NT / 2][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float p[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) { p[c] = exp2_safe(s[nt][c], mrow[c >> 1]); lrow[c >> 1] += p[c]; }
            pa[nt >> 1][(nt & 1) * 2 + 0] = pack_f16(p[0], p[1]);
            pa[nt >> 1][(nt & 1) * 2 + 1] = pack_f16(p[2], p[3]);
        }
        // rows of V beyond the longest visible prefix of this CTA may be uninitialised memory: their P is 0, but
        // 0 * NaN would poison the sum, so positions >= max_len are never multiplied (k-steps past it are skipped)
        const int valid_in_tile = min(G_TK, max_len - tile * G_TK);
#pragma unroll
        for (int kk = 0; kk < G_TK / 16; ++kk) {
            if (kk * 16 >= valid_in_tile) break;
            const bool ragged = kk * 16 + 16 > valid_in_tile;      // block-uniform
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                const int mat = lane >> 3;
                const int r = kk * 16 + (lane & 7) + ((mat & 1) << 3), d = dp * 16 + ((mat >> 1) << 3);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vb + tile_off<G_TK>(r, d), b0, b1, b2, b3);
                if (ragged) {
                    // zero the V values of positions >= valid_in_tile: after the transposing load a thread holds
                    // positions kk*16 + (lane%4)*2 + {0,1} in b0/b2 and + 8 in b1/b3
                    const int p = kk * 16 + (lane & 3) * 2;
                    const uint32_t m_lo = (p < valid_in_tile ? 0x0000ffffu : 0u) | (p + 1 < valid_in_tile ? 0xffff0000u : 0u);
                    const uint32_t m_hi = (p + 8 < valid_in_tile ? 0x0000ffffu : 0u) | (p + 9 < valid_in_tile ? 0xffff0000u : 0u);
                    b0 &= m_lo; b2 &= m_lo; b1 &= m_hi; b3 &= m_hi;
                }
                mma_f16(o[2 * dp], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], b0, b1);
                mma_f16(o[2 * dp + 1], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], b2, b3);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8 * stage);
        if (threadIdx.x == 0 && lt + G_STAGES < n_tiles) {
            if (!mbar_wait(empty0 + 8 * stage, phase, &s_abort)) { ok = false; break; }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(tile + G_STAGES, stage);
        }
    }
    if (!ok) { s_abort = 1; set_error(err, DEV_ERR_WAIT_TIMEOUT); }

    // row sums live spread over the quad
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        lrow[i] += __shfl_xor_sync(0xffffffffu, lrow[i], 1);
        lrow[i] += __shfl_xor_sync(0xffffffffu, lrow[i], 2);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        if (grow[i] < 0) continue;
        const size_t rh = (size_t)grow[i] * Hq + head[i];
        if (FINAL) {
            const float inv = lrow[i] > 0.f ? 1.f / lrow[i] : 0.f;
#pragma unroll
            for (int t = 0; t < DT; ++t) {
                const float y0 = o[t][2 * i] * inv, y1 = o[t][2 * i + 1] * inv;
                const size_t at = rh * HD + t * 8 + (lane & 3) * 2;
                if (out_lo == nullptr) {         // the output projection takes IEEE half operands
                    *reinterpret_cast<uint32_t*>(out + at) = pack_f16_guard(y0, y1, err);
                } else {
                    *reinterpret_cast<uint32_t*>(out + at) = pack_bf16(y0, y1);
                    // rounding remainder, consumed as a second bf16 operand by the output projection
                    *reinterpret_cast<uint32_t*>(out_lo + at) = pack_bf16(y0 - __bfloat162float(__float2bfloat16_rn(y0)),
                                                                          y1 - __bfloat162float(__float2bfloat16_rn(y1)));
                }
            }
        } else {
            const size_t ph = (size_t)my_part * part.stride + rh;
            if ((lane & 3) == 0) { part.m[ph] = mrow[i]; part.l[ph] = lrow[i]; }
            if (n_tiles > 0) {          // an empty range leaves (m, l) = (-inf, 0); its output is never read
#pragma unroll
                for (int t = 0; t < DT; ++t)
                    *reinterpret_cast<float2*>(part.o + ph * HD + t * 8 + (lane & 3) * 2) = make_float2(o[t][2 * i], o[t][2 * i + 1]);
            }
        }
    }
    if (s_abort) {      // let copies still in flight land before the shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Suffix kernel
// ---------------------------------------------------------------------------------------------
constexpr int S_WARPS = 4;
constexpr int S_TP = 32;            // positions per stage
constexpr int S_STAGES = 3;
template <int HD> constexpr int suffix_smem_bytes() {
    return S_WARPS * (S_STAGES * 2 * S_TP * HD * 2 + 8 * HD * 4) + 1024 + 256;
}

// With few rollouts there are about as many (rollout, KV head) streams as warps on the GPU, and one stream more than
// warps doubles the kernel's time.  The suffix of a rollout is therefore cut into ranges of tiles ("chunks") that
// are spread over the warps; every chunk leaves its own record.  Tiles per chunk (ct) and chunk slots per (row, KV
// head) item (cpi) for a step whose longest suffix has max_slen slots: among 1..MAX_SUFFIX_CHUNKS chunks per item, the
// choice that minimises (units the busiest warp gets) x (tiles per unit + 2), the + 2 standing for the fixed cost of a
// unit (length lookup, first TMA round trip, record) in tile times.  The same value serves every row of the step, and
// the merge kernel recomputes it from the same inputs.
struct SuffixPlan { int ct, cpi; };
__device__ __forceinline__ SuffixPlan suffix_plan(int max_slen, int n_items, int n_warps) {
    const int ntiles = max(1, (max_slen + S_TP - 1) / S_TP);
    SuffixPlan best{ntiles, 1};
    long long best_cost = -1;
    for (int c = 1; c <= MAX_SUFFIX_CHUNKS; ++c) {
        const int ct = (ntiles + c - 1) / c;
        const int cc = (ntiles + ct - 1) / ct;
        const long long cost = (long long)((n_items * cc + n_warps - 1) / max(n_warps, 1)) * (ct + 2);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = SuffixPlan{ct, cc}; }
    }
    return best;
}
__device__ __forceinline__ int suffix_chunks(int n, int ct) {             // records a row with n suffix slots leaves
    const int ntiles = (n + S_TP - 1) / S_TP;
    return (ntiles + ct - 1) / ct;
}

template <int HD>
__global__ void __launch_bounds__(S_WARPS * 32, 1)
attn_suffix_kernel(const __grid_constant__ CUtensorMap kv_map, const StepDesc* __restrict__ sd, int64_t n_slots, int Hq, int Hkv,
                   int layer, const __nv_bfloat16* __restrict__ q, RowGeom g, float scale_log2, PrefixPartial part, int32_t* err) {
    constexpr int KS = HD / 16;                   // k-steps of K Q^T
    constexpr int DT = HD / 16;                   // 16-dim m-tiles of O^T
    constexpr int TILE_BYTES = S_TP * HD * 2;
    constexpr int WARP_BYTES = S_STAGES * 2 * TILE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t* my_tiles = base + warp * WARP_BYTES;
    float* obuf = reinterpret_cast<float*>(base + S_WARPS * WARP_BYTES) + warp * 8 * HD;      // [8 heads][HD]
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + S_WARPS * (WARP_BYTES + 8 * HD * 4)) + warp * S_STAGES;
    __shared__ float s_ml[S_WARPS][16];
    __shared__ int s_abort;
    const uint32_t tiles_u32 = smem_u32(my_tiles), full0 = smem_u32(bars);
    const int n_rep = Hq / Hkv;

    if (threadIdx.x == 0) s_abort = 0;
    if (lane == 0) {
        for (int s = 0; s < S_STAGES; ++s) mbar_init(full0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // work unit u = (item, chunk), item = (row, kv head); units of one item are consecutive, so they land on different warps
    const int max_slen = *g.max_slen;
    const SuffixPlan sp = suffix_plan(max_slen, sd->n_rows * Hkv, part.n_suffix_warps);
    const int ct = sp.ct, cpi = sp.cpi;                                                            // tiles per chunk, unit slots per item
    const int n_items = sd->n_rows * Hkv * cpi;
    const int item_stride = gridDim.x * S_WARPS;
    const int first_item = blockIdx.x * S_WARPS + warp;
    // tile range [t0, t1) of unit u for a row with n suffix slots; empty when the row has fewer chunks
    auto unit_range = [&](int u, int n, int& t0, int& t1) {
        const int ntiles = (n + S_TP - 1) / S_TP;
        t0 = min(ntiles, (u % cpi) * ct);
        t1 = min(ntiles, t0 + ct);
    };

    // producer cursor (tracked identically by every lane; lane 0 issues)
    int p_item = first_item, p_tile = 0, p_ntiles = 0;
    int64_t p_krow = 0, p_vrow = 0;
    auto p_load_item = [&]() {
        while (p_item < n_items) {
            const int it = p_item / cpi;
            const int row = it / Hkv, kvh = it - row * Hkv;
            int t0, t1;
            unit_range(p_item, g.s_len[row], t0, t1);
            if (t1 > t0) {
                p_ntiles = t1;
                const int64_t st = g.s_start[row];
                p_krow = (((int64_t)layer * 2 + 0) * Hkv + kvh) * n_slots + st;
                p_vrow = (((int64_t)layer * 2 + 1) * Hkv + kvh) * n_slots + st;
                p_tile = t0;
                return;
            }
            p_item += item_stride;
        }
        p_ntiles = 0;
    };
    int issued = 0;
    auto p_issue = [&]() {          // loads the producer cursor's tile into the next ring slot and advances the cursor
        const int stage = issued % S_STAGES;
        if (lane == 0) {
            const uint32_t kb = tiles_u32 + stage * 2 * TILE_BYTES, vb = kb + TILE_BYTES;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            mbar_arrive_expect_tx(full0 + 8 * stage, 2 * TILE_BYTES);
#pragma unroll
            for (int b = 0; b < HD / 64; ++b) {
                tma_load_2d(kb + b * (S_TP * 128), &kv_map, full0 + 8 * stage, b * 64, (int)(p_krow + (int64_t)p_tile * S_TP));
                tma_load_2d(vb + b * (S_TP * 128), &kv_map, full0 + 8 * stage, b * 64, (int)(p_vrow + (int64_t)p_tile * S_TP));
            }
        }
        ++issued;
        if (++p_tile == p_ntiles) { p_item += item_stride; p_load_item(); }
    };
    p_load_item();
    for (int i = 0; i < S_STAGES && p_item < n_items; ++i) p_issue();

    int consumed = 0;
    bool ok = true;
    // Q^T fragments (B operand): head = lane / 4, dims ks*16 + (lane%4)*2 (+8).  The next item's fragments and
    // length are fetched while the current item streams, so that an item does not start with a global-memory stall.
    uint32_t qn[KS][2];
    int n_next = 0;
    auto fetch_item = [&](int item) {
        if (item >= n_items) return;
        const int it = item / cpi;
        const int row = it / Hkv, kvh = it - row * Hkv;
        n_next = g.s_len[row];
        const int hq = lane >> 2;
        const __nv_bfloat16* qp = q + ((size_t)row * Hq + (size_t)kvh * n_rep + hq) * HD + (lane & 3) * 2;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            qn[ks][0] = hq < n_rep ? *reinterpret_cast<const uint32_t*>(qp + ks * 16) : 0u;
            qn[ks][1] = hq < n_rep ? *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8) : 0u;
        }
    };
    fetch_item(first_item);
    for (int item = first_item; item < n_items && ok; item += item_stride) {
        const int it = item / cpi, chunk = item - it * cpi;
        const int row = it / Hkv, kvh = it - row * Hkv;
        const int n = n_next;
        int t0, t1;
        unit_range(item, n, t0, t1);
        uint32_t qb[KS][2];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) { qb[ks][0] = qn[ks][0]; qb[ks][1] = qn[ks][1]; }
        fetch_item(item + item_stride);
        if (t1 <= t0) continue;      // this row has fewer chunks: nothing to leave
        float o[DT][4];
#pragma unroll
        for (int t = 0; t < DT; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
        float mh[2] = {-INFINITY, -INFINITY}, lh[2] = {0.f, 0.f};      // heads (lane%4)*2 + {0, 1}

        for (int tile = t0; tile < t1; ++tile) {
            const int stage = consumed % S_STAGES;
            const uint32_t phase = (uint32_t)(consumed / S_STAGES) & 1u;
            if (!mbar_wait(full0 + 8 * stage, phase, &s_abort)) { ok = false; break; }
            const uint32_t kb = tiles_u32 + stage * 2 * TILE_BYTES, vb = kb + TILE_BYTES;
            const int valid = min(S_TP, n - tile * S_TP);
            // S^T = K Q^T : positions on M (two 16-row tiles), heads on N
            float s[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                s[mt][0] = s[mt][1] = s[mt][2] = s[mt][3] = 0.f;
                if (mt * 16 < valid) {
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int mat = lane >> 3;
                        const int r = mt * 16 + (lane & 7) + ((mat & 1) << 3), d = ks * 16 + ((mat >> 1) << 3);
                        uint32_t a0, a1, a2, a3;
                        ldsm_x4(kb + tile_off<S_TP>(r, d), a0, a1, a2, a3);
                        mma_f16(s[mt], a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
                    }
                }
            }
            // mask + per-head block max (a head's column is spread over the 8 lanes sharing lane % 4)
            float bmax[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int pos = mt * 16 + (lane >> 2) + ((c >> 1) << 3);
                    const float v = pos < valid ? s[mt][c] * scale_log2 : -INFINITY;
                    s[mt][c] = v;
                    bmax[c & 1] = fmaxf(bmax[c & 1], v);
                }
            }
            float corr[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                bmax[i] = fmaxf(bmax[i], __shfl_xor_sync(0xffffffffu, bmax[i], 4));
                bmax[i] = fmaxf(bmax[i], __shfl_xor_sync(0xffffffffu, bmax[i], 8));
                bmax[i] = fmaxf(bmax[i], __shfl_xor_sync(0xffffffffu, bmax[i], 16));
                const float mnew = fmaxf(mh[i], bmax[i]);
                corr[i] = exp2_safe(mh[i], mnew);
                mh[i] = mnew;
                lh[i] *= corr[i];
            }
#pragma unroll
            for (int t = 0; t < DT; ++t) { o[t][0] *= corr[0]; o[t][1] *= corr[1]; o[t][2] *= corr[0]; o[t][3] *= corr[1]; }
            // O^T += V^T P^T, 16 positions per k-step; P^T fragments come from S^T through movmatrix
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                if (mt * 16 >= valid) break;
                float p[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) { p[c] = exp2_safe(s[mt][c], mh[c & 1]); lh[c & 1] += p[c]; }
                const uint32_t b0 = movmatrix_t(pack_f16(p[0], p[1]));
                const uint32_t b1 = movmatrix_t(pack_f16(p[2], p[3]));
                const bool ragged = mt * 16 + 16 > valid;              // warp-uniform
#pragma unroll
                for (int dt = 0; dt < DT; ++dt) {
                    const int mat = lane >> 3;
                    const int r = mt * 16 + (lane & 7) + ((mat >> 1) << 3), d = dt * 16 + ((mat & 1) << 3);
                    uint32_t a0, a1, a2, a3;
                    ldsm_x4_t(vb + tile_off<S_TP>(r, d), a0, a1, a2, a3);
                    if (ragged) {
                        // slots past the rollout's last token may be uninitialised: zero them (0 * NaN = NaN).
                        // After the transposing load a thread holds positions mt*16 + (lane%4)*2 + {0,1} in a0/a1, + 8 in a2/a3.
                        const int pp = mt * 16 + (lane & 3) * 2;
                        const uint32_t m_lo = (pp < valid ? 0x0000ffffu : 0u) | (pp + 1 < valid ? 0xffff0000u : 0u);
                        const uint32_t m_hi = (pp + 8 < valid ? 0x0000ffffu : 0u) | (pp + 9 < valid ? 0xffff0000u : 0u);
                        a0 &= m_lo; a1 &= m_lo; a2 &= m_hi; a3 &= m_hi;
                    }
                    mma_f16(o[dt], a0, a1, a2, a3, b0, b1);
                }
            }
            ++consumed;
            __syncwarp();
            if (p_item < n_items) p_issue();      // refill the slot just drained
        }
        if (!ok) break;

        // reduce the per-thread partial sums of each head over the 8 lanes sharing lane % 4
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            lh[i] += __shfl_xor_sync(0xffffffffu, lh[i], 4);
            lh[i] += __shfl_xor_sync(0xffffffffu, lh[i], 8);
            lh[i] += __shfl_xor_sync(0xffffffffu, lh[i], 16);
        }
        if (lane < 4) {
            s_ml[warp][lane * 2] = mh[0]; s_ml[warp][lane * 2 + 1] = mh[1];
            s_ml[warp][8 + lane * 2] = lh[0]; s_ml[warp][8 + lane * 2 + 1] = lh[1];
        }
        // O^T fragment (dims dt*16 + lane/4 (+8), heads (lane%4)*2 + {0,1}) -> obuf[head][dim]
#pragma unroll
        for (int dt = 0; dt < DT; ++dt) {
            const int d = dt * 16 + (lane >> 2), hh = (lane & 3) * 2;
            obuf[hh * HD + d] = o[dt][0];
            obuf[(hh + 1) * HD + d] = o[dt][1];
            obuf[hh * HD + d + 8] = o[dt][2];
            obuf[(hh + 1) * HD + d + 8] = o[dt][3];
        }
        __syncwarp();
        // leave this chunk as record number part.n_parts + chunk, next to the prefix records; attn_merge_kernel combines them
        constexpr int EPL = HD / 32;
        const size_t base = (size_t)(part.n_parts + chunk) * part.stride + (size_t)row * Hq + (size_t)kvh * n_rep;
        if (lane < n_rep) { part.m[base + lane] = s_ml[warp][lane]; part.l[base + lane] = s_ml[warp][8 + lane]; }
        for (int j = 0; j < n_rep; ++j) {
            float* dst = part.o + (base + j) * HD + lane * EPL;
            const float* src = obuf + j * HD + lane * EPL;
            if (EPL == 4) *reinterpret_cast<float4*>(dst) = *reinterpret_cast<const float4*>(src);
            else *reinterpret_cast<float2*>(dst) = *reinterpret_cast<const float2*>(src);
        }
        __syncwarp();
    }
    if (!ok) { s_abort = 1; if (lane == 0) set_error(err, DEV_ERR_WAIT_TIMEOUT); }
    // drain: tiles issued but not consumed must land before the shared memory is released
    while (ok && consumed < issued) {
        const int stage = consumed % S_STAGES;
        if (!mbar_wait(full0 + 8 * stage, (uint32_t)(consumed / S_STAGES) & 1u, &s_abort)) break;
        ++consumed;
    }
    if (s_abort) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Merge of the prefix records 0 .. n_parts-1 and the suffix record n_parts of every (row, query head) by their
// log-sum-exp:  M = max m_i,  out = sum_i O_i 2^(m_i - M) / sum_i l_i 2^(m_i - M).  Records are added in index order.
// One warp per (row, head); a lane owns HD/32 consecutive dims.
// ---------------------------------------------------------------------------------------------
// rh = row * Hq + head (the caller keeps it below n_live * Hq).  ct = tiles per suffix chunk of this step (suffix_plan);
// n_load > 0 = how many records to request: every record index the step can have produced (part.n_parts + chunk slots per
// item), so that the loads do not wait for the row's suffix length; records past the row's own count are ignored.
// STREAM: wait for the suffix length and request the row's own records only, one after the other (n_load is not used).
template <int HD, bool STREAM = false>
__device__ __forceinline__ void merge_item_warp(int lane, size_t rh, int Hq, const RowGeom& g, const PrefixPartial& part, int ct, int n_load,
                                                __nv_bfloat16* __restrict__ out, __nv_bfloat16* __restrict__ out_lo, int32_t* err) {
    constexpr int EPL = HD / 32;
    const int row = (int)(rh / Hq);
    const int slen = g.s_len[row];
    float M = -INFINITY;
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    float denom = 0.f;
    if constexpr (STREAM) {
        // Large batches: the row's own records only, streamed (few registers, so many warps are resident): first the
        // largest m, then the weighted sums in index order -- the same operations in the same order as below.
        const int n_own = part.n_parts + suffix_chunks(slen, ct);
        for (int i = 0; i < n_own; ++i) M = fmaxf(M, part.m[(size_t)i * part.stride + rh]);
#pragma unroll 2
        for (int i = 0; i < n_own; ++i) {
            const float w = exp2_safe(part.m[(size_t)i * part.stride + rh], M);
            if (w > 0.f) {
                denom += part.l[(size_t)i * part.stride + rh] * w;
                const float* src = part.o + ((size_t)i * part.stride + rh) * HD + lane * EPL;
                if (EPL == 4) {
                    const float4 v = *reinterpret_cast<const float4*>(src);
                    acc[0] += v.x * w; acc[1] += v.y * w; acc[2] += v.z * w; acc[3] += v.w * w;
                } else {
                    const float2 v = *reinterpret_cast<const float2*>(src);
                    acc[0] += v.x * w; acc[1] += v.y * w;
                }
            }
        }
    } else {
    float mi[MAX_RECORDS], li[MAX_RECORDS];
    float ov[MAX_RECORDS][EPL];
#pragma unroll
    for (int i = 0; i < MAX_RECORDS; ++i) {
        const bool ld = i < n_load;
        mi[i] = ld ? part.m[(size_t)i * part.stride + rh] : -INFINITY;
        li[i] = ld ? part.l[(size_t)i * part.stride + rh] : 0.f;
        const float* src = part.o + ((size_t)i * part.stride + rh) * HD + lane * EPL;
        if (EPL == 4) {
            const float4 v = ld ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
            ov[i][0] = v.x; ov[i][1] = v.y; ov[i][2] = v.z; ov[i][3] = v.w;
        } else {
            const float2 v = ld ? *reinterpret_cast<const float2*>(src) : make_float2(0.f, 0.f);
            ov[i][0] = v.x; ov[i][1] = v.y;
        }
    }
    const int n_rec = part.n_parts + suffix_chunks(slen, ct);
#pragma unroll
    for (int i = 0; i < MAX_RECORDS; ++i)
        if (i >= n_rec) mi[i] = -INFINITY;           // not a record of this row (stale memory)
#pragma unroll
    for (int i = 0; i < MAX_RECORDS; ++i) M = fmaxf(M, mi[i]);
#pragma unroll
    for (int i = 0; i < MAX_RECORDS; ++i) {
        const float w = exp2_safe(mi[i], M);
        if (i < n_rec && w > 0.f) {          // a record with m = -inf was left by an empty range: its output slice is not defined
            denom += li[i] * w;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[e] += ov[i][e] * w;
        }
    }
    }
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    float lo[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        acc[e] *= inv;
        lo[e] = acc[e] - __bfloat162float(__float2bfloat16_rn(acc[e]));     // rounding remainder: second operand of the O projection
    }
    __nv_bfloat16* dst = out + rh * HD + lane * EPL;
    if (out_lo == nullptr) {                 // the output projection takes IEEE half operands: no remainder needed
        if (EPL == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(pack_f16_guard(acc[0], acc[1], err), pack_f16_guard(acc[2], acc[3], err));
        else *reinterpret_cast<uint32_t*>(dst) = pack_f16_guard(acc[0], acc[1], err);
        return;
    }
    __nv_bfloat16* dst_lo = out_lo + rh * HD + lane * EPL;
    if (EPL == 4) {
        *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]));
        *reinterpret_cast<uint2*>(dst_lo) = make_uint2(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]));
    } else {
        *reinterpret_cast<uint32_t*>(dst) = pack_bf16(acc[0], acc[1]);
        *reinterpret_cast<uint32_t*>(dst_lo) = pack_bf16(lo[0], lo[1]);
    }
}

// Stand-alone form: the grid covers the row bound of the step.
template <int HD, bool STREAM>
__global__ void __launch_bounds__(256) attn_merge_kernel(const StepDesc* __restrict__ sd, int Hq, RowGeom g, PrefixPartial part,
                                                         __nv_bfloat16* __restrict__ out, __nv_bfloat16* __restrict__ out_lo, int32_t* err) {
    const size_t rh = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    grid_dep_launch_dependents();          // the output projection may set itself up and request its first weight tiles
    const int n_live = sd->n_rows;
    if (rh >= (size_t)n_live * Hq) return;
    const SuffixPlan sp = suffix_plan(*g.max_slen, n_live * part.n_kv_heads, part.n_suffix_warps);
    // few items (host: STREAM = false): request every record slot of the step at once (latency); many items: only the row's
    // own records, with few registers (occupancy)
    merge_item_warp<HD, STREAM>(threadIdx.x & 31, rh, Hq, g, part, sp.ct, part.n_parts + sp.cpi, out, out_lo, err);
}

}  // namespace am
}  // namespace pc
