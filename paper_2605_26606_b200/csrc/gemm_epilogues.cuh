// GEMM epilogues that take over the row-wise kernels around a projection (IEEE-half operand mode, head_dim 128).
// Each walks the accumulator tile of its thread's row itself (kWholeTile, see gemm_tc_kernel); the GEMM must not be
// split along K, so that a tile holds complete sums.
//
//   EpiResNorm    output projection:  h += acc;  a = half(h * gain) for the NEXT RMSNorm, WITHOUT its 1/rms factor;
//                 the row's sum of squares over the tile's columns goes to ssq[tile][row].  The consumer of `a` scales
//                 its accumulators by rstd = rsqrt(sum of the row's ssq entries / d + eps): RMSNorm(h; g) W^T =
//                 rstd * ((h * g) W^T), so the norm kernel between the two GEMMs disappears.
//   EpiSwiGLUNorm gate/up projection of such an operand: (gate, up) *= rstd, then silu(gate) * up.
//   EpiQkvPost    QKV projection: bias, per-head RMSNorm of q and k (Qwen3), RoPE, q to its buffer, K / V to the row's
//                 KV slot -- the arithmetic of qkv_post_kernel, one thread per row and one head (128 columns) at a time.
//                 When the previous layer's down projection ran with EpiResNorm (unsplit: large passes), it also applies
//                 the attention norm's 1/rms, and that layer boundary has no norm kernel either.
#pragma once

#include "gemm_tc.cuh"
#include "kernels_basic.cuh"

namespace pc {

// 1 / rms of a row from the per-tile sums of squares an EpiResNorm GEMM left (entries added in tile order).
__device__ __forceinline__ float rstd_from_ssq(const float* __restrict__ ssq, int n_ssq, int m_stride, int row, int d, float eps) {
    // entries added in tile order; six loads in flight at a time (one at a time would be n_ssq dependent L2 round trips at
    // the head of every tile's epilogue)
    float s = 0.f;
    const float* p = ssq + row;
    int t = 0;
    for (; t + 6 <= n_ssq; t += 6) {
        float x[6];
#pragma unroll
        for (int i = 0; i < 6; ++i) x[i] = p[(size_t)(t + i) * m_stride];
#pragma unroll
        for (int i = 0; i < 6; ++i) s += x[i];
    }
    for (; t < n_ssq; ++t) s += p[(size_t)t * m_stride];
    return rsqrtf(s / (float)d + eps);
}

struct EpiResNorm {
    static constexpr bool kWholeTile = true;
    float* h; int ld;                  // residual stream [rows, ld]
    const float* gain;                 // gains of the RMSNorm that follows
    __half* a;                         // [rows, ld] operand of the next GEMM: half(h * gain)
    float* ssq; int m_stride;          // [tiles of this GEMM][m_stride]
    int32_t* err;
    __device__ __forceinline__ void set_rows(int) {}
    // The residual values of the next 32 columns are requested before the current 32 are worked on: a thread owns a
    // row, so its loads are a latency chain of their own and one chunk's round trip at a time would dominate the tile.
    template <int BN>
    __device__ __forceinline__ void tile(uint32_t taddr, int row, bool live, int n0, int N) const {
        float ss = 0.f;
        int bad = 0;
        const int n_chunks = min(BN, N - n0) >> 5;      // warp-uniform (N is a multiple of 32)
        float* hrow = h + (size_t)(live ? row : 0) * ld + n0;
        float4 cur[8], nxt[8];
        if (live) {
#pragma unroll
            for (int i = 0; i < 8; ++i) cur[i] = reinterpret_cast<const float4*>(hrow)[i];
        }
#pragma unroll 1
        for (int ci = 0; ci < n_chunks; ++ci) {
            const int c = ci << 5;
            if (live && ci + 1 < n_chunks) {
#pragma unroll
                for (int i = 0; i < 8; ++i) nxt[i] = reinterpret_cast<const float4*>(hrow + c + 32)[i];
            }
            float v[32];
            tc::tmem_ld32(taddr + c, v);
            if (live) {
                const float4* gp = reinterpret_cast<const float4*>(gain + n0 + c);
                uint32_t w[16];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float4 x = cur[i];
                    const float4 g = __ldg(gp + i);
                    x.x += v[4 * i]; x.y += v[4 * i + 1]; x.z += v[4 * i + 2]; x.w += v[4 * i + 3];
                    cur[i] = x;
                    ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                    const float y0 = x.x * g.x, y1 = x.y * g.y, y2 = x.z * g.z, y3 = x.w * g.w;
                    bad |= half_bad(y0) | half_bad(y1) | half_bad(y2) | half_bad(y3);
                    const __half2 p0 = __floats2half2_rn(half_clamp(y0), half_clamp(y1)), p1 = __floats2half2_rn(half_clamp(y2), half_clamp(y3));
                    w[2 * i] = *reinterpret_cast<const uint32_t*>(&p0);
                    w[2 * i + 1] = *reinterpret_cast<const uint32_t*>(&p1);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) reinterpret_cast<float4*>(hrow + c)[i] = cur[i];
                uint4* ap = reinterpret_cast<uint4*>(a + (size_t)row * ld + n0 + c);
#pragma unroll
                for (int i = 0; i < 4; ++i) ap[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
#pragma unroll
                for (int i = 0; i < 8; ++i) cur[i] = nxt[i];
            }
        }
        if (live) {
            ssq[(size_t)(n0 / BN) * m_stride + row] = ss;
            if (bad) set_error(err, DEV_ERR_HALF_RANGE);
        }
    }
};

struct EpiSwiGLUNorm {              // columns (2j, 2j+1) = (gate_j, up_j) of an operand that still lacks its 1/rms factor
    static constexpr bool kWholeTile = true;
    __half* out; int ld;               // [rows, ld = d_ff]
    const float* ssq; int n_ssq, m_stride, d; float eps;
    int32_t* err;
    __device__ __forceinline__ void set_rows(int) {}
    template <int BN>
    __device__ __forceinline__ void tile(uint32_t taddr, int row, bool live, int n0, int N) const {
        const float rstd = live ? rstd_from_ssq(ssq, n_ssq, m_stride, row, d, eps) : 0.f;
        int bad = 0;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            if (n0 + c >= N) break;
            float v[32];
            tc::tmem_ld32(taddr + c, v);
            if (!live) continue;
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float g0 = v[4 * i] * rstd, u0 = v[4 * i + 1] * rstd, g1 = v[4 * i + 2] * rstd, u1 = v[4 * i + 3] * rstd;
                const float y0 = g0 / (1.f + expf(-g0)) * u0, y1 = g1 / (1.f + expf(-g1)) * u1;
                bad |= half_bad(y0) | half_bad(y1);
                const __half2 p = __floats2half2_rn(half_clamp(y0), half_clamp(y1));
                w[i] = *reinterpret_cast<const uint32_t*>(&p);
            }
            uint4* dst = reinterpret_cast<uint4*>(out + (size_t)row * ld + ((n0 + c) >> 1));
            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
        if (live && bad) set_error(err, DEV_ERR_HALF_RANGE);
    }
};

struct EpiQkvPost {
    static constexpr bool kWholeTile = true;
    static constexpr int HD = 128;
    int Hq, Hkv, layer;
    const float* bias;                 // [(Hq + 2 Hkv) * HD] or nullptr
    const float* q_gain;               // [HD] or nullptr (no QK-norm)
    const float* k_gain;
    float eps;
    const float2* rope;                // [rows, HD / 2] (cos, sin)
    RowGeom g;
    KvArena prompt_arena, suffix_arena;
    __half* q_out;                     // [rows, Hq * HD]
    int32_t* err;
    // n_ssq > 0: the operand is half(h * gain) without the attention norm's 1/rms (left by an EpiResNorm down projection
    // together with the row's sums of squares); the accumulators are scaled by it before the bias is added
    const float* ssq; int n_ssq, m_stride, d_model;
    __device__ __forceinline__ void set_rows(int) {}
    template <int BN>
    __device__ __forceinline__ void tile(uint32_t taddr, int row, bool live, int n0, int N) const {
        static_assert(BN % HD == 0, "QKV tiles must hold whole heads");
        int64_t slot = -1;
        int to_suffix = 0;
        float rstd = 1.f;
        if (live) {
            slot = g.wslot[row]; to_suffix = g.warena[row];
            if (n_ssq > 0) rstd = rstd_from_ssq(ssq, n_ssq, m_stride, row, d_model, eps);
        }
#pragma unroll 1
        for (int ho = 0; ho < BN; ho += HD) {
            if (n0 + ho >= N) break;                 // warp-uniform
            float x[HD];
#pragma unroll
            for (int c = 0; c < HD; c += 32) tc::tmem_ld32(taddr + ho + c, x + c);
            if (!live) continue;
            const int head = (n0 + ho) / HD;
            const bool is_q = head < Hq, is_k = !is_q && head < Hq + Hkv;
            if (n_ssq > 0) {
#pragma unroll
                for (int i = 0; i < HD; ++i) x[i] *= rstd;
            }
            if (bias != nullptr) {
                const float4* bp = reinterpret_cast<const float4*>(bias + (size_t)head * HD);
#pragma unroll
                for (int i = 0; i < HD / 4; ++i) {
                    const float4 b = bp[i];
                    x[4 * i] += b.x; x[4 * i + 1] += b.y; x[4 * i + 2] += b.z; x[4 * i + 3] += b.w;
                }
            }
            if (is_q || is_k) {
                const float* gain = is_q ? q_gain : k_gain;
                if (gain != nullptr) {
                    float ss = 0.f;
#pragma unroll
                    for (int i = 0; i < HD; ++i) ss += x[i] * x[i];
                    const float rstd = rsqrtf(ss / (float)HD + eps);
#pragma unroll
                    for (int i = 0; i < HD; ++i) x[i] = x[i] * rstd * gain[i];
                }
                const float4* cp = reinterpret_cast<const float4*>(rope + (size_t)row * (HD / 2));      // two (cos, sin) pairs per load
#pragma unroll
                for (int i = 0; i < HD / 2; i += 2) {
                    const float4 cs = cp[i >> 1];
                    const float a0 = x[i], b0 = x[i + HD / 2], a1 = x[i + 1], b1 = x[i + 1 + HD / 2];
                    x[i] = a0 * cs.x - b0 * cs.y;
                    x[i + HD / 2] = b0 * cs.x + a0 * cs.y;
                    x[i + 1] = a1 * cs.z - b1 * cs.w;
                    x[i + 1 + HD / 2] = b1 * cs.z + a1 * cs.w;
                }
            }
            __half* dst;
            if (is_q) {
                dst = q_out + ((size_t)row * Hq + head) * HD;
            } else {
                if (slot < 0) continue;
                const KvArena ar = to_suffix ? suffix_arena : prompt_arena;
                const int kvh = is_k ? head - Hq : head - Hq - Hkv;
                const int64_t plane = ((int64_t)layer * 2 + (is_k ? 0 : 1)) * Hkv + kvh;
                dst = reinterpret_cast<__half*>(ar.base) + (plane * ar.n_slots + slot) * HD;
            }
            int bad = 0;
#pragma unroll
            for (int i = 0; i < HD; i += 8) {
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float y0 = x[i + 2 * j], y1 = x[i + 2 * j + 1];
                    bad |= half_bad(y0) | half_bad(y1);
                    const __half2 p = __floats2half2_rn(half_clamp(y0), half_clamp(y1));
                    w[j] = *reinterpret_cast<const uint32_t*>(&p);
                }
                *reinterpret_cast<uint4*>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            if (bad) set_error(err, DEV_ERR_HALF_RANGE);
        }
    }
};

}  // namespace pc
