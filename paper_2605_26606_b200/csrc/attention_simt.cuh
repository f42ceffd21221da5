// Straightforward attention for one query position per row: every (row, KV head) block walks the row's prompt
// slots and then its suffix slots with an online softmax, serving all query heads that share the KV head.
// It is the plain-FP32 form: used for float32 models, for prefill, and as the cross-check of the
// shared-prefix tensor-core kernels.
#pragma once

#include "common.cuh"
#include "kernels_basic.cuh"

namespace pc {

constexpr int ATTN_MAX_REP = 8;   // query heads per KV head supported

// HD = head_dim (64 or 128); each lane owns EPL = HD / 32 consecutive dims of every K/V row.
template <typename T, int HD>
__global__ void __launch_bounds__(128) attn_row_simt_kernel(const StepDesc* __restrict__ sd, int Hq, int Hkv, int layer, const T* __restrict__ q,
                                                            RowGeom g, KvArena prompt_arena, KvArena suffix_arena,
                                                            float scale, T* __restrict__ out) {
    constexpr int EPL = HD / 32;
    constexpr int NW = 4;
    const int r = blockIdx.x, kvh = blockIdx.y;
    if (r >= sd->n_rows) return;
    const int n_rep = Hq / Hkv;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    float qf[ATTN_MAX_REP][EPL];
    float acc[ATTN_MAX_REP][EPL];
    float mx[ATTN_MAX_REP], ls[ATTN_MAX_REP];
#pragma unroll
    for (int j = 0; j < ATTN_MAX_REP; ++j) {
        mx[j] = -INFINITY; ls[j] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) { acc[j][e] = 0.f; qf[j][e] = 0.f; }
        if (j < n_rep) {
            VecLoad<T, EPL>::load(q + ((size_t)r * Hq + (size_t)kvh * n_rep + j) * HD + lane * EPL, qf[j]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) qf[j][e] *= scale;
        }
    }

    const int64_t kplane = ((int64_t)layer * 2 + 0) * Hkv + kvh, vplane = ((int64_t)layer * 2 + 1) * Hkv + kvh;
#pragma unroll 1
    for (int part = 0; part < 2; ++part) {
        const KvArena ar = part ? suffix_arena : prompt_arena;
        const int64_t start = part ? g.s_start[r] : g.p_start[r];
        const int n = part ? g.s_len[r] : g.p_len[r];
        const T* kb = reinterpret_cast<const T*>(ar.base) + (kplane * ar.n_slots + start) * HD + lane * EPL;
        const T* vb = reinterpret_cast<const T*>(ar.base) + (vplane * ar.n_slots + start) * HD + lane * EPL;
        for (int t = warp; t < n; t += NW) {
            float kf[EPL], vf[EPL];
            VecLoad<T, EPL>::load(kb + (size_t)t * HD, kf);
            VecLoad<T, EPL>::load(vb + (size_t)t * HD, vf);
#pragma unroll
            for (int j = 0; j < ATTN_MAX_REP; ++j) {
                if (j < n_rep) {
                    float s = 0.f;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) s = fmaf(qf[j][e], kf[e], s);
                    s = warp_sum(s);
                    const float mnew = fmaxf(mx[j], s);
                    const float corr = expf(mx[j] - mnew);      // exp(-inf) = 0 on the first position
                    const float p = expf(s - mnew);
                    ls[j] = ls[j] * corr + p;
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[j][e] = fmaf(p, vf[e], acc[j][e] * corr);
                    mx[j] = mnew;
                }
            }
        }
    }

    // merge the four warps' partial softmaxes
    __shared__ float s_m[NW][ATTN_MAX_REP], s_l[NW][ATTN_MAX_REP];
    __shared__ float s_acc[NW][ATTN_MAX_REP][HD];
#pragma unroll
    for (int j = 0; j < ATTN_MAX_REP; ++j) {
        if (j < n_rep) {
            if (lane == 0) { s_m[warp][j] = mx[j]; s_l[warp][j] = ls[j]; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) s_acc[warp][j][lane * EPL + e] = acc[j][e];
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < n_rep * HD; idx += blockDim.x) {
        const int j = idx / HD, e = idx - j * HD;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, s_m[w][j]);
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float c = s_m[w][j] == -INFINITY ? 0.f : expf(s_m[w][j] - M);
            L += s_l[w][j] * c;
            O += s_acc[w][j][e] * c;
        }
        out[((size_t)r * Hq + (size_t)kvh * n_rep + j) * HD + e] = from_f32<T>(L > 0.f ? O / L : 0.f);
    }
}

}  // namespace pc
