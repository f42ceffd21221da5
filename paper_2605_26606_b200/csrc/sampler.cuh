// Seeded Gumbel-max sampling over the whole vocabulary (temperature T, top_p = 1: an exact categorical draw).
// Philox4x32-10 follows the published definition (Salmon et al., SC'11): one 128-bit block per four
// vocabulary ids, key = seed, counter = (v >> 2, step, rollout, prompt).
#pragma once

#include "common.cuh"

namespace pc {

struct Philox4 { uint32_t x, y, z, w; };

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += W0; k1 += W1;
    }
    return Philox4{c0, c1, c2, c3};
}

// u = ((w >> 9) + 1/2) / 2^23 is exact in float and lies strictly inside (0, 1).
__device__ __forceinline__ float gumbel_from_word(uint32_t w) {
    const float u = ((float)(w >> 9) + 0.5f) * 1.1920928955078125e-07f;   // 2^-23
    return -logf(-logf(u));
}

struct Top2 {
    float best, second;
    int idx;
};

__device__ __forceinline__ void top2_push(Top2& t, float s, int v) {
    // strict ">" keeps the lowest id among equal scores because ids arrive in increasing order per thread
    if (s > t.best) { t.second = t.best; t.best = s; t.idx = v; }
    else if (s > t.second) t.second = s;
}

__device__ __forceinline__ Top2 top2_merge(const Top2& a, const Top2& b) {
    Top2 o;
    const bool a_wins = a.best > b.best || (a.best == b.best && a.idx < b.idx);
    o.best = a_wins ? a.best : b.best;
    o.idx = a_wins ? a.idx : b.idx;
    o.second = fmaxf(a_wins ? b.best : a.best, fmaxf(a.second, b.second));
    return o;
}

__device__ __forceinline__ Top2 top2_warp_reduce(Top2 t) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 other;
        other.best = __shfl_xor_sync(0xffffffffu, t.best, o);
        other.second = __shfl_xor_sync(0xffffffffu, t.second, o);
        other.idx = __shfl_xor_sync(0xffffffffu, t.idx, o);
        t = top2_merge(t, other);
    }
    return t;
}

// One block per row.
__global__ void __launch_bounds__(256) sample_kernel(const StepDesc* __restrict__ sd, int vocab, const float* __restrict__ logits,
                                                     const int32_t* __restrict__ logits_row, float temperature,
                                                     uint32_t k0, uint32_t k1, const int32_t* __restrict__ row_prompt,
                                                     const int32_t* __restrict__ row_rollout, const int32_t* __restrict__ row_step,
                                                     int step_offset, int32_t* __restrict__ out_tokens,
                                                     const int64_t* __restrict__ out_index, int64_t out_index_offset,
                                                     float* __restrict__ out_gap) {
    const int r = blockIdx.x;
    int64_t ro = r;                         // index into the caller's row arrays
    if (sd != nullptr) {
        if (r >= sd->n_rows) return;
        ro += sd->row_off;
    }
    const float* lg = logits + (size_t)(logits_row ? logits_row[ro] : r) * vocab;
    const uint32_t c1 = (uint32_t)(row_step[ro] + step_offset), c2 = (uint32_t)row_rollout[ro], c3 = (uint32_t)row_prompt[ro];
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    const int n_blocks = (vocab + 3) >> 2;
    for (int b = threadIdx.x; b < n_blocks; b += blockDim.x) {
        const Philox4 w = philox4x32_10((uint32_t)b, c1, c2, c3, k0, k1);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int v = b * 4 + i;
            if (v < vocab) top2_push(t, lg[v] / temperature + gumbel_from_word(ww[i]), v);
        }
    }
    t = top2_warp_reduce(t);
    __shared__ Top2 sh[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sh[warp] = t;
    __syncthreads();
    if (warp == 0) {
        Top2 u = lane < (int)(blockDim.x >> 5) ? sh[lane] : Top2{-INFINITY, -INFINITY, 0x7fffffff};
        u = top2_warp_reduce(u);
        if (lane == 0) {
            out_tokens[out_index ? out_index[ro] + out_index_offset : (int64_t)r] = u.idx;
            if (out_gap) out_gap[r] = u.best - u.second;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Two-pass form for small batches: with few rows one block per row leaves most SMs idle, so the vocabulary of a row is
// cut into n_chunks ranges scored by different blocks.  Every range leaves its (best, second, arg-best) in scratch and a
// second kernel folds the ranges in order.  Maxima are exact, so the result is identical to the one-pass kernel's.
// ---------------------------------------------------------------------------------------------
struct Top2Rec { float best, second; int idx; int pad; };

__global__ void __launch_bounds__(256) sample_partial_kernel(const StepDesc* __restrict__ sd, int vocab, int n_chunks,
                                                             const float* __restrict__ logits, const int32_t* __restrict__ logits_row,
                                                             float temperature, uint32_t k0, uint32_t k1,
                                                             const int32_t* __restrict__ row_prompt, const int32_t* __restrict__ row_rollout,
                                                             const int32_t* __restrict__ row_step, int step_offset, Top2Rec* __restrict__ scratch) {
    const int r = blockIdx.x, chunk = blockIdx.y;
    int64_t ro = r;
    if (sd != nullptr) {
        if (r >= sd->n_rows) return;
        ro += sd->row_off;
    }
    const float* lg = logits + (size_t)(logits_row ? logits_row[ro] : r) * vocab;
    const uint32_t c1 = (uint32_t)(row_step[ro] + step_offset), c2 = (uint32_t)row_rollout[ro], c3 = (uint32_t)row_prompt[ro];
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    const int n_blocks = (vocab + 3) >> 2;
    const int per_chunk = (n_blocks + n_chunks - 1) / n_chunks;
    const int b_end = min(n_blocks, (chunk + 1) * per_chunk);
    for (int b = chunk * per_chunk + threadIdx.x; b < b_end; b += blockDim.x) {
        const Philox4 w = philox4x32_10((uint32_t)b, c1, c2, c3, k0, k1);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int v = b * 4 + i;
            if (v < vocab) top2_push(t, lg[v] / temperature + gumbel_from_word(ww[i]), v);
        }
    }
    t = top2_warp_reduce(t);
    __shared__ Top2 sh[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sh[warp] = t;
    __syncthreads();
    if (warp == 0) {
        Top2 u = lane < (int)(blockDim.x >> 5) ? sh[lane] : Top2{-INFINITY, -INFINITY, 0x7fffffff};
        u = top2_warp_reduce(u);
        if (lane == 0) scratch[(size_t)r * n_chunks + chunk] = Top2Rec{u.best, u.second, u.idx, 0};
    }
}

__global__ void sample_reduce_kernel(const StepDesc* __restrict__ sd, int n_rows, int n_chunks, const Top2Rec* __restrict__ scratch,
                                     int32_t* __restrict__ out_tokens, const int64_t* __restrict__ out_index,
                                     int64_t out_index_offset, float* __restrict__ out_gap) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    int64_t ro = r;
    if (sd != nullptr) {
        if (r >= sd->n_rows) return;
        ro += sd->row_off;
    } else if (r >= n_rows) {
        return;
    }
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    for (int c = 0; c < n_chunks; ++c) {
        const Top2Rec x = scratch[(size_t)r * n_chunks + c];
        t = top2_merge(t, Top2{x.best, x.second, x.idx});
    }
    out_tokens[out_index ? out_index[ro] + out_index_offset : (int64_t)r] = t.idx;
    if (out_gap) out_gap[r] = t.best - t.second;
}

constexpr int SAMPLE_MAX_CHUNKS = 32;
// Ranges per row so that about four blocks per SM are in flight; 1 means the one-pass kernel is the better choice.
inline int sample_chunks(int n_rows, int num_sms) {
    const int want = (4 * num_sms + n_rows - 1) / (n_rows > 0 ? n_rows : 1);
    return want < 2 ? 1 : (want > SAMPLE_MAX_CHUNKS ? SAMPLE_MAX_CHUNKS : want);
}

}  // namespace pc
