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
        // one 32 x 32 -> 64 bit product per multiplier (high and low word of the same multiplication)
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
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

// Same fold when candidates arrive in arbitrary id order: equal scores keep the lowest id.
__device__ __forceinline__ void top2_push_unordered(Top2& t, float s, int v) {
    if (s > t.best || (s == t.best && v < t.idx)) { t.second = t.best; t.best = s; t.idx = v; }
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

// Scores the 4-id blocks b0, b0 + stride, ... < b1 of one row and folds them into t.
//
// Almost every candidate is rejected without evaluating its Gumbel noise: v can enter the thread's top two only if
// logit_v / T + g_v > t.second, hence only if g_v > t.second - lmax (lmax >= every logit_v / T of the range), i.e. only if
// 1 - u_v < 1 - exp(-exp(-(t.second - lmax))).  u_v is an affine function of the random word, so this is one integer
// comparison per candidate against a bound that is refreshed whenever the thread's second-best score rises.  The bound
// carries a slack far above the float error of its evaluation, and candidates that pass are scored exactly as before, so
// the result is identical to scoring everything.
constexpr int SAMPLE_QUEUE = 160;       // per-warp queue of candidates that passed the bound: 32 waiting + up to 128 new

__device__ __forceinline__ void scan_blocks(Top2& t, const float* __restrict__ lg, int vocab, int b_begin, int b_end,
                                            float temperature, float lmax, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1, uint2* __restrict__ queue /*this warp's SAMPLE_QUEUE slots*/) {
    // The bound uses the largest second-best score of the warp: the final second-best is at least that, so a candidate
    // below it can change neither the winner nor the gap.  Candidates that pass are not scored where they are found (a
    // lane or two would drag the whole warp through the logarithms on most draws) but parked in a warp-private queue
    // and scored 32 at a time, one per lane.  Trip counts are warp-uniform (shuffles and ballots need every lane).
    int pass_above = -1;                        // a candidate is scored iff (int)(w >> 9) > pass_above  (-1: every candidate)
    float bound_for = -INFINITY;                // warp-wide score the bound was computed for
    bool stale = true;                          // a score was folded since the bound was computed (warp-uniform)
    const int lane = threadIdx.x & 31;
    const uint32_t lt_mask = (1u << lane) - 1u;
    int queued = 0;                             // warp-uniform
    auto drain = [&](int keep) {                // scores queued candidates, 32 at a time, until at most `keep` remain
        while (queued > keep) {
            const int take = min(32, queued);
            __syncwarp();
            if (lane < take) {
                const uint2 c = queue[queued - take + lane];
                top2_push_unordered(t, lg[c.x] / temperature + gumbel_from_word(c.y), (int)c.x);
            }
            queued -= take;
            stale = true;
            __syncwarp();
        }
    };
    for (int base = b_begin + (threadIdx.x - lane); base < b_end; base += blockDim.x) {
        if (stale) {                             // the second-best scores only move when candidates were scored
            stale = false;
            const float ws = warp_max(t.second);
            if (ws > bound_for) {
                bound_for = ws;
                const float T = ws - lmax - 1e-3f * (1.f + fabsf(ws) + fabsf(lmax));     // conservative
                // (1 - U0) * 2^23 with U0 = exp(-exp(-T)); expm1f keeps the relative accuracy when U0 is close to 1
                const float d = -expm1f(-expf(-T)) * 8388608.f;
                // scored iff 2^23 - (w >> 9) < d * 1.001 + 2, i.e. iff (w >> 9) > 2^23 - (that bound)
                pass_above = d >= 8388608.f ? -1 : 8388608 - (int)(uint32_t)(d * 1.001f + 2.f);
            }
        }
        const int b = base + lane;
        Philox4 w{0, 0, 0, 0};
        if (b < b_end) w = philox4x32_10((uint32_t)b, c1, c2, c3, k0, k1);
        // Almost every block holds no candidate above the bound: one comparison on the block's largest word and one vote
        // decide that for the whole warp; only blocks that may hold one go through the per-word test and the queue.
        const uint32_t top = max(max(w.x, w.y), max(w.z, w.w));
        if (!__any_sync(0xffffffffu, b < b_end && (int)(top >> 9) > pass_above)) continue;
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int v = b * 4 + i;
            const bool pass = b < b_end && v < vocab && (int)(ww[i] >> 9) > pass_above;
            const uint32_t m = __ballot_sync(0xffffffffu, pass);
            if (pass) queue[queued + __popc(m & lt_mask)] = make_uint2((uint32_t)v, ww[i]);
            queued += __popc(m);
        }
        drain(31);
    }
    drain(0);
}

// Largest logit / T over the blocks a thread block will scan (block-wide); `red` is 33 floats of shared memory.
__device__ __forceinline__ float range_max(const float* __restrict__ lg, int v0, int v1, float temperature, float* red) {
    float m = -INFINITY;
    // 16-byte loads, four in flight per thread: a row is hundreds of KB and one scalar load per thread at a time would
    // leave the pass bound by memory latency
    int v = v0;
    while (v < v1 && (reinterpret_cast<uintptr_t>(lg + v) & 15u) != 0) { if (threadIdx.x == 0) m = fmaxf(m, lg[v]); ++v; }
    const int n4 = (v1 - v) >> 2;
    const float4* p4 = reinterpret_cast<const float4*>(lg + v);
    int i = threadIdx.x;
    for (; i + 3 * (int)blockDim.x < n4; i += 4 * blockDim.x) {
        const float4 a = p4[i], b = p4[i + blockDim.x], c = p4[i + 2 * blockDim.x], d = p4[i + 3 * blockDim.x];
        m = fmaxf(m, fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w))));
        m = fmaxf(m, fmaxf(fmaxf(fmaxf(c.x, c.y), fmaxf(c.z, c.w)), fmaxf(fmaxf(d.x, d.y), fmaxf(d.z, d.w))));
    }
    for (; i < n4; i += blockDim.x) { const float4 a = p4[i]; m = fmaxf(m, fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w))); }
    for (int t = v + 4 * n4 + threadIdx.x; t < v1; t += blockDim.x) m = fmaxf(m, lg[t]);
    m = warp_max(m) / temperature;          // temperature > 0: the division is monotone
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) red[warp] = m;
    __syncthreads();
    if (warp == 0) {
        float x = lane < (int)(blockDim.x >> 5) ? red[lane] : -INFINITY;
        x = warp_max(x);
        if (lane == 0) red[32] = x;
    }
    __syncthreads();
    return red[32];
}

// One block per row.
__global__ void __launch_bounds__(256) sample_kernel(const StepDesc* __restrict__ sd, int vocab, const float* __restrict__ logits,
                                                     const int32_t* __restrict__ logits_row, float temperature,
                                                     uint32_t k0, uint32_t k1, const int32_t* __restrict__ row_prompt,
                                                     const int32_t* __restrict__ row_rollout, const int32_t* __restrict__ row_step,
                                                     int step_offset, int32_t* __restrict__ out_tokens,
                                                     const int64_t* __restrict__ out_index, int64_t out_index_offset,
                                                     float* __restrict__ out_gap, const int32_t* __restrict__ prompt_key,
                                                     const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x;
    const int64_t ro = r;                   // index into the row arrays
    if (sd != nullptr && r >= sd->n_rows) return;
    if (da != nullptr) {                    // decode step: token buffer, temperature and seed from the device-resident arguments
        out_tokens = da->tokens; temperature = da->temperature; k0 = da->k0; k1 = da->k1;
    }
    const float* lg = logits + (size_t)(logits_row ? logits_row[ro] : r) * vocab;
    const uint32_t c1 = (uint32_t)(row_step[ro] + step_offset), c2 = (uint32_t)row_rollout[ro],
                   c3 = (uint32_t)(prompt_key ? prompt_key[row_prompt[ro]] : row_prompt[ro]);    // key id of the prompt
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    const int n_blocks = (vocab + 3) >> 2;
    __shared__ float red[33];
    __shared__ uint2 queue[8][SAMPLE_QUEUE];
    const float lmax = range_max(lg, 0, vocab, temperature, red);
    scan_blocks(t, lg, vocab, 0, n_blocks, temperature, lmax, c1, c2, c3, k0, k1, queue[threadIdx.x >> 5]);
    t = top2_warp_reduce(t);
    __shared__ Top2 sh[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sh[warp] = t;
    __syncthreads();
    if (warp == 0) {
        Top2 u = lane < (int)(blockDim.x >> 5) ? sh[lane] : Top2{-INFINITY, -INFINITY, 0x7fffffff};
        u = top2_warp_reduce(u);
        if (lane == 0) {
            const int64_t at = out_index ? out_index[ro] + out_index_offset : (int64_t)r;
            if (at >= 0) out_tokens[at] = u.idx;
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
                                                             const int32_t* __restrict__ row_step, int step_offset, Top2Rec* __restrict__ scratch,
                                                             const int32_t* __restrict__ prompt_key, const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x, chunk = blockIdx.y;
    const int64_t ro = r;
    if (sd != nullptr && r >= sd->n_rows) return;
    if (da != nullptr) { temperature = da->temperature; k0 = da->k0; k1 = da->k1; }
    const float* lg = logits + (size_t)(logits_row ? logits_row[ro] : r) * vocab;
    const uint32_t c1 = (uint32_t)(row_step[ro] + step_offset), c2 = (uint32_t)row_rollout[ro],
                   c3 = (uint32_t)(prompt_key ? prompt_key[row_prompt[ro]] : row_prompt[ro]);    // key id of the prompt
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    const int n_blocks = (vocab + 3) >> 2;
    const int per_chunk = (n_blocks + n_chunks - 1) / n_chunks;
    const int b_end = min(n_blocks, (chunk + 1) * per_chunk);
    __shared__ float red[33];
    __shared__ uint2 queue[8][SAMPLE_QUEUE];
    const float lmax = range_max(lg, min(vocab, chunk * per_chunk * 4), min(vocab, b_end * 4), temperature, red);
    scan_blocks(t, lg, vocab, chunk * per_chunk, b_end, temperature, lmax, c1, c2, c3, k0, k1, queue[threadIdx.x >> 5]);
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
                                     int64_t out_index_offset, float* __restrict__ out_gap, const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t ro = r;
    if (r >= (sd != nullptr ? sd->n_rows : n_rows)) return;
    if (da != nullptr) out_tokens = da->tokens;
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    for (int c = 0; c < n_chunks; ++c) {
        const Top2Rec x = scratch[(size_t)r * n_chunks + c];
        t = top2_merge(t, Top2{x.best, x.second, x.idx});
    }
    const int64_t at = out_index ? out_index[ro] + out_index_offset : (int64_t)r;
    if (at >= 0) out_tokens[at] = t.idx;
    if (out_gap) out_gap[r] = t.best - t.second;
}

// log softmax(logits / T)[token]: the behaviour log-probability of an already drawn token.  One block per row;
// max and sum of exponentials are block reductions in a fixed shape, so the value does not depend on timing.
__global__ void __launch_bounds__(256) token_logprob_kernel(const StepDesc* __restrict__ sd, int vocab, const float* __restrict__ logits,
                                                            const int32_t* __restrict__ logits_row, float temperature,
                                                            const int32_t* __restrict__ tokens, const int64_t* __restrict__ tok_index,
                                                            int64_t tok_index_offset, float* __restrict__ out,
                                                            const int64_t* __restrict__ out_index, int64_t out_index_offset,
                                                            const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x;
    const int64_t ro = r;
    if (sd != nullptr && r >= sd->n_rows) return;
    if (da != nullptr) { tokens = da->tokens; out = da->logprobs; temperature = da->temperature; }
    const float* lg = logits + (size_t)(logits_row ? logits_row[ro] : r) * vocab;
    __shared__ float red[33];
    const float mx = range_max(lg, 0, vocab, temperature, red);          // max of logits / T
    const float inv_t = 1.f / temperature;
    float s = 0.f;
    {
        // 16-byte loads, four in flight per thread (one scalar load at a time leaves the pass bound by memory latency);
        // every thread adds its elements in a fixed order, so the sum does not depend on timing
        int v = 0;
        while (v < vocab && (reinterpret_cast<uintptr_t>(lg + v) & 15u) != 0) { if (threadIdx.x == 0) s += expf(lg[v] * inv_t - mx); ++v; }
        const int n4 = (vocab - v) >> 2;
        const float4* p4 = reinterpret_cast<const float4*>(lg + v);
        auto add4 = [&](const float4 a) {
            s += expf(a.x * inv_t - mx); s += expf(a.y * inv_t - mx); s += expf(a.z * inv_t - mx); s += expf(a.w * inv_t - mx);
        };
        int i = threadIdx.x;
        for (; i + 3 * (int)blockDim.x < n4; i += 4 * blockDim.x) {
            const float4 a = p4[i], b = p4[i + blockDim.x], c = p4[i + 2 * blockDim.x], d = p4[i + 3 * blockDim.x];
            add4(a); add4(b); add4(c); add4(d);
        }
        for (; i < n4; i += blockDim.x) add4(p4[i]);
        for (int t = v + 4 * n4 + threadIdx.x; t < vocab; t += blockDim.x) s += expf(lg[t] * inv_t - mx);
    }
    s = block_sum(s, red);
    if (threadIdx.x == 0) {
        const int64_t ti = tok_index ? tok_index[ro] + tok_index_offset : (int64_t)r;
        if (ti < 0) return;
        const int tok = tokens[ti];
        const float lp = (tok >= 0 && tok < vocab) ? lg[tok] * inv_t - mx - logf(s) : -INFINITY;
        out[out_index ? out_index[ro] + out_index_offset : (int64_t)r] = lp;
    }
}

constexpr int SAMPLE_MAX_CHUNKS = 32;
// Ranges per row so that about four blocks per SM are in flight; 1 means the one-pass kernel is the better choice.
inline int sample_chunks(int n_rows, int num_sms) {
    const int want = (4 * num_sms + n_rows - 1) / (n_rows > 0 ? n_rows : 1);
    return want < 2 ? 1 : (want > SAMPLE_MAX_CHUNKS ? SAMPLE_MAX_CHUNKS : want);
}

}  // namespace pc
