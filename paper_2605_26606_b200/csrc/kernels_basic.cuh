// Row bookkeeping, embedding gather, RMSNorm, rotary tables, q/k/v post-processing, reward rule.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace pc {

// Per-row attention geometry shared by prefill and decode.
struct RowGeom {
    int32_t* pos;        // [M] absolute position of the row's token
    int64_t* wslot;      // [M] slot the row's K/V is written to
    int32_t* warena;     // [M] 0: write into the prompt arena, 1: into the suffix arena
    int64_t* p_start;    // [M] first prompt-arena slot attended
    int32_t* p_len;      // [M] number of prompt-arena slots attended
    int64_t* s_start;    // [M] first suffix-arena slot attended
    int32_t* s_len;      // [M] number of suffix-arena slots attended
    int32_t* token;      // [M] input token id
    int32_t* max_slen;   // [1] largest s_len of the step (decode only)
};

__global__ void set_step_desc(StepDesc* sd, int n_rows, int n_groups, int max_group_rows, int32_t* max_slen) {
    *max_slen = 0;
    sd->n_rows = n_rows; sd->n_groups = n_groups; sd->max_group_rows = max_group_rows; sd->reserved = 0;
    sd->row_off = 0; sd->group_off = 0;
}
// First node of a captured decode step: takes the next descriptor of the caller's schedule.
__global__ void load_step_desc(const StepDesc* __restrict__ steps, int32_t* counter, StepDesc* sd, int32_t* max_slen) {
    *max_slen = 0;
    const int i = *counter;
    *sd = steps[i];
    *counter = i + 1;
}

// Decode: row r of prompt p with `step` suffix tokens cached attends prompt slots [start_p, start_p + Lp)
// and suffix slots [kv_start_r, kv_start_r + step + 1); its own K/V goes to suffix slot kv_start_r + step.
__global__ void prep_decode_rows(const StepDesc* __restrict__ sd, const int32_t* row_prompt, const int32_t* row_step,
                                 const int64_t* row_kv_start, const int32_t* tokens, const int64_t* row_tok_index,
                                 const int32_t* prompt_len, const int64_t* prompt_kv_start, int64_t prompt_slots,
                                 int64_t suffix_slots, int vocab, RowGeom g, int32_t* err) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= sd->n_rows) return;
    const int64_t ro = sd->row_off + r;
    const int p = row_prompt[ro];
    const int step = row_step[ro];
    const int Lp = prompt_len[p];
    const int64_t ps = prompt_kv_start[p];
    const int64_t ss = row_kv_start[ro];
    int tok = tokens[row_tok_index[ro]];
    bool ok = true;
    if (tok < 0 || tok >= vocab) { set_error(err, DEV_ERR_TOKEN_RANGE); tok = 0; }
    if (ps < 0 || Lp < 0 || ps + Lp > prompt_slots || ss < 0 || step < 0 || ss + step + 1 > suffix_slots) {
        set_error(err, DEV_ERR_SLOT_RANGE);
        ok = false;
    }
    g.pos[r] = Lp + step;
    g.token[r] = tok;
    g.warena[r] = 1;
    g.wslot[r] = ok ? ss + step : -1;
    g.p_start[r] = ps;
    g.p_len[r] = ok ? Lp : 0;
    g.s_start[r] = ss;
    g.s_len[r] = ok ? step + 1 : 0;
    if (ok) atomicMax(g.max_slen, step + 1);
}

// Prefill: packed token t of prompt p at position i attends prompt slots [start_p, start_p + i + 1).
__global__ void prep_prefill_rows(int n_prompts, const int32_t* prompt_tokens, const int32_t* prompt_offsets,
                                  const int64_t* prompt_kv_start, int64_t prompt_slots, int vocab, RowGeom g,
                                  int32_t* last_row, int32_t* err) {
    const int p = blockIdx.x;
    const int b = prompt_offsets[p], e = prompt_offsets[p + 1];
    const int64_t ps = prompt_kv_start[p];
    const bool ok = ps >= 0 && ps + (e - b) <= prompt_slots;
    if (!ok && threadIdx.x == 0) set_error(err, DEV_ERR_SLOT_RANGE);
    if (threadIdx.x == 0) last_row[p] = e - 1;
    for (int t = b + threadIdx.x; t < e; t += blockDim.x) {
        int tok = prompt_tokens[t];
        if (tok < 0 || tok >= vocab) { set_error(err, DEV_ERR_TOKEN_RANGE); tok = 0; }
        const int i = t - b;
        g.pos[t] = i;
        g.token[t] = tok;
        g.warena[t] = 0;
        g.wslot[t] = ok ? ps + i : -1;
        g.p_start[t] = ps;
        g.p_len[t] = ok ? i + 1 : 0;
        g.s_start[t] = 0;
        g.s_len[t] = 0;
    }
}

// cos/sin of pos * theta^(-2i/hd), evaluated in double so that long positions keep float accuracy.
__global__ void rope_table_kernel(const StepDesc* __restrict__ sd, int half, double theta, const int32_t* pos, float2* table) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= sd->n_rows * half) return;
    const int r = idx / half, i = idx - r * half;
    const double inv_freq = pow(theta, -(double)i / (double)half);
    double s, c;
    sincos((double)pos[r] * inv_freq, &s, &c);
    table[idx] = make_float2((float)c, (float)s);
}

// h[r, :] = E[token[r], :] (float residual stream); a[r, :] = RMSNorm(h[r, :]; gain) in storage type T.
template <typename T>
__global__ void embed_rmsnorm_kernel(const StepDesc* __restrict__ sd, int d, const int32_t* token, const T* __restrict__ embed,
                                     const float* __restrict__ gain, float eps, float* __restrict__ h, T* __restrict__ a,
                                     T* __restrict__ a_lo, int half_out) {
    __shared__ float red[33];
    const int r = blockIdx.x;
    if (r >= sd->n_rows) return;
    const T* e = embed + (size_t)token[r] * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = to_f32<T>(e[i]);
        h[(size_t)r * d + i] = v;
        ss += v * v;
    }
    ss = block_sum(ss, red);
    const float rstd = rsqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float y = h[(size_t)r * d + i] * rstd * gain[i];
        if (sizeof(T) == 2 && half_out) reinterpret_cast<__half*>(a)[(size_t)r * d + i] = __float2half_rn(y);
        else a[(size_t)r * d + i] = from_f32<T>(y);
        if (a_lo != nullptr) a_lo[(size_t)r * d + i] = from_f32<T>(y - to_f32<T>(from_f32<T>(y)));
    }
}

// K-slice sums left by a split GEMM: value(row, col) = sum over s < n of p[s * stride + row * ld + col], added in
// the order s = 0, 1, ... so that the result does not depend on which CTA finished first.
struct Partials {
    const float* p;
    int n;              // 0: nothing pending; at most PARTIALS_MAX
    size_t stride;
    int ld;
};
constexpr int PARTIALS_MAX = 8;

// Optional residual update followed by the norm:  h[row, :] += pending partial sums of row r;  a[r, :] = RMSNorm(h[row, :]; gain)
// with row = src ? src[r] : r.  The partial sums are indexed by row, like h.
template <typename T> __device__ __forceinline__ void store4(T* p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float4 v) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

// Rounding remainder of a float4 after its conversion to bf16 (what a second, "low" bf16 operand carries).
__device__ __forceinline__ float4 bf16_remainder(float4 v) {
    return make_float4(v.x - __bfloat162float(__float2bfloat16_rn(v.x)), v.y - __bfloat162float(__float2bfloat16_rn(v.y)),
                       v.z - __bfloat162float(__float2bfloat16_rn(v.z)), v.w - __bfloat162float(__float2bfloat16_rn(v.w)));
}

// One block of 256 threads per row; d is a multiple of 8 and at most 8192, so a thread keeps its <= 8 float4 of the
// row in registers between the sum of squares and the scaling (one pass over global memory).
template <typename T>
__global__ void __launch_bounds__(256) rmsnorm_kernel(const StepDesc* __restrict__ sd, int d, float* __restrict__ h,
                                                      const int32_t* __restrict__ src, Partials pend, const float* __restrict__ gain,
                                                      float eps, T* __restrict__ a, T* __restrict__ a_lo, int half_out) {
    __shared__ float red[33];
    const int r = blockIdx.x;
    // The grid covers the row bound of the step; rows past the live count are dropped only after this row's data has
    // been requested (buffers hold the bound, so the reads are in range): the step descriptor, the row and its
    // pending slices then arrive together instead of one memory latency after the other.
    const int n_live = sd != nullptr ? sd->n_rows : gridDim.x;
    const int row = src ? src[r] : r;
    float4* x = reinterpret_cast<float4*>(h + (size_t)row * d);
    const int n4 = d >> 2;
    float4 v[8];
    float4 p[2][PARTIALS_MAX];
    float4 gg2[2];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = threadIdx.x + k * 256;
        if (i < n4) {
            v[k] = x[i];
            if (k < 2) {
                gg2[k] = *reinterpret_cast<const float4*>(gain + 4 * i);
#pragma unroll
                for (int s = 0; s < PARTIALS_MAX; ++s)
                    p[k][s] = s < pend.n ? *reinterpret_cast<const float4*>(pend.p + (size_t)s * pend.stride + (size_t)row * pend.ld + 4 * i)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
    if (r >= n_live) return;
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = threadIdx.x + k * 256;
        if (i < n4) {
            if (pend.n > 0) {
                // the adds stay in slice order
                if (k < 2) {
#pragma unroll
                    for (int s = 0; s < PARTIALS_MAX; ++s)
                        if (s < pend.n) { v[k].x += p[k][s].x; v[k].y += p[k][s].y; v[k].z += p[k][s].z; v[k].w += p[k][s].w; }
                } else {
                    for (int s = 0; s < pend.n; ++s) {
                        const float4 q = *reinterpret_cast<const float4*>(pend.p + (size_t)s * pend.stride + (size_t)row * pend.ld + 4 * i);
                        v[k].x += q.x; v[k].y += q.y; v[k].z += q.z; v[k].w += q.w;
                    }
                }
                x[i] = v[k];
            }
            ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        }
    }
    ss = block_sum(ss, red);
    const float rstd = rsqrtf(ss / (float)d + eps);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = threadIdx.x + k * 256;
        if (i < n4) {
            const float4 gg = k < 2 ? gg2[k] : *reinterpret_cast<const float4*>(gain + 4 * i);
            const float4 y = make_float4(v[k].x * rstd * gg.x, v[k].y * rstd * gg.y, v[k].z * rstd * gg.z, v[k].w * rstd * gg.w);
            if (sizeof(T) == 2 && half_out) {          // IEEE half instead of bfloat16 (operand of a half-precision GEMM)
                const __half2 lo = __floats2half2_rn(y.x, y.y), hi = __floats2half2_rn(y.z, y.w);
                *reinterpret_cast<uint2*>(a + (size_t)r * d + 4 * i) =
                    make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
            } else {
                store4<T>(a + (size_t)r * d + 4 * i, y);
            }
            if (a_lo != nullptr) store4<T>(a_lo + (size_t)r * d + 4 * i, bf16_remainder(y));
        }
    }
}

struct KvArena {
    void* base;
    int64_t n_slots;
};

// One block per (row, head of the fused q|k|v projection); thread i handles the rotary pair (i, i + hd/2).
// The projection arrives as K-slice partial sums (one slice when the GEMM was not split); the bias is added here.
// q heads: optional RMSNorm over head_dim, RoPE, stored to q_out [M, Hq*hd] as T.
// k heads: optional RMSNorm, RoPE, stored to the row's KV slot.  v heads: stored to the row's KV slot.
template <typename T>
__global__ void qkv_post_kernel(const StepDesc* __restrict__ sd, int Hq, int Hkv, int hd, int layer, Partials qkv,
                                const float* __restrict__ bias,
                                const float* __restrict__ q_gain, const float* __restrict__ k_gain, float eps,
                                const float2* __restrict__ rope, RowGeom g, KvArena prompt_arena, KvArena suffix_arena,
                                T* __restrict__ q_out) {
    __shared__ float red[33];
    const int r = blockIdx.x, head = blockIdx.y, i = threadIdx.x, half = hd >> 1;
    // rows past the live count are dropped after the loads have been requested (buffers hold the step's row bound)
    const int n_live = sd->n_rows;
    const float2 cs = rope[(size_t)r * half + i];
    const int64_t slot = g.wslot[r];
    const int to_suffix = g.warena[r];
    const size_t col = (size_t)head * hd + i;
    float x1 = bias ? bias[col] : 0.f, x2 = bias ? bias[col + half] : 0.f;
    {
        float p1[PARTIALS_MAX], p2[PARTIALS_MAX];          // requested together, added in slice order
#pragma unroll
        for (int s = 0; s < PARTIALS_MAX; ++s) {
            const float* src = qkv.p + (size_t)s * qkv.stride + (size_t)r * qkv.ld + col;
            p1[s] = s < qkv.n ? src[0] : 0.f;
            p2[s] = s < qkv.n ? src[half] : 0.f;
        }
#pragma unroll
        for (int s = 0; s < PARTIALS_MAX; ++s)
            if (s < qkv.n) { x1 += p1[s]; x2 += p2[s]; }
    }
    if (r >= n_live) return;
    const bool is_q = head < Hq, is_k = !is_q && head < Hq + Hkv;
    if (is_q || is_k) {
        const float* gain = is_q ? q_gain : k_gain;
        if (gain != nullptr) {
            const float ss = block_sum(x1 * x1 + x2 * x2, red);
            const float rstd = rsqrtf(ss / (float)hd + eps);
            x1 = x1 * rstd * gain[i];
            x2 = x2 * rstd * gain[i + half];
        }
        const float y1 = x1 * cs.x - x2 * cs.y;
        const float y2 = x2 * cs.x + x1 * cs.y;
        x1 = y1; x2 = y2;
    }
    if (is_q) {
        T* dst = q_out + (size_t)r * Hq * hd + (size_t)head * hd;
        dst[i] = from_f32<T>(x1);
        dst[i + half] = from_f32<T>(x2);
        return;
    }
    if (slot < 0) return;
    const KvArena ar = to_suffix ? suffix_arena : prompt_arena;
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    const int64_t plane = ((int64_t)layer * 2 + (is_k ? 0 : 1)) * Hkv + kvh;
    T* dst = reinterpret_cast<T*>(ar.base) + (plane * ar.n_slots + slot) * hd;
    if (!is_k && sizeof(T) == 2) {
        // 16-bit models keep V as IEEE half (same two bytes, three more mantissa bits than bfloat16): V is a linear map
        // of a unit-RMS vector, far inside half's range, and its rounding is the largest single error source of the logits
        __half* dv = reinterpret_cast<__half*>(dst);
        dv[i] = __float2half_rn(x1);
        dv[i + half] = __float2half_rn(x2);
        return;
    }
    dst[i] = from_f32<T>(x1);
    dst[i + half] = from_f32<T>(x2);
}

__global__ void reward_last_token_kernel(int n, const int32_t* tokens, const int64_t* last_index,
                                         const int32_t* threshold, float* reward) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) reward[i] = tokens[last_index[i]] < threshold[i] ? 1.f : 0.f;
}

}  // namespace pc
