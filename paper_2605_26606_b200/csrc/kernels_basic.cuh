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

// Both step-descriptor kernels also zero the grid-barrier words of the persistent decode kernel (bar, n_bar words;
// launched with STEP_DESC_THREADS threads).
constexpr int STEP_DESC_THREADS = 128;
__global__ void set_step_desc(StepDesc* sd, int n_rows, int n_groups, int max_group_rows, int32_t* max_slen, int32_t* bar, int n_bar) {
    for (int i = threadIdx.x; i < n_bar; i += blockDim.x) bar[i] = 0;
    if (threadIdx.x != 0) return;
    *max_slen = 0;
    sd->n_rows = n_rows; sd->n_groups = n_groups; sd->max_group_rows = max_group_rows; sd->reserved = 0;
    sd->row_off = 0; sd->group_off = 0;
}
// First node of a captured decode step: takes the next descriptor of the caller's schedule.
__global__ void load_step_desc(const DecodeArgsDev* __restrict__ da, int32_t* counter, StepDesc* sd, int32_t* max_slen, int32_t* bar, int n_bar) {
    for (int i = threadIdx.x; i < n_bar; i += blockDim.x) bar[i] = 0;
    if (threadIdx.x != 0) return;
    *max_slen = 0;
    const int i = *counter;
    *sd = da->steps[i];
    *counter = i + 1;
}

// Decode: row r of prompt p with `step` suffix tokens cached attends prompt slots [start_p, start_p + Lp)
// and suffix slots [kv_start_r, kv_start_r + step + 1); its own K/V goes to suffix slot kv_start_r + step.
// Also compacts the row's sampling key, the position of its next token and the step's group boundaries into the
// workspace.  A row whose indices do not fit their arrays is switched off (no KV access, token 0) and flagged.
__global__ void prep_decode_rows(const StepDesc* __restrict__ sd, const DecodeArgsDev* __restrict__ da, int64_t prompt_slots,
                                 int64_t suffix_slots, int vocab, RowGeom g, RowKeys keys, int32_t* err) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    const int n_rows = sd->n_rows;
    if (r <= sd->n_groups) keys.group_start[r] = da->group_row_start[sd->group_off + r];
    if (r >= n_rows) return;
    const int64_t ro = sd->row_off + r;
    int p = da->row_prompt[ro];
    const int step = da->row_step[ro];
    const int64_t ti = da->row_tok_index[ro];
    bool ok = true;
    if (p < 0 || (da->n_prompts > 0 && p >= da->n_prompts) || ti < 0 || (da->n_tokens > 0 && ti + 1 >= da->n_tokens)) {
        set_error(err, DEV_ERR_GROUP_RANGE);
        ok = false;
        p = 0;
    }
    const int Lp = ok ? da->prompt_len[p] : 0;
    const int64_t ps = ok ? da->prompt_kv_start[p] : 0;
    const int64_t ss = da->row_kv_start[ro];
    int tok = ok ? da->tokens[ti] : 0;
    if (tok < 0 || tok >= vocab) { set_error(err, DEV_ERR_TOKEN_RANGE); tok = 0; }
    if (ok && (ps < 0 || Lp < 0 || ps + Lp > prompt_slots || ss < 0 || step < 0 || ss + step + 1 > suffix_slots)) {
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
    keys.key_prompt[r] = ok && da->prompt_key ? da->prompt_key[p] : p;
    keys.rollout[r] = da->row_rollout[ro];
    keys.step_key[r] = step + 1;
    keys.out_index[r] = ok ? ti + 1 : -1;            // -1: nothing is stored for this row
    keys.sample_bound[r] = score_to_ordered(-INFINITY);      // no tile of the row has reported a second-best score yet
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

// K-slice sums left by a split GEMM: value(row, col) = sum over s < n of p[s * stride + row * ld + col], added in
// the order s = 0, 1, ... so that the result does not depend on which CTA finished first.
struct Partials {
    const float* p;
    int n;              // 0: nothing pending; at most PARTIALS_MAX
    size_t stride;
    int ld;
};
constexpr int PARTIALS_MAX = 8;

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

// The row-wise operations below are written for ONE WARP per row (or per (row, head)), so that the stand-alone kernels
// and the phases of the persistent decode kernel (decode_chain.cuh) run the very same arithmetic in the same order.

// half_out: 0 = storage type T, 1 = IEEE half (operand of a half-precision GEMM); err = the device error flag (range guard).
template <typename T>
__device__ __forceinline__ void store_norm_out(T* __restrict__ a_row, T* __restrict__ a_lo_row, int i4, float4 y, int half_out,
                                               int32_t* err = nullptr) {
    if (sizeof(T) == 2 && half_out) {
        if (half_bad(y.x) | half_bad(y.y) | half_bad(y.z) | half_bad(y.w)) set_error(err, DEV_ERR_HALF_RANGE);
        const __half2 lo = __floats2half2_rn(half_clamp(y.x), half_clamp(y.y)), hi = __floats2half2_rn(half_clamp(y.z), half_clamp(y.w));
        *reinterpret_cast<uint2*>(a_row + 4 * i4) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    } else {
        store4<T>(a_row + 4 * i4, y);
    }
    if (a_lo_row != nullptr) store4<T>(a_lo_row + 4 * i4, bf16_remainder(y));
}

// Residual update followed by the norm:
//   h_row[:] += pending K-slice sums (pend_row = their row offset, in slice order);  a_row[:] = RMSNorm(h_row; gain).
// d is a multiple of 8.  The row is cut into NORM_SEGS interleaved segments (the 128-element block b belongs to segment
// b mod NORM_SEGS); a segment's sum of squares is the warp sum of its lanes' partial sums (blocks in increasing order) and
// the row's sum adds the segments in order.  That fixes the arithmetic whether one warp walks all segments
// (norm_row_warp) or NORM_SEGS warps of a CTA take one segment each (the persistent decode kernel at small batches).
constexpr int NORM_SEGS = 6;
constexpr int NORM_REG4 = 12;            // blocks of a row one warp keeps in registers (d <= 1536)

// One 128-element block of the row: loads value, gain and every pending slice (straight-line, all requested before the
// first add waits), returns the updated value.
__device__ __forceinline__ float4 norm_block_load(const float4* __restrict__ x, int i, const Partials& pend, size_t pend_row) {
    float4 v = x[i];
    float4 q[PARTIALS_MAX];
#pragma unroll
    for (int s = 0; s < PARTIALS_MAX; ++s)
        q[s] = s < pend.n ? *reinterpret_cast<const float4*>(pend.p + (size_t)s * pend.stride + pend_row + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int s = 0; s < PARTIALS_MAX; ++s)          // the adds stay in slice order
        if (s < pend.n) { v.x += q[s].x; v.y += q[s].y; v.z += q[s].z; v.w += q[s].w; }
    return v;
}
// Explicitly rounded operations: the compiler must not contract them differently in the two forms of the row norm.
__device__ __forceinline__ float sq4(float4 v) {
    return __fmaf_rn(v.w, v.w, __fmaf_rn(v.z, v.z, __fmaf_rn(v.y, v.y, __fmul_rn(v.x, v.x))));
}

template <typename T>
__device__ __forceinline__ void norm_row_warp(int lane, int d, float* __restrict__ h_row, Partials pend, size_t pend_row,
                                              const float* __restrict__ gain, float eps, T* __restrict__ a_row,
                                              T* __restrict__ a_lo_row, int half_out, int32_t* err = nullptr) {
    const int n4 = d >> 2;
    float4* x = reinterpret_cast<float4*>(h_row);
    float seg[NORM_SEGS];
#pragma unroll
    for (int g = 0; g < NORM_SEGS; ++g) seg[g] = 0.f;
    if (n4 <= NORM_REG4 * 32) {
        float4 v[NORM_REG4], gg[NORM_REG4];
#pragma unroll
        for (int k = 0; k < NORM_REG4; ++k) {
            const int i = lane + 32 * k;
            if (i < n4) {
                gg[k] = *reinterpret_cast<const float4*>(gain + 4 * i);
                v[k] = norm_block_load(x, i, pend, pend_row);
                seg[k % NORM_SEGS] = __fadd_rn(seg[k % NORM_SEGS], sq4(v[k]));
            }
        }
        if (pend.n > 0) {
#pragma unroll
            for (int k = 0; k < NORM_REG4; ++k)
                if (lane + 32 * k < n4) x[lane + 32 * k] = v[k];
        }
        float ss = 0.f;
#pragma unroll
        for (int g = 0; g < NORM_SEGS; ++g) ss = __fadd_rn(ss, warp_sum(seg[g]));
        const float rstd = rsqrtf(__fadd_rn(__fdiv_rn(ss, (float)d), eps));
#pragma unroll
        for (int k = 0; k < NORM_REG4; ++k) {
            const int i = lane + 32 * k;
            if (i < n4)
                store_norm_out<T>(a_row, a_lo_row, i,
                                  make_float4(v[k].x * rstd * gg[k].x, v[k].y * rstd * gg[k].y, v[k].z * rstd * gg[k].z, v[k].w * rstd * gg[k].w),
                                  half_out, err);
        }
        return;
    }
    const int nk = (n4 + 31) >> 5;
#pragma unroll
    for (int g = 0; g < NORM_SEGS; ++g) {
        for (int k = g; k < nk; k += NORM_SEGS) {
            const int i = lane + 32 * k;
            if (i < n4) {
                const float4 v = norm_block_load(x, i, pend, pend_row);
                if (pend.n > 0) x[i] = v;
                seg[g] = __fadd_rn(seg[g], sq4(v));
            }
        }
    }
    float ss = 0.f;
#pragma unroll
    for (int g = 0; g < NORM_SEGS; ++g) ss = __fadd_rn(ss, warp_sum(seg[g]));
    const float rstd = rsqrtf(__fadd_rn(__fdiv_rn(ss, (float)d), eps));
    for (int i = lane; i < n4; i += 32) {
        const float4 v = x[i], gg = *reinterpret_cast<const float4*>(gain + 4 * i);     // this lane's own writes
        store_norm_out<T>(a_row, a_lo_row, i, make_float4(v.x * rstd * gg.x, v.y * rstd * gg.y, v.z * rstd * gg.z, v.w * rstd * gg.w), half_out, err);
    }
}

// The same row handled by NORM_SEGS warps of one CTA, warp w taking segment w: every load of the row is in flight at once,
// which is what a latency-bound batch wants.  The segment sums are exchanged through shared memory: red[NORM_SEGS] floats
// and one counter, both used once (zero before); the wait on the counter is bounded and returns false when it ran out.
// KK = blocks per warp kept in registers; rows need (d / 128) <= NORM_SEGS * KK.
template <typename T, int KK>
__device__ __forceinline__ bool norm_row_cta_kk(int w, int lane, int d, float* __restrict__ h_row, Partials pend, size_t pend_row,
                                                const float* __restrict__ gain, float eps, T* __restrict__ a_row, T* __restrict__ a_lo_row,
                                                int half_out, volatile float* red, int* counter, int32_t* err) {
    const int n4 = d >> 2;
    float4* x = reinterpret_cast<float4*>(h_row);
    float4 v[KK], gg[KK];
    float part = 0.f;
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
        const int i = lane + 32 * (w + NORM_SEGS * kk);
        if (i < n4) {
            gg[kk] = *reinterpret_cast<const float4*>(gain + 4 * i);
            v[kk] = norm_block_load(x, i, pend, pend_row);
            part = __fadd_rn(part, sq4(v[kk]));
        }
    }
    if (pend.n > 0) {
#pragma unroll
        for (int kk = 0; kk < KK; ++kk) {
            const int i = lane + 32 * (w + NORM_SEGS * kk);
            if (i < n4) x[i] = v[kk];
        }
    }
    part = warp_sum(part);
    if (lane == 0) {
        red[w] = part;
        __threadfence_block();
        atomicAdd(counter, 1);
    }
    bool ok = false;
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (*reinterpret_cast<volatile int*>(counter) >= NORM_SEGS) { ok = true; break; }
        __nanosleep(20);
    }
    __threadfence_block();
    if (!ok) return false;
    float ss = 0.f;
#pragma unroll
    for (int g = 0; g < NORM_SEGS; ++g) ss = __fadd_rn(ss, red[g]);
    const float rstd = rsqrtf(__fadd_rn(__fdiv_rn(ss, (float)d), eps));
#pragma unroll
    for (int kk = 0; kk < KK; ++kk) {
        const int i = lane + 32 * (w + NORM_SEGS * kk);
        if (i < n4)
            store_norm_out<T>(a_row, a_lo_row, i,
                              make_float4(v[kk].x * rstd * gg[kk].x, v[kk].y * rstd * gg[kk].y, v[kk].z * rstd * gg[kk].z, v[kk].w * rstd * gg[kk].w),
                              half_out, err);
    }
    return true;
}
__device__ __forceinline__ bool norm_row_fits_cta(int d) { return ((d >> 2) + 31) / 32 <= NORM_SEGS * 8; }
template <typename T>
__device__ __forceinline__ bool norm_row_cta(int w, int lane, int d, float* __restrict__ h_row, Partials pend, size_t pend_row,
                                             const float* __restrict__ gain, float eps, T* __restrict__ a_row, T* __restrict__ a_lo_row,
                                             int half_out, volatile float* red, int* counter, int32_t* err = nullptr) {
    const int nk = ((d >> 2) + 31) / 32;
    if (nk <= NORM_SEGS * 2) return norm_row_cta_kk<T, 2>(w, lane, d, h_row, pend, pend_row, gain, eps, a_row, a_lo_row, half_out, red, counter, err);
    if (nk <= NORM_SEGS * 4) return norm_row_cta_kk<T, 4>(w, lane, d, h_row, pend, pend_row, gain, eps, a_row, a_lo_row, half_out, red, counter, err);
    return norm_row_cta_kk<T, 8>(w, lane, d, h_row, pend, pend_row, gain, eps, a_row, a_lo_row, half_out, red, counter, err);
}

// h_row[:] = E[token, :] as float (the residual stream), one warp per row; d is a multiple of 8.
template <typename T>
__device__ __forceinline__ void embed_row_warp(int lane, int d, const T* __restrict__ e_row, float* __restrict__ h_row) {
    for (int i = lane; i < (d >> 2); i += 32) {
        float v[4];
        VecLoad<T, 4>::load(e_row + 4 * i, v);
        reinterpret_cast<float4*>(h_row)[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

constexpr int ROW_WARPS = 8;         // items per block of the stand-alone per-(row, head) kernels
constexpr int NORM_THREADS = NORM_SEGS * 32;

// h[r, :] = E[token[r], :] (float residual stream); a[r, :] = RMSNorm(h[r, :]; gain) in storage type T.  One block per row.
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) embed_rmsnorm_kernel(const StepDesc* __restrict__ sd, int d, const int32_t* token,
                                                                     const T* __restrict__ embed, const float* __restrict__ gain, float eps,
                                                                     float* __restrict__ h, T* __restrict__ a, T* __restrict__ a_lo, int half_out,
                                                                     int32_t* err) {
    __shared__ float red[8];
    __shared__ int counter;
    const int r = blockIdx.x, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dep_launch_dependents();          // the projection that follows may set itself up and request its first weight tiles
    if (r >= sd->n_rows) return;
    if (threadIdx.x == 0) counter = 0;
    const T* e_row = embed + (size_t)token[r] * d;
    float* h_row = h + (size_t)r * d;
    for (int i = threadIdx.x; i < (d >> 2); i += NORM_THREADS) {
        float v[4];
        VecLoad<T, 4>::load(e_row + 4 * i, v);
        reinterpret_cast<float4*>(h_row)[i] = make_float4(v[0], v[1], v[2], v[3]);
    }
    __syncthreads();
    if (norm_row_fits_cta(d))
        norm_row_cta<T>(w, lane, d, h_row, Partials{nullptr, 0, 0, 0}, 0, gain, eps, a + (size_t)r * d, a_lo ? a_lo + (size_t)r * d : nullptr,
                        half_out, red, &counter, err);
    else if (w == 0)
        norm_row_warp<T>(lane, d, h_row, Partials{nullptr, 0, 0, 0}, 0, gain, eps, a + (size_t)r * d, a_lo ? a_lo + (size_t)r * d : nullptr,
                         half_out, err);
}

// Optional residual update followed by the norm:  h[row, :] += pending partial sums of row;  a[r, :] = RMSNorm(h[row, :]; gain)
// with row = src ? src[r] : r.  The partial sums are indexed by row, like h.  n_rows bounds r when there is no step descriptor.
// One block per row.
template <typename T>
__global__ void __launch_bounds__(NORM_THREADS) rmsnorm_kernel(const StepDesc* __restrict__ sd, int n_rows, int d, float* __restrict__ h,
                                                               const int32_t* __restrict__ src, Partials pend, const float* __restrict__ gain,
                                                               float eps, T* __restrict__ a, T* __restrict__ a_lo, int half_out, int32_t* err) {
    __shared__ float red[8];
    __shared__ int counter;
    const int r = blockIdx.x, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dep_launch_dependents();          // the projection that follows may set itself up and request its first weight tiles
    if (r >= (sd != nullptr ? sd->n_rows : n_rows)) return;
    if (threadIdx.x == 0) counter = 0;
    __syncthreads();
    const int row = src ? src[r] : r;
    if (norm_row_fits_cta(d))
        norm_row_cta<T>(w, lane, d, h + (size_t)row * d, pend, (size_t)row * pend.ld, gain, eps, a + (size_t)r * d,
                        a_lo ? a_lo + (size_t)r * d : nullptr, half_out, red, &counter, err);
    else if (w == 0)
        norm_row_warp<T>(lane, d, h + (size_t)row * d, pend, (size_t)row * pend.ld, gain, eps, a + (size_t)r * d,
                         a_lo ? a_lo + (size_t)r * d : nullptr, half_out, err);
}

struct KvArena {
    void* base;
    int64_t n_slots;
};

// Everything the q/k/v post-processing needs besides the item index.
template <typename T>
struct QkvPostArgs {
    int Hq, Hkv, hd, layer;
    Partials qkv;                 // the projection as K-slice partial sums (one slice when the GEMM was not split)
    const float* bias;            // or nullptr
    const float* q_gain;          // per-head RMSNorm gains, or nullptr
    const float* k_gain;
    float eps;
    const float2* rope;           // [rows, hd/2] (cos, sin)
    RowGeom g;
    KvArena prompt_arena, suffix_arena;
    T* q_out;                     // [rows, Hq * hd]
    int32_t* err;                 // device error flag (range guard of the half V cache)
};

// One warp per (row, head of the fused q|k|v projection); lane i handles the rotary pairs (i, i + hd/2) and, for
// head_dim 128, (i + 32, i + 32 + hd/2).  The bias is added here.
// q heads: optional RMSNorm over head_dim, RoPE, stored to q_out as T.
// k heads: optional RMSNorm, RoPE, stored to the row's KV slot.  v heads: stored to the row's KV slot.
// NB items are processed together so that their loads are all in flight before the first one is used (callers pass
// n_items = NB: the code is then straight-line).
template <typename T, int NB>
__device__ __forceinline__ void qkv_post_items_warp(int lane, const QkvPostArgs<T>& A, const int* rows, const int* heads, int n_items) {
    const int half = A.hd >> 1, npair = half > 32 ? 2 : 1;
    float x1[NB][2], x2[NB][2];
    float2 cs[NB][2];
    int64_t slot[NB];
    int to_suffix[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (b >= n_items) continue;
        const int r = rows[b], head = heads[b];
        slot[b] = A.g.wslot[r];
        to_suffix[b] = A.g.warena[r];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (j >= npair) continue;
            const int i = lane + 32 * j;
            const size_t col = (size_t)head * A.hd + i;
            cs[b][j] = A.rope[(size_t)r * half + i];
            float p1[PARTIALS_MAX], p2[PARTIALS_MAX];          // requested together, added in slice order
#pragma unroll
            for (int s = 0; s < PARTIALS_MAX; ++s) {
                const float* src = A.qkv.p + (size_t)s * A.qkv.stride + (size_t)r * A.qkv.ld + col;
                p1[s] = s < A.qkv.n ? src[0] : 0.f;
                p2[s] = s < A.qkv.n ? src[half] : 0.f;
            }
            float a1 = A.bias ? A.bias[col] : 0.f, a2 = A.bias ? A.bias[col + half] : 0.f;
#pragma unroll
            for (int s = 0; s < PARTIALS_MAX; ++s)
                if (s < A.qkv.n) { a1 += p1[s]; a2 += p2[s]; }
            x1[b][j] = a1; x2[b][j] = a2;
        }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
        if (b >= n_items) continue;
        const int r = rows[b], head = heads[b];
        const bool is_q = head < A.Hq, is_k = !is_q && head < A.Hq + A.Hkv;
        if (is_q || is_k) {
            const float* gain = is_q ? A.q_gain : A.k_gain;
            if (gain != nullptr) {
                float ss = 0.f;
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    if (j < npair) ss += x1[b][j] * x1[b][j] + x2[b][j] * x2[b][j];
                ss = warp_sum(ss);
                const float rstd = rsqrtf(ss / (float)A.hd + A.eps);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                    if (j < npair) {
                        x1[b][j] = x1[b][j] * rstd * gain[lane + 32 * j];
                        x2[b][j] = x2[b][j] * rstd * gain[lane + 32 * j + half];
                    }
            }
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (j < npair) {
                    const float y1 = x1[b][j] * cs[b][j].x - x2[b][j] * cs[b][j].y;
                    const float y2 = x2[b][j] * cs[b][j].x + x1[b][j] * cs[b][j].y;
                    x1[b][j] = y1; x2[b][j] = y2;
                }
        }
        // 16-bit models keep q, K and V as IEEE half (same two bytes, three more mantissa bits than bfloat16): the rounding of
        // V, and for models with QK-norm that of q and K (their scores are of order one), is the largest single error source
        // of the logits.  Values outside half's range are stored saturated and reported.
        if (is_q) {
            T* dst = A.q_out + (size_t)r * A.Hq * A.hd + (size_t)head * A.hd;
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (j < npair) {
                    if (sizeof(T) == 2) {
                        reinterpret_cast<__half*>(dst)[lane + 32 * j] = __float2half_rn(half_guard(x1[b][j], A.err));
                        reinterpret_cast<__half*>(dst)[lane + 32 * j + half] = __float2half_rn(half_guard(x2[b][j], A.err));
                    } else {
                        dst[lane + 32 * j] = from_f32<T>(x1[b][j]);
                        dst[lane + 32 * j + half] = from_f32<T>(x2[b][j]);
                    }
                }
            continue;
        }
        if (slot[b] < 0) continue;
        const KvArena ar = to_suffix[b] ? A.suffix_arena : A.prompt_arena;
        const int kvh = is_k ? head - A.Hq : head - A.Hq - A.Hkv;
        const int64_t plane = ((int64_t)A.layer * 2 + (is_k ? 0 : 1)) * A.Hkv + kvh;
        T* dst = reinterpret_cast<T*>(ar.base) + (plane * ar.n_slots + slot[b]) * A.hd;
        if (sizeof(T) == 2) {
            __half* dv = reinterpret_cast<__half*>(dst);
#pragma unroll
            for (int j = 0; j < 2; ++j)
                if (j < npair) {
                    dv[lane + 32 * j] = __float2half_rn(half_guard(x1[b][j], A.err));
                    dv[lane + 32 * j + half] = __float2half_rn(half_guard(x2[b][j], A.err));
                }
            continue;
        }
#pragma unroll
        for (int j = 0; j < 2; ++j)
            if (j < npair) { dst[lane + 32 * j] = from_f32<T>(x1[b][j]); dst[lane + 32 * j + half] = from_f32<T>(x2[b][j]); }
    }
}

// Stand-alone form: one warp per (row, head), ROW_WARPS items per block, item = row * n_heads + head.
template <typename T>
__global__ void __launch_bounds__(ROW_WARPS * 32) qkv_post_kernel(const StepDesc* __restrict__ sd, QkvPostArgs<T> A) {
    const int n_heads = A.Hq + 2 * A.Hkv;
    const int item = blockIdx.x * ROW_WARPS + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    grid_dep_launch_dependents();          // the shared-prefix attention kernel may request its first prompt K/V tiles
    if (item >= sd->n_rows * n_heads) return;
    const int row = item / n_heads, head = item - row * n_heads;
    qkv_post_items_warp<T, 1>(lane, A, &row, &head, 1);
}

__global__ void reward_last_token_kernel(int n, const int32_t* tokens, const int64_t* last_index,
                                         const int32_t* threshold, float* reward) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int tok = tokens[last_index[i]];
    reward[i] = tok >= 0 && tok < threshold[i] ? 1.f : 0.f;        // a cell that was never generated (-1) earns nothing
}

}  // namespace pc
