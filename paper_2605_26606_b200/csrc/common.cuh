// Shared device helpers: storage-type conversion, warp/block reductions, error flag codes.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pc {

// Codes stored in the caller's device error flag (first one wins is not guaranteed; any non-zero means failure).
enum DevError : int32_t {
    DEV_OK = 0,
    DEV_ERR_SLOT_RANGE = 1,     // a KV slot outside its arena
    DEV_ERR_TOKEN_RANGE = 2,    // a token id outside [0, vocab)
    DEV_ERR_WAIT_TIMEOUT = 3,   // a bounded wait on an mbarrier ran out
    DEV_ERR_GROUP_RANGE = 4,    // group / row bookkeeping inconsistent
    DEV_ERR_HALF_RANGE = 5,     // a GEMM operand or V value did not fit IEEE half (stored saturated)
};

// What one forward pass covers, kept in device memory so that a captured CUDA graph can be replayed for
// every decode step: kernels are launched with grids sized for an upper bound and read the live counts here.
struct StepDesc {
    int32_t n_rows;           // live rows (decode) or packed prompt tokens (prefill)
    int32_t n_groups;         // groups of contiguous rows sharing a prompt
    int32_t max_group_rows;
    int32_t reserved;
    int64_t row_off;          // offset of this step's rows in the caller's flat row arrays
    int64_t group_off;        // offset of this step's group_row_start entries
};

// The caller's arrays of a decode call, kept in device memory (part of the workspace) and rewritten, in stream order, by
// every pc_decode_step / pc_decode_run: captured decode steps read the pointers here, so a CUDA graph does not depend on
// where a stage's schedule happens to live.
struct DecodeArgsDev {
    const StepDesc* steps;            // pc_decode_run: the schedule (the device counter indexes it)
    const int32_t* row_prompt;
    const int32_t* row_rollout;
    const int32_t* row_step;
    const int64_t* row_kv_start;
    int32_t* tokens;
    const int64_t* row_tok_index;
    const int32_t* group_row_start;
    const int32_t* prompt_len;
    const int64_t* prompt_kv_start;
    float* logprobs;                  // or nullptr
    const int32_t* prompt_key;        // or nullptr
    float temperature;
    uint32_t k0, k1;                  // sampling seed
    int32_t n_prompts;                // entries of prompt_len / prompt_kv_start / prompt_key (0: unknown, not checked)
    int64_t n_tokens;                 // length of the token buffer (0: unknown, not checked)
};

// Per-row sampling keys and output positions of a decode step, compacted into the workspace by prep_decode_rows.
struct RowKeys {
    int32_t* key_prompt;     // [M] prompt id of the sampling key
    int32_t* rollout;        // [M]
    int32_t* step_key;       // [M] step counter of the key: suffix tokens cached + 1
    int64_t* out_index;      // [M] where the drawn token goes in the token buffer
    int32_t* group_start;    // [groups + 1] first row of every group of the step
    int32_t* sample_bound;   // [M] largest second-best score any vocabulary tile of the row has reported so far (ordered-int form)
};

// float <-> int with the same order (atomicMax on scores of either sign); -infinity maps to the smallest value in use
__device__ __forceinline__ int32_t score_to_ordered(float f) {
    const int32_t i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float ordered_to_score(int32_t i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// Programmatic dependent launch (griddepcontrol): a kernel launched with the programmatic-serialization attribute may
// start while the kernel before it in the stream is still running; it must not touch anything that kernel writes until
// grid_dep_wait() has returned (which is when that kernel has finished and its writes are visible).  Launched without
// the attribute, both instructions do nothing.  The rule followed here: before the wait a kernel only sets up its own
// shared / tensor memory and reads weights (never written during a pass); every CTA executes the wait on every path.
__device__ __forceinline__ void grid_dep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void set_error(int32_t* flag, int32_t code) {
    if (flag != nullptr) atomicCAS(flag, 0, code);
}

// Values headed for IEEE half storage: anything beyond the largest finite half is stored saturated (NaN as the largest
// finite value) and reported.  half_clamp is branch-free; callers OR half_bad over a batch of values and report once.
constexpr float HALF_MAX_F = 65504.f;
__device__ __forceinline__ float half_clamp(float x) { return fminf(fmaxf(x, -HALF_MAX_F), HALF_MAX_F); }
__device__ __forceinline__ int half_bad(float x) { return !(fabsf(x) <= HALF_MAX_F); }
__device__ __forceinline__ float half_guard(float x, int32_t* err) {
    if (half_bad(x)) set_error(err, DEV_ERR_HALF_RANGE);
    return half_clamp(x);
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Sum over a block of up to 1024 threads; every thread gets the result.  `red` is 33 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (warp == 0) {
        float t = lane < nwarp ? red[lane] : 0.f;
        t = warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}

// Loads `N` consecutive elements of storage type T (N * sizeof(T) in {4, 8, 16} bytes, aligned) as floats.
template <typename T, int N> struct VecLoad;
template <> struct VecLoad<float, 4> {
    static __device__ __forceinline__ void load(const float* p, float* out) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct VecLoad<float, 2> {
    static __device__ __forceinline__ void load(const float* p, float* out) {
        const float2 v = *reinterpret_cast<const float2*>(p);
        out[0] = v.x; out[1] = v.y;
    }
};
template <> struct VecLoad<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
        out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
    }
};
template <> struct VecLoad<__nv_bfloat16, 2> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
        out[0] = __uint_as_float(v << 16); out[1] = __uint_as_float(v & 0xffff0000u);
    }
};

}  // namespace pc
