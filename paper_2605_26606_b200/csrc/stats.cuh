// Per-group reward statistics (Eq. 3), pilot filter / eviction / commit allocation (Algorithm 1) and
// group-relative advantages (Section 3.1).  Groups are tiny (G <= a few hundred): one warp per group,
// double accumulation so that the results are independent of the reduction shape to well below 1e-6.
#pragma once

#include "common.cuh"

namespace pc {

constexpr int STATUS_COMMIT = 0, STATUS_BUFFERED = 1, STATUS_DEFER_HARD = 2, STATUS_SKIP_EASY = 3, STATUS_LOW_VARIANCE = 4;

__global__ void group_stats_kernel(int n_groups, const float* __restrict__ rewards, const int32_t* __restrict__ start,
                                   const int32_t* __restrict__ count, int32_t* __restrict__ n_out,
                                   int32_t* __restrict__ m_out, float* __restrict__ mean_out, float* __restrict__ var_out) {
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (g >= n_groups) return;
    const int n = max(count[g], 0);
    const float* r = rewards + start[g];
    double s = 0.0;
    int m = 0;
    for (int i = lane; i < n; i += 32) { const float v = r[i]; s += (double)v; m += (v == 1.f); }
    s = warp_sum(s);
    m = warp_sum(m);
    const double mu = n > 0 ? s / (double)n : 0.0;
    double q = 0.0;
    for (int i = lane; i < n; i += 32) { const double d = (double)r[i] - mu; q += d * d; }
    q = warp_sum(q);
    if (lane == 0) {
        n_out[g] = n;
        m_out[g] = m;
        mean_out[g] = (float)mu;
        var_out[g] = n > 0 ? (float)(q / (double)n) : 0.f;
    }
}

// Single block.  Prompts are taken in batch order; the first b_t that pass the filter commit.
// pilot_var != nullptr selects the filter for general scalar rewards: keep iff the pilot variance (Eq. 3, as float) is at
// least var_min; the success-rate thresholds and the eviction rule are then not used (evict = 0).
__global__ void __launch_bounds__(1024) allocate_kernel(int n_prompts, const int32_t* __restrict__ success,
                                                        const int32_t* __restrict__ pilot_n, const float* __restrict__ pilot_var,
                                                        double var_min, double p_lower, double p_upper,
                                                        double p_solve, int n_commit, int b_t, int32_t* __restrict__ status,
                                                        int32_t* __restrict__ extra, int32_t* __restrict__ evict,
                                                        int32_t* __restrict__ n_selected, long long* __restrict__ total_rollouts) {
    __shared__ int warp_tot[32];
    __shared__ int chunk_base;
    __shared__ long long pilot_total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { chunk_base = 0; pilot_total = 0; }
    __syncthreads();
    for (int c0 = 0; c0 < n_prompts; c0 += blockDim.x) {
        const int p = c0 + threadIdx.x;
        int keep = 0, st = STATUS_DEFER_HARD, ev = 0, np = 0;
        if (p < n_prompts) {
            np = max(pilot_n[p], 0);
            if (pilot_var != nullptr) {
                keep = np > 0 && (double)pilot_var[p] >= var_min;
                st = keep ? STATUS_COMMIT : STATUS_LOW_VARIANCE;
            } else {
                const double p_hat = np > 0 ? (double)success[p] / (double)np : 0.0;   // IEEE division, same as the host's
                keep = (p_lower <= p_hat) && (p_hat <= p_upper);
                ev = p_hat >= p_solve;
                st = keep ? STATUS_COMMIT : (p_hat < p_lower ? STATUS_DEFER_HARD : STATUS_SKIP_EASY);
            }
        }
        // exclusive prefix count of `keep` in batch order
        const unsigned ballot = __ballot_sync(0xffffffffu, keep);
        const int before_in_warp = __popc(ballot & ((1u << lane) - 1u));
        if (lane == 0) warp_tot[warp] = __popc(ballot);
        const int np_sum = warp_sum(np);
        if (lane == 0 && np_sum) atomicAdd((unsigned long long*)&pilot_total, (unsigned long long)np_sum);
        __syncthreads();
        int before = chunk_base + before_in_warp;
        for (int w = 0; w < warp; ++w) before += warp_tot[w];
        if (p < n_prompts) {
            if (keep && before >= b_t) st = STATUS_BUFFERED;
            status[p] = st;
            extra[p] = st == STATUS_COMMIT ? n_commit : 0;
            if (evict != nullptr) evict[p] = ev;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int tot = 0;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += warp_tot[w];
            chunk_base += tot;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int sel = min(chunk_base, max(b_t, 0));
        *n_selected = sel;
        *total_rollouts = pilot_total + (long long)sel * (long long)n_commit;
    }
}

__global__ void grpo_advantage_kernel(int n_groups, const float* __restrict__ rewards, const int32_t* __restrict__ start,
                                      const int32_t* __restrict__ count, const int32_t* __restrict__ status,
                                      float* __restrict__ adv) {
    const int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (g >= n_groups) return;
    const int n = max(count[g], 0);
    const float* r = rewards + start[g];
    float* a = adv + start[g];
    float lo = INFINITY, hi = -INFINITY;
    double s = 0.0;
    for (int i = lane; i < n; i += 32) { const float v = r[i]; s += (double)v; lo = fminf(lo, v); hi = fmaxf(hi, v); }
    s = warp_sum(s);
    lo = warp_min(lo);
    hi = warp_max(hi);
    const bool live = (status == nullptr || status[g] == STATUS_COMMIT) && n > 0 && lo != hi;
    if (!live) {                       // zero-variance group (or not selected): zero advantage
        for (int i = lane; i < n; i += 32) a[i] = 0.f;
        return;
    }
    const double mu = s / (double)n;
    double q = 0.0;
    for (int i = lane; i < n; i += 32) { const double d = (double)r[i] - mu; q += d * d; }
    q = warp_sum(q);
    const double sigma = sqrt(q / (double)n);
    for (int i = lane; i < n; i += 32) a[i] = (float)(((double)r[i] - mu) / sigma);
}

}  // namespace pc
