// LM head with the Gumbel-max draw in its epilogue: the logits of a decode step never reach memory.
//
// The GEMM is the tensor-core kernel of gemm_tc.cuh with EpiSample as its epilogue.  For every (row, 256-column tile of
// the vocabulary) the epilogue thread that owns the row reads its accumulators from TMEM twice: once for the largest
// logit of the tile, once to score the candidates -- score_v = logit_v / T + g_v with the same Philox word, the same
// float arithmetic and the same exact integer prefilter as the stand-alone sampler (sampler.cuh), so the largest and the
// second-largest score of the tile and the arg-max are bit for bit what that sampler finds on stored logits.  The tile
// leaves one (best, second, arg-best) record; sample_tiles_reduce_kernel folds a row's records in tile order.  Maxima are
// exact, so the drawn token and the top-two gap equal the unfused path's.
#pragma once

#include "gemm_tc.cuh"
#include "sampler.cuh"

namespace pc {

struct EpiSample {
    static constexpr bool kWholeTile = true;
    Top2Rec* rec;                  // [vocabulary tiles][m_stride]
    int m_stride;
    const int32_t* key_prompt;     // per row: prompt id of the sampling key, rollout, step counter (RowKeys)
    const int32_t* rollout;
    const int32_t* step_key;
    const DecodeArgsDev* da;       // temperature and seed
    __device__ __forceinline__ void set_rows(int) {}

    template <int BN>
    __device__ __forceinline__ void tile(uint32_t taddr, int row, bool live, int n0, int N) const {
        float lmax = -INFINITY;
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            if (n0 + c >= N) break;                 // warp-uniform
            float v[32];
            tc::tmem_ld32(taddr + c, v);
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (n0 + c + i < N) lmax = fmaxf(lmax, v[i]);
        }
        const float temperature = da->temperature;
        const uint32_t k0 = da->k0, k1 = da->k1;
        uint32_t c1 = 0, c2 = 0, c3 = 0;
        if (live) { c1 = (uint32_t)step_key[row]; c2 = (uint32_t)rollout[row]; c3 = (uint32_t)key_prompt[row]; }
        lmax = lmax / temperature;
        Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
        uint32_t pass_below = 0xffffffffu;          // a candidate is scored iff (2^23 - (w >> 9)) < pass_below
        float bound_for = -INFINITY;                // second-best score the bound was computed for
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
            if (n0 + c >= N) break;
            float v[32];
            tc::tmem_ld32(taddr + c, v);            // every lane takes part in the load; rows past the live count do no more
            if (!live) continue;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const int col = n0 + c + 4 * b;
                if (col >= N) break;
                const Philox4 w = philox4x32_10((uint32_t)(col >> 2), c1, c2, c3, k0, k1);
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (col + i >= N) break;
                    if (t.second > bound_for) {
                        // same conservative bound as scan_blocks: a candidate that fails it cannot enter this row's top two
                        bound_for = t.second;
                        const float T = t.second - lmax - 1e-3f * (1.f + fabsf(t.second) + fabsf(lmax));
                        const float d = -expm1f(-expf(-T)) * 8388608.f;
                        pass_below = d >= 8388608.f ? 0xffffffffu : (uint32_t)(d * 1.001f + 2.f);
                    }
                    if ((8388608u - (ww[i] >> 9)) < pass_below)
                        top2_push(t, v[4 * b + i] / temperature + gumbel_from_word(ww[i]), col + i);
                }
            }
        }
        if (live) rec[(size_t)(n0 / BN) * m_stride + row] = Top2Rec{t.best, t.second, t.idx, 0};
    }
};

// One warp per row: folds the row's records of all vocabulary tiles (in tile order within a lane, then across lanes with
// the order-independent merge) and stores the token.
__global__ void __launch_bounds__(256) sample_tiles_reduce_kernel(const StepDesc* __restrict__ sd, int n_tiles, const Top2Rec* __restrict__ rec,
                                                                  int m_stride, const int64_t* __restrict__ out_index,
                                                                  const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= sd->n_rows) return;
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    for (int i = lane; i < n_tiles; i += 32) {
        const Top2Rec x = rec[(size_t)i * m_stride + r];
        t = top2_merge(t, Top2{x.best, x.second, x.idx});
    }
    t = top2_warp_reduce(t);
    if (lane == 0) {
        const int64_t at = out_index[r];
        if (at >= 0) da->tokens[at] = t.idx;
    }
}

}  // namespace pc
