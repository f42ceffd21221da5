// LM head with the Gumbel-max draw in its epilogue: the logits of a decode step never reach memory.
//
// The GEMM is the tensor-core kernel of gemm_tc.cuh with EpiSample as its epilogue.  For every (row, tile of the
// vocabulary) the epilogue thread that owns the row reads its accumulators from TMEM twice: once for the largest logit of
// the tile, once to score the candidates -- score_v = logit_v / T + g_v with the same Philox word, the same float
// arithmetic and the same exact integer prefilter as the stand-alone sampler (sampler.cuh).  The tile leaves one
// (best, second, arg-best) record; sample_tiles_reduce_kernel folds a row's records.
//
// The prefilter needs a lower bound of the row's final second-best score.  A tile on its own knows only its own
// candidates, which would let a dozen of them through per tile; so the tiles of a row share the best bound found so
// far through one word per row in global memory (an ordered-int atomic max, read when a tile starts).  Every value
// ever stored there is the second-best score of some subset of the row's candidates, hence never above the final
// second-best: a candidate rejected against it can be neither the winner nor the runner-up.  Which candidates a tile
// scores therefore depends on timing, the folded (best, second, arg-best) of the row does not: the drawn token and the
// top-two gap are bit for bit the unfused path's.
#pragma once

#include "gemm_tc.cuh"
#include "sampler.cuh"

namespace pc {

struct EpiSample {
    static constexpr bool kWholeTile = true;
    static constexpr int kEpiWarps = 8;        // the Philox arithmetic of a tile is split over two warps per accumulator quarter
    Top2Rec* rec;                  // [2 * vocabulary tiles][m_stride]: one record per half tile
    int m_stride;
    const int32_t* key_prompt;     // per row: prompt id of the sampling key, rollout, step counter (RowKeys)
    const int32_t* rollout;
    const int32_t* step_key;
    int32_t* row_bound;            // per row: running lower bound of the final second-best score (ordered-int form)
    const DecodeArgsDev* da;       // temperature and seed
    __device__ __forceinline__ void set_rows(int) {}

    // scored iff (2^23 - (w >> 9)) < the returned word: the candidate's noise could lift it above `second`
    static __device__ __forceinline__ uint32_t pass_word(float second, float lmax) {
        const float T = second - lmax - 1e-3f * (1.f + fabsf(second) + fabsf(lmax));      // conservative, as in scan_blocks
        const float d = -expm1f(-expf(-T)) * 8388608.f;
        return d >= 8388608.f ? 0xffffffffu : (uint32_t)(d * 1.001f + 2.f);
    }

    template <int BN>
    __device__ __forceinline__ void tile_part(uint32_t taddr, int row, bool live, int n0_tile, int N, int part) const {
        static_assert(BN % 64 == 0, "half tiles must be whole 32-column chunks");
        const int n0 = n0_tile + part * (BN / 2);
        taddr += part * (BN / 2);
        const int n_cols = min(BN / 2, N - n0);            // warp-uniform; may be <= 0 in the last tile; a multiple of 4 is not required
        if (n_cols <= 0 || !__any_sync(0xffffffffu, live)) {
            // nothing to score (columns past the vocabulary, or none of the warp's 32 rows is live): an empty record
            if (live) rec[(size_t)(2 * (n0_tile / BN) + part) * m_stride + row] = Top2Rec{-INFINITY, -INFINITY, 0x7fffffff, 0};
            return;
        }
        float lmax = -INFINITY;
#pragma unroll 1
        for (int c = 0; c < n_cols; c += 32) {
            float v[32];
            tc::tmem_ld32(taddr + c, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) lmax = fmaxf(lmax, c + i < n_cols ? v[i] : -INFINITY);
        }
        const float temperature = da->temperature;
        const uint32_t k0 = da->k0, k1 = da->k1;
        uint32_t c1 = 0, c2 = 0, c3 = 0;
        float shared_bound = -INFINITY;
        if (live) {
            c1 = (uint32_t)step_key[row]; c2 = (uint32_t)rollout[row]; c3 = (uint32_t)key_prompt[row];
            shared_bound = ordered_to_score(__ldcg(row_bound + row));
        }
        lmax = lmax / temperature;
        Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
        float bound_for = shared_bound;                    // score the pass word was computed for
        uint32_t pass_below = live ? pass_word(shared_bound, lmax) : 0u;      // rows past the live count score nothing
        if (shared_bound == -INFINITY && live) pass_below = 0xffffffffu;
#pragma unroll 1
        for (int c = 0; c < n_cols; c += 32) {
            float v[32];
            tc::tmem_ld32(taddr + c, v);                   // every lane takes part in the load
            // all eight Philox blocks of the chunk first, without a branch between them (eight independent dependency
            // chains in flight), then one mask of the candidates that pass the integer bound: it is empty almost always
            uint32_t word[32];
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const Philox4 w = philox4x32_10((uint32_t)((n0 + c) >> 2) + b, c1, c2, c3, k0, k1);
                word[4 * b] = w.x; word[4 * b + 1] = w.y; word[4 * b + 2] = w.z; word[4 * b + 3] = w.w;
            }
            uint32_t pass = 0;
#pragma unroll
            for (int i = 0; i < 32; ++i) pass |= (uint32_t)((8388608u - (word[i] >> 9)) < pass_below) << i;
            if (c + 32 > n_cols) pass &= (1u << (n_cols - c)) - 1u;          // columns past the vocabulary
            if (pass == 0) continue;
            // candidates in increasing id order; the bound tightens as they are pushed (a candidate that passed the older,
            // looser bound is scored all the same: scoring more than necessary never changes the top two)
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                if (pass & (1u << i)) {
                    if ((8388608u - (word[i] >> 9)) < pass_below) {
                        top2_push(t, v[i] / temperature + gumbel_from_word(word[i]), n0 + c + i);
                        if (t.second > bound_for) {
                            bound_for = t.second;
                            pass_below = pass_word(t.second, lmax);
                        }
                    }
                }
            }
        }
        if (live) {
            rec[(size_t)(2 * (n0_tile / BN) + part) * m_stride + row] = Top2Rec{t.best, t.second, t.idx, 0};
            if (t.second > shared_bound) atomicMax(row_bound + row, score_to_ordered(t.second));
        }
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
