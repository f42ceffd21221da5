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

// Eight Philox4x32-10 blocks with consecutive first counter words, advanced round by round: the eight dependency chains
// are independent, and written this way they are in flight together (two epilogue warps per scheduler have no other
// way to hide the multiplier's latency).  word[4 b + i] is word i of block c0 + b.
__device__ __forceinline__ void philox4x32_10_x8(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                                 uint32_t (&word)[32]) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t x0[8], x1[8], x2[8], x3[8];
#pragma unroll
    for (int b = 0; b < 8; ++b) { x0[b] = c0 + b; x1[b] = c1; x2[b] = c2; x3[b] = c3; }
#pragma unroll
    for (int r = 0; r < 10; ++r) {
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            const uint64_t p0 = (uint64_t)M0 * x0[b], p1 = (uint64_t)M1 * x2[b];
            const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
            const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
            x0[b] = hi1 ^ x1[b] ^ k0; x1[b] = lo1; x2[b] = hi0 ^ x3[b] ^ k1; x3[b] = lo0;
        }
        k0 += W0; k1 += W1;
    }
#pragma unroll
    for (int b = 0; b < 8; ++b) { word[4 * b] = x0[b]; word[4 * b + 1] = x1[b]; word[4 * b + 2] = x2[b]; word[4 * b + 3] = x3[b]; }
}

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
            philox4x32_10_x8((uint32_t)((n0 + c) >> 2), c1, c2, c3, k0, k1, word);
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

// One block of 128 threads per row: folds the row's records of all half tiles (the merge is order-independent: equal scores
// keep the lowest id) and stores the token.  A thread's loads are issued four at a time.
constexpr int TILES_REDUCE_THREADS = 128;
__global__ void __launch_bounds__(TILES_REDUCE_THREADS) sample_tiles_reduce_kernel(const StepDesc* __restrict__ sd, int n_tiles, const Top2Rec* __restrict__ rec,
                                                                                   int m_stride, const int64_t* __restrict__ out_index,
                                                                                   const DecodeArgsDev* __restrict__ da) {
    const int r = blockIdx.x;
    if (r >= sd->n_rows) return;
    const int4* p = reinterpret_cast<const int4*>(rec) + r;
    Top2 t{-INFINITY, -INFINITY, 0x7fffffff};
    int i = threadIdx.x;
    for (; i + 3 * TILES_REDUCE_THREADS < n_tiles; i += 4 * TILES_REDUCE_THREADS) {
        int4 x[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) x[j] = __ldcg(p + (size_t)(i + j * TILES_REDUCE_THREADS) * m_stride);
#pragma unroll
        for (int j = 0; j < 4; ++j) t = top2_merge(t, Top2{__int_as_float(x[j].x), __int_as_float(x[j].y), x[j].z});
    }
    for (; i < n_tiles; i += TILES_REDUCE_THREADS) {
        const int4 x = __ldcg(p + (size_t)i * m_stride);
        t = top2_merge(t, Top2{__int_as_float(x.x), __int_as_float(x.y), x.z});
    }
    t = top2_warp_reduce(t);
    __shared__ Top2 sh[TILES_REDUCE_THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sh[warp] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 1; w < TILES_REDUCE_THREADS / 32; ++w) t = top2_merge(t, sh[w]);
        const int64_t at = out_index[r];
        if (at >= 0) da->tokens[at] = t.idx;
    }
}

}  // namespace pc
