// Persistent decode kernel: the GEMMs and row-wise operations between two attention calls of a decode step run as
// PHASES of one cooperative kernel (one CTA per SM) separated by grid-wide barriers, instead of one launch each.
//
//   segment -1 :  embedding + RMSNorm  |  QKV GEMM of layer 0  |  bias / QK-norm / RoPE / KV append
//   segment  l :  [merge of the attention records]  |  output projection  |  residual + RMSNorm  |  gate/up GEMM + SwiGLU  |
//                 down projection  |  residual + RMSNorm (gains of layer l+1, or the final norm)  |
//                 QKV GEMM of layer l+1  |  its post-processing          (last layer: LM head instead of the last two)
//
// Warp roles.  Warp 0 (one thread) is the TMA producer of every GEMM phase of the launch, warp 1 (one thread) issues the
// tcgen05 MMAs, warps 4..7 drain the TMEM accumulators (epilogues) and, with warps 2..3, do the row-wise phases.  The
// producer runs ahead of the barriers: the weight tile of a k-block is requested as soon as a shared-memory slot is
// free, also while the previous phase is still running anywhere on the GPU; only the activation tile of the first
// k-block waits for the barrier.  So the weight stream does not stop at phase boundaries.
//
// Grid barrier b is one int32 in global memory, zeroed by the step's first kernel and used once: a CTA adds 1 when all its
// worker warps have finished the phase (their writes fenced), waiters poll until it reaches gridDim.x.  Activations written
// by other CTAs with ordinary stores are read here by TMA, so the producer issues a proxy fence between its acquire of the
// barrier and the copy.  Every wait (mbarrier or grid barrier) is bounded; a wait that runs out raises
// DEV_ERR_WAIT_TIMEOUT, every role leaves its loops and the CTA frees its TMEM before it returns.  There is no
// CTA-wide barrier between roles inside the phase loop, so a role that gave up cannot leave another one stuck.
//
// The arithmetic is that of the stand-alone kernels (same device functions, same GEMM epilogues, same K-slice order),
// so both forms give identical bits for the same tile plan.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include "attention_mma.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "kernels_basic.cuh"

namespace pc {
namespace chain {

using tc::BK;
using tc::BM;
using tc::mbar_arrive;
using tc::mbar_arrive_expect_tx;
using tc::mbar_init;
using tc::mbar_wait;
using tc::smem_u32;
using tc::tma_load_2d;

constexpr int THREADS = 256;
constexpr int WORKER_WARP0 = 2, N_WORKER_WARPS = 6;
constexpr int A_BYTES = BM * BK * 2;
constexpr int RING_BYTES = 192 * 1024;           // operand ring: slots of (activation tile 16 KB + widest weight tile of the launch)
constexpr int MAX_SLOTS = 8;
constexpr int ACC_COLS = 256;                    // TMEM columns per accumulator (two accumulators)
constexpr uint32_t TMEM_COLS = 512;
constexpr int MAX_PHASES = 10;
constexpr int BAR_WORDS_PER_SEG = 16;
constexpr int SMEM_BYTES = RING_BYTES + 1024 /*align*/ + 512 /*barriers, flags*/;
constexpr uint32_t GRID_WAIT_LIMIT = 1u << 22;

enum Phase : int { PH_END = 0, PH_EMBED, PH_MERGE, PH_O, PH_NORM_MLP, PH_GU, PH_DOWN, PH_NORM_NEXT, PH_QKV, PH_POST, PH_LM };
enum GemmKindId : int { GK_QKV = 0, GK_O = 1, GK_GU = 2, GK_DOWN = 3, GK_LM = 4 };

__host__ __device__ constexpr int bn_index(int bn) { return bn == 64 ? 0 : (bn == 128 ? 1 : 2); }

// Per-layer constants in device memory (part of the workspace; written once by pc_set_workspace).
struct alignas(128) LayerTab {
    CUtensorMap wqkv[3], wo[3], wgu[3], wdown[3];       // boxes of 64 / 128 / 256 weight rows
    const float* attn_norm;
    const float* mlp_norm;
    const float* bqkv;
    const float* q_norm;
    const float* k_norm;
};
struct alignas(128) GlobalTab {
    CUtensorMap a, attn, act;                           // activation buffers, boxes of 128 rows
    CUtensorMap lm[3];
    const float* final_norm;
};

// TMA descriptors of one launch, passed in the kernel parameters (descriptor fetches then hit the constant cache).
enum MapId : int { MAP_A = 0, MAP_ATTN, MAP_ACT, MAP_WO, MAP_WGU, MAP_WDOWN, MAP_WNEXT /* QKV of the next layer, or the LM head */, N_MAPS };

struct ChainParams {
    CUtensorMap maps[N_MAPS];
    const StepDesc* sd;
    int M;                       // row bound the tiles and the partial-sum layout are sized for
    int seg;                     // -1: embedding .. QKV of layer 0;  l >= 0: output projection of layer l .. QKV of layer l + 1
    int with_merge;              // segment l starts with the merge of the attention records
    int n_layers, d_model, n_qkv, q_dim, d_ff, vocab, Hq, Hkv, hd;
    float eps;
    int bn[5], splits[5];        // tile width and K-slices per GEMM kind
    int slot_bytes, slots;       // operand ring of this launch: 16 KB + 128 B x the widest tile, RING_BYTES / slot_bytes slots
    const LayerTab* layers;
    const GlobalTab* glob;
    const void* embed;
    float* h;
    __nv_bfloat16* a;
    float* qkv;
    float* res_part;
    __nv_bfloat16* q;
    __nv_bfloat16* attn;
    __nv_bfloat16* act;
    float* logits;
    const float2* rope;
    RowGeom g;
    KvArena prompt_arena, suffix_arena;
    am::PrefixPartial part;
    int32_t* bar;                // BAR_WORDS_PER_SEG words per segment, zero when the step starts
    int32_t* err;
    long long* trace;            // optional: SM clock stamps of the first TRACE_CTAS CTAs, [segment][phase][cta][TRACE_EVENTS]
};
constexpr int TRACE_CTAS = 4, TRACE_EVENTS = 16;
enum TraceEvent : int { TR_W_BEGIN = 0, TR_W_WAITED, TR_W_DONE, TR_P_BEGIN, TR_P_BARRIER, TR_P_DONE, TR_M_FIRST_FULL, TR_M_DONE,
                        TR_E_FIRST_FULL, TR_E_DONE, TR_KERNEL_BEGIN, TR_KERNEL_END };
__device__ __forceinline__ void stamp(const ChainParams& p, int j, int ev) {
    if (p.trace != nullptr && blockIdx.x < TRACE_CTAS)
        p.trace[((size_t)((p.seg + 1) * MAX_PHASES + j) * TRACE_CTAS + blockIdx.x) * TRACE_EVENTS + ev] = clock64();
}

__device__ __forceinline__ bool is_gemm(int ph) { return ph == PH_O || ph == PH_GU || ph == PH_DOWN || ph == PH_QKV || ph == PH_LM; }

// Phase j of segment seg (PH_END after the last one).
__device__ __forceinline__ int phase_at(const ChainParams& p, int j) {
    if (p.seg < 0) return j == 0 ? PH_EMBED : (j == 1 ? PH_QKV : (j == 2 ? PH_POST : PH_END));
    const bool last = p.seg == p.n_layers - 1;
    if (!p.with_merge) ++j;
    switch (j) {
        case 0: return PH_MERGE;
        case 1: return PH_O;
        case 2: return PH_NORM_MLP;
        case 3: return PH_GU;
        case 4: return PH_DOWN;
        case 5: return PH_NORM_NEXT;
        case 6: return last ? PH_LM : PH_QKV;
        case 7: return last ? PH_END : PH_POST;
        default: return PH_END;
    }
}

struct GemmDesc {
    int map_a, map_w;            // MapId
    int N, K, BN, splits;
};
__device__ __forceinline__ GemmDesc gemm_desc(const ChainParams& p, int ph) {
    GemmDesc g;
    switch (ph) {
        case PH_O:
            g.BN = p.bn[GK_O]; g.splits = p.splits[GK_O]; g.N = p.d_model; g.K = p.q_dim;
            g.map_a = MAP_ATTN; g.map_w = MAP_WO;
            break;
        case PH_GU:
            g.BN = p.bn[GK_GU]; g.splits = 1; g.N = 2 * p.d_ff; g.K = p.d_model;
            g.map_a = MAP_A; g.map_w = MAP_WGU;
            break;
        case PH_DOWN:
            g.BN = p.bn[GK_DOWN]; g.splits = p.splits[GK_DOWN]; g.N = p.d_model; g.K = p.d_ff;
            g.map_a = MAP_ACT; g.map_w = MAP_WDOWN;
            break;
        case PH_QKV:
            g.BN = p.bn[GK_QKV]; g.splits = p.splits[GK_QKV]; g.N = p.n_qkv; g.K = p.d_model;
            g.map_a = MAP_A; g.map_w = MAP_WNEXT;
            break;
        default:    // PH_LM
            g.BN = p.bn[GK_LM]; g.splits = 1; g.N = p.vocab; g.K = p.d_model;
            g.map_a = MAP_A; g.map_w = MAP_WNEXT;
            break;
    }
    return g;
}

__device__ __forceinline__ int ld_relaxed(const int32_t* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until the grid barrier has been reached by every CTA (relaxed polls, one fence once it has: together an
// acquire).  False: gave up (or another role did).
__device__ __forceinline__ bool grid_wait(const int32_t* bar, int target, volatile int* abort_flag) {
    for (uint32_t it = 0; it < GRID_WAIT_LIMIT; ++it) {
        if (ld_relaxed(bar) >= target) {
            __threadfence();
            return true;
        }
        if ((it & 7u) == 7u && *abort_flag) return false;
        __nanosleep(32);
    }
    return false;
}
// The same for the worker warps of a CTA: warp WORKER_WARP0 polls global memory and passes the news on through shared
// memory, the other warps poll that word only.
__device__ __forceinline__ bool grid_wait_relayed(const int32_t* bar, int target, volatile int* relay, bool poller, volatile int* abort_flag) {
    if (poller) {
        const bool ok = grid_wait(bar, target, abort_flag);
        *relay = ok ? 1 : -1;
        return ok;
    }
    for (uint32_t it = 0; it < GRID_WAIT_LIMIT; ++it) {
        const int v = *relay;
        if (v != 0) {
            __threadfence();
            return v > 0;
        }
        if ((it & 7u) == 7u && *abort_flag) return false;
        __nanosleep(32);
    }
    return false;
}

__global__ void __launch_bounds__(THREADS, 1) decode_chain_kernel(const __grid_constant__ ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + RING_BYTES);
    // bars: full[MAX_SLOTS], empty[MAX_SLOTS], tmem_full[2], tmem_empty[2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_SLOTS + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* s_arrive = reinterpret_cast<int*>(tmem_slot + 2);          // [MAX_PHASES]
    volatile int* s_relay = reinterpret_cast<volatile int*>(s_arrive + MAX_PHASES);       // [MAX_PHASES]
    int* s_norm_cnt = s_arrive + 2 * MAX_PHASES;                    // [MAX_PHASES]
    volatile float* s_norm_red = reinterpret_cast<volatile float*>(s_norm_cnt + MAX_PHASES);     // [MAX_PHASES][8]
    const int SLOTS = p.slots, SLOT_BYTES = p.slot_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * MAX_SLOTS, tfull0 = empty0 + 8 * MAX_SLOTS, tempty0 = tfull0 + 16;
    const uint32_t tiles_u32 = smem_u32(tiles);

    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_SLOTS; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull0 + 8 * b, 1); mbar_init(tempty0 + 8 * b, 4); }
        *abort_flag = 0;
        for (int j = 0; j < MAX_PHASES; ++j) {
            s_arrive[j] = 0; s_relay[j] = 0; s_norm_cnt[j] = 0;
            for (int g = 0; g < 8; ++g) s_norm_red[j * 8 + g] = 0.f;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tc::tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (threadIdx.x == 0) stamp(p, 0, TR_KERNEL_BEGIN);
    const int M = p.M, tiles_m = (M + BM - 1) / BM;
    int32_t* bar = p.bar + (p.seg + 1) * BAR_WORDS_PER_SEG;
    const int n_cta = gridDim.x;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer of every GEMM phase ----------------
            uint32_t slot = 0, phase = 0;
            bool ok = true;
            for (int j = 0; ok; ++j) {
                const int ph = phase_at(p, j);
                if (ph == PH_END) break;
                if (!is_gemm(ph)) continue;
                const GemmDesc gd = gemm_desc(p, ph);
                const int tiles_n = (gd.N + gd.BN - 1) / gd.BN, n_tiles = tiles_m * tiles_n * gd.splits, kbt = gd.K / BK;
                const uint32_t stage_tx = A_BYTES + gd.BN * BK * 2;
                const CUtensorMap* map_a = &p.maps[gd.map_a];
                const CUtensorMap* map_w = &p.maps[gd.map_w];
                // k-blocks of this CTA in this phase, in order: (tile, kb).  The weight tile of a k-block is requested as
                // soon as its slot is free; the activation tile follows once the previous phase is complete everywhere,
                // so up to SLOTS weight tiles are already on their way when the barrier opens.
                stamp(p, j, TR_P_BEGIN);
                struct Cursor { int t, kb, kb1, m0, n0; };
                auto seek = [&](Cursor& c) {                        // geometry of tile c.t (a few integer divisions: once per tile)
                    if (c.t >= n_tiles) return;
                    const int sp = (c.t / tiles_m) % gd.splits;
                    c.m0 = (c.t % tiles_m) * BM; c.n0 = (c.t / (tiles_m * gd.splits)) * gd.BN;
                    c.kb = sp * kbt / gd.splits; c.kb1 = (sp + 1) * kbt / gd.splits;
                };
                auto advance = [&](Cursor& c) { if (++c.kb == c.kb1) { c.t += n_cta; seek(c); } };
                Cursor cb{(int)blockIdx.x, 0, 0, 0, 0};
                seek(cb);
                if (j > 0 && cb.t < n_tiles) {
                    // the phase reads what the previous phase wrote: weight tiles first, as many as there are slots
                    Cursor ca = cb;
                    uint32_t slot_b = slot, phase_b = phase;
                    int ahead = 0;
                    while (cb.t < n_tiles && ahead < SLOTS) {
                        if (!mbar_wait(empty0 + 8 * slot_b, phase_b ^ 1u, abort_flag)) { ok = false; break; }
                        mbar_arrive_expect_tx(full0 + 8 * slot_b, stage_tx);
                        tma_load_2d(tiles_u32 + slot_b * SLOT_BYTES + A_BYTES, map_w, full0 + 8 * slot_b, cb.kb * BK, cb.n0);
                        ++ahead;
                        if (++slot_b == (uint32_t)SLOTS) { slot_b = 0; phase_b ^= 1u; }
                        advance(cb);
                    }
                    if (!ok) break;
                    if (!grid_wait(bar + (j - 1), n_cta, abort_flag)) { ok = false; break; }
                    asm volatile("fence.proxy.async;" ::: "memory");             // other CTAs' stores before this thread's TMA reads
                    stamp(p, j, TR_P_BARRIER);
                    for (; ahead > 0; --ahead) {
                        tma_load_2d(tiles_u32 + slot * SLOT_BYTES, map_a, full0 + 8 * slot, ca.kb * BK, ca.m0);
                        if (++slot == (uint32_t)SLOTS) { slot = 0; phase ^= 1u; }
                        advance(ca);
                    }
                }
                while (cb.t < n_tiles) {
                    if (!mbar_wait(empty0 + 8 * slot, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t sa = tiles_u32 + slot * SLOT_BYTES;
                    mbar_arrive_expect_tx(full0 + 8 * slot, stage_tx);
                    tma_load_2d(sa + A_BYTES, map_w, full0 + 8 * slot, cb.kb * BK, cb.n0);
                    tma_load_2d(sa, map_a, full0 + 8 * slot, cb.kb * BK, cb.m0);
                    if (++slot == (uint32_t)SLOTS) { slot = 0; phase ^= 1u; }
                    advance(cb);
                }
                if (!ok) break;
                stamp(p, j, TR_P_DONE);
            }
            if (!ok) { *abort_flag = 1; set_error(p.err, DEV_ERR_WAIT_TIMEOUT); }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            uint32_t slot = 0, phase = 0, acc = 0, acc_phase = 0;
            bool ok = true;
            for (int j = 0; ok; ++j) {
                const int ph = phase_at(p, j);
                if (ph == PH_END) break;
                if (!is_gemm(ph)) continue;
                const GemmDesc gd = gemm_desc(p, ph);
                const int tiles_n = (gd.N + gd.BN - 1) / gd.BN, n_tiles = tiles_m * tiles_n * gd.splits, kbt = gd.K / BK;
                const uint32_t idesc = tc::make_idesc(BM, gd.BN, true);
                bool first = true;
                for (int t = blockIdx.x; t < n_tiles && ok; t += n_cta) {
                    if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * ACC_COLS;
                    const int sp = (t / tiles_m) % gd.splits;
                    const int k_blocks = (sp + 1) * kbt / gd.splits - sp * kbt / gd.splits;
                    for (int kb = 0; kb < k_blocks; ++kb) {
                        if (!mbar_wait(full0 + 8 * slot, phase, abort_flag)) { ok = false; break; }
                        if (first) { stamp(p, j, TR_M_FIRST_FULL); first = false; }
                        tc::tc_fence_after();
                        const uint32_t sa = tiles_u32 + slot * SLOT_BYTES, sb = sa + A_BYTES;
                        const uint64_t da = tc::make_smem_desc(sa), db = tc::make_smem_desc(sb);
#pragma unroll
                        for (int kk = 0; kk < BK / tc::UMMA_K; ++kk)
                            tc::umma_bf16(d_tmem, da + 2 * kk, db + 2 * kk, idesc, (kb | kk) != 0 ? 1u : 0u);
                        tc::umma_commit(empty0 + 8 * slot);
                        if (++slot == (uint32_t)SLOTS) { slot = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    tc::umma_commit(tfull0 + 8 * acc);
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
                stamp(p, j, TR_M_DONE);
            }
            if (!ok) { *abort_flag = 1; set_error(p.err, DEV_ERR_WAIT_TIMEOUT); }
        }
    } else {
        // ---------------- worker warps: epilogues (warps 4..7) and row-wise phases (warps 2..7) ----------------
        const int m_live = min(M, p.sd->n_rows);
        const int gw = blockIdx.x * N_WORKER_WARPS + (warp - WORKER_WARP0), n_gw = n_cta * N_WORKER_WARPS;
        const int quarter = warp & 3;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int j = 0; ok; ++j) {
            const int ph = phase_at(p, j);
            if (ph == PH_END) break;
            const int l_here = p.seg < 0 ? 0 : p.seg;
            const bool last_layer = p.seg == p.n_layers - 1;
            const bool tracer = lane == 0 && warp == (is_gemm(ph) ? 4 : WORKER_WARP0);
            if (tracer) stamp(p, j, TR_W_BEGIN);
            if (is_gemm(ph)) {
                if (warp >= 4) {
                    const GemmDesc gd = gemm_desc(p, ph);
                    const int tiles_n = (gd.N + gd.BN - 1) / gd.BN, n_tiles = tiles_m * tiles_n * gd.splits;
                    tc::EpiPartial e_part{nullptr, 0, 0};
                    tc::EpiResidual e_res{p.h, p.d_model};
                    const tc::EpiSwiGLU e_glu{p.act, p.d_ff, 1, p.err};
                    const tc::EpiStoreF32 e_st{p.logits, p.vocab, nullptr};
                    int ek;                                      // 0 partial, 1 residual, 2 SwiGLU, 3 store
                    if (ph == PH_QKV) { e_part = tc::EpiPartial{p.qkv, p.n_qkv, (size_t)M * p.n_qkv}; ek = 0; }
                    else if (ph == PH_GU) ek = 2;
                    else if (ph == PH_LM) ek = 3;
                    else if (gd.splits > 1) { e_part = tc::EpiPartial{p.res_part, p.d_model, (size_t)M * p.d_model}; ek = 0; }
                    else ek = 1;
                    for (int t = blockIdx.x; t < n_tiles && ok; t += n_cta) {
                        const int m0 = (t % tiles_m) * BM, sp = (t / tiles_m) % gd.splits, n0 = (t / (tiles_m * gd.splits)) * gd.BN;
                        if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
                        if (tracer && t == (int)blockIdx.x) stamp(p, j, TR_E_FIRST_FULL);
                        tc::tc_fence_after();
                        const int row = m0 + quarter * 32 + lane;
#pragma unroll 1
                        for (int c = 0; c < gd.BN; c += 32) {
                            if (n0 + c >= gd.N) break;                 // warp-uniform
                            float v[32];
                            tc::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * ACC_COLS + c, v);
                            if (row < m_live) {
                                const int nv = min(32, gd.N - (n0 + c));
                                if (ek == 0) e_part(row, n0 + c, v, nv, sp);
                                else if (ek == 1) e_res(row, n0 + c, v, nv, sp);
                                else if (ek == 2) e_glu(row, n0 + c, v, nv, sp);
                                else e_st(row, n0 + c, v, nv, sp);
                            }
                        }
                        tc::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
                        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                    }
                }
            } else {
                // a row-wise phase reads what the previous phase wrote anywhere on the GPU
                if (j > 0) {
                    int good = 1;
                    if (lane == 0) good = grid_wait_relayed(bar + (j - 1), n_cta, s_relay + j, warp == WORKER_WARP0, abort_flag) ? 1 : 0;
                    good = __shfl_sync(0xffffffffu, good, 0);
                    if (!good) { ok = false; break; }
                }
                if (tracer) stamp(p, j, TR_W_WAITED);
                if (ph == PH_EMBED || ph == PH_NORM_MLP || ph == PH_NORM_NEXT) {
                    Partials pend{nullptr, 0, 0, 0};
                    const float* gain;
                    if (ph == PH_EMBED) gain = p.layers[0].attn_norm;
                    else if (ph == PH_NORM_MLP) {
                        gain = p.layers[l_here].mlp_norm;
                        if (p.splits[GK_O] > 1) pend = Partials{p.res_part, p.splits[GK_O], (size_t)M * p.d_model, p.d_model};
                    } else {
                        gain = last_layer ? p.glob->final_norm : p.layers[l_here + 1].attn_norm;
                        if (p.splits[GK_DOWN] > 1) pend = Partials{p.res_part, p.splits[GK_DOWN], (size_t)M * p.d_model, p.d_model};
                    }
                    if (m_live <= n_cta && norm_row_fits_cta(p.d_model)) {
                        // few rows: one row per CTA, its segments spread over the worker warps (one memory round trip per row)
                        const int r = blockIdx.x, w = warp - WORKER_WARP0;
                        if (r < m_live) {
                            float* h_row = p.h + (size_t)r * p.d_model;
                            if (ph == PH_EMBED) {
                                const __nv_bfloat16* e_row = reinterpret_cast<const __nv_bfloat16*>(p.embed) + (size_t)p.g.token[r] * p.d_model;
                                for (int kk = 0; kk < 8; ++kk) {
                                    const int i = lane + 32 * (w + NORM_SEGS * kk);
                                    if (i < (p.d_model >> 2)) {
                                        float v[4];
                                        VecLoad<__nv_bfloat16, 4>::load(e_row + 4 * i, v);
                                        reinterpret_cast<float4*>(h_row)[i] = make_float4(v[0], v[1], v[2], v[3]);
                                    }
                                }
                            }
                            if (!norm_row_cta<__nv_bfloat16>(w, lane, p.d_model, h_row, pend, (size_t)r * p.d_model, gain, p.eps,
                                                             p.a + (size_t)r * p.d_model, nullptr, 1, s_norm_red + j * 8, s_norm_cnt + j, p.err)) {
                                ok = false;
                                break;
                            }
                        }
                    } else {
                        for (int r = gw; r < m_live; r += n_gw) {
                            float* h_row = p.h + (size_t)r * p.d_model;
                            if (ph == PH_EMBED)
                                embed_row_warp<__nv_bfloat16>(lane, p.d_model,
                                                              reinterpret_cast<const __nv_bfloat16*>(p.embed) + (size_t)p.g.token[r] * p.d_model, h_row);
                            norm_row_warp<__nv_bfloat16>(lane, p.d_model, h_row, pend, (size_t)r * p.d_model, gain, p.eps,
                                                         p.a + (size_t)r * p.d_model, nullptr, 1, p.err);
                        }
                    }
                } else if (ph == PH_POST) {
                    const int layer = p.seg + 1;
                    const LayerTab& lt = p.layers[layer];
                    const QkvPostArgs<__nv_bfloat16> A{p.Hq, p.Hkv, p.hd, layer,
                                                      Partials{p.qkv, p.splits[GK_QKV], (size_t)M * p.n_qkv, p.n_qkv},
                                                      lt.bqkv, lt.q_norm, lt.k_norm, p.eps, p.rope, p.g, p.prompt_arena, p.suffix_arena, p.q, p.err};
                    const int n_heads = p.Hq + 2 * p.Hkv, items = m_live * n_heads;
                    const int per_warp = (items + n_gw - 1) / n_gw;
                    const int i_end = min(items, (gw + 1) * per_warp);
                    for (int i0 = gw * per_warp; i0 < i_end; i0 += 4) {
                        int rows[4], heads[4];
                        const int nb = min(4, i_end - i0);
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            const int it = min(i0 + b, items - 1);
                            rows[b] = it / n_heads;
                            heads[b] = it - rows[b] * n_heads;
                        }
                        // straight-line code per batch size: the loads of all items are in flight together
                        if (nb == 4) qkv_post_items_warp<__nv_bfloat16, 4>(lane, A, rows, heads, 4);
                        else if (nb == 3) qkv_post_items_warp<__nv_bfloat16, 3>(lane, A, rows, heads, 3);
                        else if (nb == 2) qkv_post_items_warp<__nv_bfloat16, 2>(lane, A, rows, heads, 2);
                        else qkv_post_items_warp<__nv_bfloat16, 1>(lane, A, rows, heads, 1);
                    }
                } else if (ph == PH_MERGE) {
                    const int items = m_live * p.Hq;
                    const am::SuffixPlan sp = am::suffix_plan(*p.g.max_slen, p.sd->n_rows * p.part.n_kv_heads, p.part.n_suffix_warps);
                    const int n_load = p.part.n_parts + sp.cpi;
                    for (int it = gw; it < items; it += n_gw) {
                        if (p.hd == 128) am::merge_item_warp<128>(lane, it, p.Hq, p.g, p.part, sp.ct, n_load, p.attn, nullptr, p.err);
                        else am::merge_item_warp<64>(lane, it, p.Hq, p.g, p.part, sp.ct, n_load, p.attn, nullptr, p.err);
                    }
                }
            }
            // this warp's part of phase j is done: the CTA's last worker warp signals the grid barrier
            if (tracer) stamp(p, j, TR_W_DONE);
            __threadfence();
            __syncwarp();
            if (lane == 0) {
                const int old = atomicAdd(&s_arrive[j], 1);
                if (old == N_WORKER_WARPS - 1) {
                    __threadfence();
                    atomicAdd(bar + j, 1);
                }
            }
        }
        if (!ok && lane == 0) { *abort_flag = 1; set_error(p.err, DEV_ERR_WAIT_TIMEOUT); }
    }

    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp(p, 0, TR_KERNEL_END);
    if (*abort_flag) {
        // give copies that may still be in flight time to land before the shared memory is released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace chain
}  // namespace pc
