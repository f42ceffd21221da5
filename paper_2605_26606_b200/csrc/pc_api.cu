// C ABI of the Pilot-Commit rollout engine: argument checks, workspace carving and kernel sequencing.
// See include/pc.h for the contract of every entry point.
#include "../../include/pc.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <type_traits>
#include <utility>
#include <vector>

#include "attention_mma.cuh"
#include "attention_simt.cuh"
#include "common.cuh"
#include "decode_chain.cuh"
#include "gemm_simt.cuh"
#include "gemm_epilogues.cuh"
#include "gemm_tc.cuh"
#include "kernels_basic.cuh"
#include "lm_sample.cuh"
#include "sampler.cuh"
#include "stats.cuh"
#include "tensor_map.h"

namespace {

thread_local std::string g_cuda_error;
std::atomic<unsigned long long> g_launches{0};     // kernels launched by this library since it was loaded (all contexts, all threads)
thread_local long long g_capture_launches = -1;    // >= 0 while this thread captures a decode step: launches recorded, not run
inline void count_launches(int n) {
    if (g_capture_launches >= 0) g_capture_launches += n;
    else g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed);
}

int cuda_fail(cudaError_t e, const char* what) {
    g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    return PC_ERR_CUDA;
}

#define PC_CUDA_CHECK_LAUNCH(what)                                  \
    do {                                                            \
        cudaError_t e__ = cudaGetLastError();                       \
        if (e__ != cudaSuccess) return cuda_fail(e__, what);        \
    } while (0)

// Kernel launch through the extensible launch call (one place to add launch attributes).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

// The same launch as a programmatic dependent of the kernel before it in the stream (see grid_dep_wait in common.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k_dep(bool dep, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (dep) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

constexpr size_t kSplitMaxRows = 512;   // row count up to which the partial-sum buffers hold kMaxSplits K-slices; narrow tiles split only up to here
constexpr int kMaxSplits = pc::PARTIALS_MAX;

struct Carve {
    size_t h, a, qkv, q, attn, act, logits, rope, pos, wslot, warena, p_start, p_len, s_start, s_len, token, last_row,
        part_m, part_l, part_o, res_part, step_desc, step_counter, max_slen, sample_scratch, a_lo, attn_lo, chain_layers, chain_glob,
        chain_bar, dargs, key_prompt, key_rollout, key_step, out_index, group_start, sample_tiles, sample_bound, ssq, total;
};

// A captured decode step, replayable for every step that fits the same upper bounds on the same KV arenas.  The
// caller's row arrays, token buffer and sampling parameters are not part of the key: the captured kernels read them
// from the device-resident argument block (DecodeArgsDev) that every call rewrites.
struct GraphKey {
    int m_bound, groups_bound, group_rows_bound, sample, logprobs, decode_mode;
    const void* prompt_kv; int64_t prompt_slots;
    const void* suffix_kv; int64_t suffix_slots;
};
struct GraphEntry {
    GraphKey key;
    cudaGraphExec_t exec;
    int launches;       // kernels in the graph
};

// TMA descriptors of one bf16 weight matrix [N, K], one per tile width the GEMM may pick.
struct WMap {
    CUtensorMap wide, narrow, mid;   // boxes of 256, 64 and 128 rows
    int N = 0, K = 0;
};

}  // namespace

struct pc_ctx {
    pc_model_desc d;
    const void* embed;
    const void* lm_head;
    const float* final_norm;
    std::vector<const float*> attn_norm, bqkv, q_norm, k_norm, mlp_norm;
    std::vector<const void*> wqkv, wo, w_gate_up, w_down;
    // workspace
    char* ws = nullptr;
    size_t ws_bytes = 0;
    int max_rows = 0, max_prefill = 0;
    int32_t* err = nullptr;
    Carve cv{};
    // bf16 models: TMA descriptors of the weights (built by pc_create) and of the activation buffers
    // (built by pc_set_workspace over the full capacity of each buffer)
    std::vector<WMap> m_wqkv, m_wo, m_wgu, m_wdown;
    WMap m_lm;
    pc::Partials pend{nullptr, 0, 0, 0};     // residual K-slices produced by the last GEMM and not yet folded into h
    CUtensorMap map_a, map_attn, map_act, map_a_lo, map_attn_lo;
    int num_sms = 148;
    // TMA descriptors of the KV arenas, rebuilt when a call brings another arena
    const void* prompt_arena_ptr = nullptr; int64_t prompt_arena_slots = -1; CUtensorMap map_prompt_kv;
    const void* suffix_arena_ptr = nullptr; int64_t suffix_arena_slots = -1; CUtensorMap map_suffix_kv;
    // one-shot profiling request (pc_profile_step): events recorded at the phase boundaries of one layer and of the step's tail
    int prof_layer = -1;                     // armed when >= 0
    int prof_active_layer = -1;              // the step being issued records into prof_ev
    cudaEvent_t prof_ev[PC_PROFILE_MARKS] = {};
    void mark(cudaStream_t st, int layer, int m) {      // layer < 0: a boundary of the step's tail (LM head, sampler)
        if (prof_active_layer >= 0 && (layer < 0 || layer == prof_active_layer) && prof_ev[m] != nullptr) cudaEventRecord(prof_ev[m], st);
    }
    float* logprobs = nullptr;       // pc_set_logprob_buffer
    const int32_t* prompt_key = nullptr;    // pc_set_prompt_keys

    // tile width / K-split forced through pc_set_gemm_plan (0 = built-in choice), indexed by GemmKind
    int plan_bn[5] = {0, 0, 0, 0, 0}, plan_splits[5] = {0, 0, 0, 0, 0};
    size_t split_capacity_rows = 0;          // rows x K-slices the partial-sum buffers hold

    int decode_mode = 0;                     // 1: persistent chain kernel between attention calls (half-operand bf16 models); 0: one kernel per operation
    bool chain_ready = false;                // tables uploaded by pc_set_workspace
    long long* chain_trace = nullptr;        // pc_set_chain_trace
    unsigned long long captures = 0;         // decode steps captured and instantiated so far (pc_capture_count)
    int32_t n_prompts_hint = 0;              // pc_set_index_bounds: sizes of the caller's per-prompt arrays and token buffer (0: unknown)
    int64_t n_tokens_hint = 0;

    int fused_epilogues = 1;                 // half-operand models with head_dim 128: QKV post-processing and the MLP norm inside GEMM epilogues
    int fused_sampler = 0;                   // decode steps that only sample: Gumbel-max in the LM head's epilogue, no logits stored
    int dep_launch = 63;                     // bit per kernel (1 QKV, 2 output, 4 gate/up, 8 down projection, 16 LM head, 32 shared-prefix attention): launched as a programmatic dependent of the kernel before it
    int attn_overlap = 0;                    // decode: shared-prefix and suffix attention kernels of a layer on two streams
    cudaStream_t side_stream = nullptr;      // second branch of that fork (created on first use)
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;

    std::vector<GraphEntry> graphs;
    cudaStream_t capture_stream = nullptr;      // decode steps are captured here (the caller's stream may be the default one)
    void drop_graphs() {
        for (auto& g : graphs) cudaGraphExecDestroy(g.exec);
        graphs.clear();
    }
    ~pc_ctx() {
        drop_graphs();
        if (capture_stream) cudaStreamDestroy(capture_stream);
        if (side_stream) cudaStreamDestroy(side_stream);
        if (ev_fork) cudaEventDestroy(ev_fork);
        if (ev_join) cudaEventDestroy(ev_join);
    }

    int n_qkv() const { return (d.n_q_heads + 2 * d.n_kv_heads) * d.head_dim; }
    int q_dim() const { return d.n_q_heads * d.head_dim; }
    size_t eb() const { return d.dtype == PC_DTYPE_F32 ? 4 : 2; }
};

namespace {

inline size_t chain_bar_words(int n_layers) { return (size_t)(n_layers + 1) * pc::chain::BAR_WORDS_PER_SEG; }

Carve carve(const pc_ctx* c, int max_rows, int max_prefill) {
    const pc_model_desc& d = c->d;
    const size_t M = (size_t)std::max(max_rows, max_prefill), eb = c->eb();
    Carve v{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    v.h = take(M * d.d_model * 4);
    v.a = take(M * d.d_model * eb);
    const size_t split_rows = std::min<size_t>(M, kSplitMaxRows) * kMaxSplits;      // rows x K-slices of a split GEMM
    v.qkv = take(std::max(M, split_rows) * c->n_qkv() * 4);
    v.res_part = take(split_rows * d.d_model * 4);
    v.a_lo = take(M * d.d_model * eb);
    v.attn_lo = take(M * c->q_dim() * eb);
    v.chain_layers = take((size_t)d.n_layers * sizeof(pc::chain::LayerTab));
    v.chain_glob = take(sizeof(pc::chain::GlobalTab));
    v.chain_bar = take(chain_bar_words(d.n_layers) * 4);
    v.step_desc = take(sizeof(pc::StepDesc));
    v.step_counter = take(4);
    v.max_slen = take(4);
    v.sample_scratch = take((size_t)std::max(max_rows, 1) * pc::SAMPLE_MAX_CHUNKS * sizeof(pc::Top2Rec));
    v.q = take(M * c->q_dim() * eb);
    v.attn = take(M * c->q_dim() * eb);
    v.act = take(M * (size_t)d.d_ff * eb);
    v.logits = take((size_t)std::max(max_rows, 1) * d.vocab * 4);
    v.rope = take(M * (d.head_dim / 2) * 8);
    v.pos = take(M * 4);
    v.wslot = take(M * 8);
    v.warena = take(M * 4);
    v.p_start = take(M * 8);
    v.p_len = take(M * 4);
    v.s_start = take(M * 8);
    v.s_len = take(M * 4);
    v.token = take(M * 4);
    v.last_row = take(M * 4);
    v.dargs = take(sizeof(pc::DecodeArgsDev));
    v.key_prompt = take(M * 4);
    v.key_rollout = take(M * 4);
    v.key_step = take(M * 4);
    v.out_index = take(M * 8);
    v.group_start = take((M + 1) * 4);
    v.ssq = take((size_t)((d.d_model + 63) / 64) * M * 4);       // per-tile sums of squares of the residual rows (EpiResNorm)
    // fused LM head + sampler: one record per (vocabulary tile of the narrowest tile width, row)
    v.sample_tiles = take(2 * (size_t)((d.vocab + 63) / 64) * (size_t)std::max(max_rows, 1) * sizeof(pc::Top2Rec));   // one record per half tile
    v.sample_bound = take((size_t)std::max(max_rows, 1) * sizeof(int32_t));
    // prefix part of the shared-prefix attention: (max, sum, unnormalised output) per (row, query head)
    const size_t R = (size_t)std::max(max_rows, 1);
    v.part_m = take(pc::am::MAX_RECORDS * R * d.n_q_heads * 4);
    v.part_l = take(pc::am::MAX_RECORDS * R * d.n_q_heads * 4);
    v.part_o = take(pc::am::MAX_RECORDS * R * d.n_q_heads * d.head_dim * 4);
    v.total = off;
    return v;
}

pc::RowGeom geom(const pc_ctx* c) {
    pc::RowGeom g;
    char* w = c->ws;
    g.pos = reinterpret_cast<int32_t*>(w + c->cv.pos);
    g.wslot = reinterpret_cast<int64_t*>(w + c->cv.wslot);
    g.warena = reinterpret_cast<int32_t*>(w + c->cv.warena);
    g.p_start = reinterpret_cast<int64_t*>(w + c->cv.p_start);
    g.p_len = reinterpret_cast<int32_t*>(w + c->cv.p_len);
    g.s_start = reinterpret_cast<int64_t*>(w + c->cv.s_start);
    g.s_len = reinterpret_cast<int32_t*>(w + c->cv.s_len);
    g.token = reinterpret_cast<int32_t*>(w + c->cv.token);
    g.max_slen = reinterpret_cast<int32_t*>(w + c->cv.max_slen);
    return g;
}

bool make_wmap(WMap* w, const void* base, int N, int K) {
    w->N = N;
    w->K = K;
    return pc::make_bf16_map(&w->wide, base, N, K, 256) && pc::make_bf16_map(&w->narrow, base, N, K, 64) &&
           pc::make_bf16_map(&w->mid, base, N, K, 128);
}

// Tile width and K-split of a bf16 GEMM over M rows.  Large batches take 128 x 256 tiles.  Small batches would
// leave most SMs idle (the weight matrix is then streamed by a few CTAs only), so they take 128 x 64 tiles and,
// where the epilogue allows it, split K so that about one CTA per SM is busy; the K-slices are summed in a
// fixed order by the kernel that consumes the result.
struct GemmPlan {
    bool wide;
    int splits;
    bool mid = false;      // 128-column tiles (split-K partial sums and the SwiGLU epilogue with one operand matrix only)
};
enum GemmKind { GEMM_QKV = 0, GEMM_O = 1, GEMM_GATE_UP = 2, GEMM_DOWN = 3, GEMM_LM_HEAD = 4 };
enum DepBit { DEP_QKV = 1, DEP_O = 2, DEP_GATE_UP = 4, DEP_DOWN = 8, DEP_LM_HEAD = 16, DEP_GROUP = 32 };      // bits of pc_ctx::dep_launch
GemmPlan plan_gemm(const pc_ctx* c, GemmKind kind, const WMap& w, int M, bool may_split) {
    const int tiles_m = (M + pc::tc::BM - 1) / pc::tc::BM;
    const int k_blocks = w.K / pc::tc::BK;
    // K-slices the partial-sum buffers can hold for M rows, and never fewer than 4 k-blocks per slice
    const int max_splits = !may_split ? 1 : std::max(1, std::min(std::min((int)(c->split_capacity_rows / (size_t)std::max(M, 1)), kMaxSplits), k_blocks / 4));
    GemmPlan p{true, 1};
    if (c->plan_bn[kind] != 0) {
        p.wide = c->plan_bn[kind] == 256;
        p.mid = c->plan_bn[kind] == 128;
        p.splits = std::max(1, std::min(c->plan_splits[kind], max_splits));
        return p;
    }
    const int tiles_wide = tiles_m * ((w.N + 255) / 256);
    if (tiles_wide >= c->num_sms / 2) return p;
    // gate/up with one row tile: 128-column tiles give one tile per SM (140 for the 1.5B shape), where 256 columns leave half
    // the SMs without a weight stream and 64 columns fetch the activation tile twice as often (measured: -4 % of a 64-row step)
    if (kind == GEMM_GATE_UP && !may_split && tiles_m * ((w.N + 127) / 128) <= c->num_sms) {
        p.wide = false;
        p.mid = true;
        return p;
    }
    // Too few wide tiles to keep the SMs busy.  A wide tile moves half as many bytes from L2 into shared memory per
    // flop as a narrow one, so from three row tiles on (and enough K per tile for that traffic to matter; crossover
    // measured on the 1.5B shape at 128..896 rows) the wide tile stays and K is split until about every SM has a CTA.
    if (may_split && tiles_m >= 3 && (long long)tiles_m * w.K >= 7680) {
        p.splits = std::max(1, std::min(c->num_sms / tiles_wide, max_splits));
        return p;
    }
    p.wide = false;
    const int tiles = tiles_m * ((w.N + 63) / 64);
    if ((size_t)M <= kSplitMaxRows) p.splits = std::max(1, std::min(c->num_sms / tiles, max_splits));
    return p;
}

// Whether a projection over M rows is launched as a programmatic dependent (pc_set_dependent_launch).  Not in steps that
// record phase events (an event between two kernels is no kernel-to-kernel edge), and not for passes of two row tiles:
// measured on the 1.5B shape, decode steps of 16 / 64 / 128 rows take 6.7 / 5.4 / 4.4 % less time with it, steps of 192 and
// 256 rows 1.8 % more, 384 rows the same, 560 rows 2 % less.
inline bool dependent_launch(const pc_ctx* c, int dep_bit, int M) {
    return (c->dep_launch & dep_bit) != 0 && c->prof_active_layer < 0 && (dep_bit == DEP_GROUP || !(M > pc::tc::BM && M <= 2 * pc::tc::BM));
}

// map_a_lo != nullptr: the activations come as a high bf16 part and its rounding remainder, both multiplied with the
// weights (used for the projections whose input rounding would otherwise dominate the logit error).
template <class Epi>
int gemm_bf16(pc_ctx* c, cudaStream_t st, const pc::StepDesc* sd, const CUtensorMap& map_a, const CUtensorMap* map_a_lo, const WMap& w,
              int M, GemmPlan p, Epi epi, bool half_operands = false, int dep_bit = 0) {
    // dep: launched as a programmatic dependent.  Every projection of a pass follows a kernel that signals its dependents
    // early (a row norm, the attention merge, another projection), so this launch may set itself up and request its first
    // weight tiles while that kernel is still running; after any other kernel it simply starts when that one has ended.
    const bool dep = dependent_launch(c, dep_bit, M);
    cudaError_t e;
    if (map_a_lo != nullptr)
        e = p.wide ? pc::tc::launch<256, true>(st, map_a, *map_a_lo, w.wide, sd, M, w.N, w.K, p.splits, epi, c->err, c->num_sms, false, dep)
                   : pc::tc::launch<64, true>(st, map_a, *map_a_lo, w.narrow, sd, M, w.N, w.K, p.splits, epi, c->err, c->num_sms, false, dep);
    else if (p.mid && !p.wide && (std::is_same<Epi, pc::tc::EpiPartial>::value || std::is_same<Epi, pc::tc::EpiSwiGLU>::value)) {
        if constexpr (std::is_same<Epi, pc::tc::EpiPartial>::value || std::is_same<Epi, pc::tc::EpiSwiGLU>::value)
            e = pc::tc::launch<128, false>(st, map_a, map_a, w.mid, sd, M, w.N, w.K, p.splits, epi, c->err, c->num_sms, half_operands, dep);
        else
            e = cudaErrorInvalidValue;
    } else
        e = p.wide ? pc::tc::launch<256, false>(st, map_a, map_a, w.wide, sd, M, w.N, w.K, p.splits, epi, c->err, c->num_sms, half_operands, dep)
                   : pc::tc::launch<64, false>(st, map_a, map_a, w.narrow, sd, M, w.N, w.K, p.splits, epi, c->err, c->num_sms, half_operands, dep);
    if (e != cudaSuccess) return cuda_fail(e, "tensor-core gemm");
    return PC_OK;
}

// Unsplit GEMM with an explicit tile width (the fused epilogues need complete sums in a tile).
template <int BN, class Epi>
int gemm_half_bn(pc_ctx* c, cudaStream_t st, const pc::StepDesc* sd, const CUtensorMap& map_a, const WMap& w, int M, Epi epi, int dep_bit = 0) {
    const CUtensorMap& mw = BN == 256 ? w.wide : (BN == 128 ? w.mid : w.narrow);
    const bool dep = dependent_launch(c, dep_bit, M);
    const cudaError_t e = pc::tc::launch<BN, false>(st, map_a, map_a, mw, sd, M, w.N, w.K, 1, epi, c->err, c->num_sms, true, dep);
    if (e != cudaSuccess) return cuda_fail(e, "tensor-core gemm (fused epilogue)");
    return PC_OK;
}
inline bool wide_tiles_fill_the_gpu(const pc_ctx* c, int M, int N) {
    return ((M + pc::tc::BM - 1) / pc::tc::BM) * ((N + 255) / 256) >= c->num_sms / 2;
}

// How the rows of a forward pass group for attention.
struct AttnPlan {
    bool prefill;                      // true: causal attention inside each prompt, no suffix part
    int n_groups;                      // upper bound used for the grid; the live count is in the step descriptor
    const int32_t* group_row_start;    // device; the step's entries start at the descriptor's group_off
    int max_group_rows;                // upper bound
};

int arena_maps(pc_ctx* c, const void* prompt_kv, int64_t prompt_slots, const void* suffix_kv, int64_t suffix_slots) {
    const pc_model_desc& d = c->d;
    const uint64_t planes = (uint64_t)d.n_layers * 2 * d.n_kv_heads;
    if (prompt_kv != c->prompt_arena_ptr || prompt_slots != c->prompt_arena_slots) {
        if (planes * (uint64_t)prompt_slots >= (1ull << 31)) return PC_ERR_CAPACITY;
        if (!pc::make_bf16_map(&c->map_prompt_kv, prompt_kv, planes * prompt_slots, d.head_dim, pc::am::G_TK)) {
            g_cuda_error = "cuTensorMapEncodeTiled failed for the prompt KV arena";
            return PC_ERR_CUDA;
        }
        c->prompt_arena_ptr = prompt_kv; c->prompt_arena_slots = prompt_slots;
    }
    if (suffix_kv != nullptr && (suffix_kv != c->suffix_arena_ptr || suffix_slots != c->suffix_arena_slots)) {
        if (planes * (uint64_t)suffix_slots >= (1ull << 31)) return PC_ERR_CAPACITY;
        if (!pc::make_bf16_map(&c->map_suffix_kv, suffix_kv, planes * suffix_slots, d.head_dim, pc::am::S_TP)) {
            g_cuda_error = "cuTensorMapEncodeTiled failed for the suffix KV arena";
            return PC_ERR_CUDA;
        }
        c->suffix_arena_ptr = suffix_kv; c->suffix_arena_slots = suffix_slots;
    }
    return PC_OK;
}

// Raises the dynamic shared memory limit of every tensor-core kernel instance (once per process and device).
template <int HD>
cudaError_t configure_attention() {
    using namespace pc;
    cudaError_t e = cudaFuncSetAttribute(am::attn_group_kernel<HD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         am::group_smem_bytes<HD>());
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(am::attn_group_kernel<HD, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 am::group_smem_bytes<HD>());
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(am::attn_suffix_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, am::suffix_smem_bytes<HD>());
    return e;
}
cudaError_t configure_kernels() {
    using namespace pc;
    cudaError_t e = tc::configure<256, true, tc::EpiPartial>();
    if (e == cudaSuccess) e = tc::configure<64, true, tc::EpiPartial>();
    if (e == cudaSuccess) e = tc::configure<256, false, tc::EpiPartial>();
    if (e == cudaSuccess) e = tc::configure<64, false, tc::EpiPartial>();
    if (e == cudaSuccess) e = tc::configure<256, true, tc::EpiResidual>();
    if (e == cudaSuccess) e = tc::configure<64, true, tc::EpiResidual>();
    if (e == cudaSuccess) e = tc::configure<256, false, tc::EpiResidual>();
    if (e == cudaSuccess) e = tc::configure<64, false, tc::EpiResidual>();
    if (e == cudaSuccess) e = tc::configure<256, false, tc::EpiSwiGLU>();
    if (e == cudaSuccess) e = tc::configure<64, false, tc::EpiSwiGLU>();
    if (e == cudaSuccess) e = tc::configure<128, false, tc::EpiSwiGLU>();
    if (e == cudaSuccess) e = tc::configure<128, false, tc::EpiPartial>();
    if (e == cudaSuccess) e = tc::configure<256, true, tc::EpiStoreF32>();
    if (e == cudaSuccess) e = tc::configure<64, true, tc::EpiStoreF32>();
    if (e == cudaSuccess) e = tc::configure<256, false, tc::EpiStoreF32>();
    if (e == cudaSuccess) e = tc::configure<64, false, tc::EpiStoreF32>();
    if (e == cudaSuccess) e = tc::configure<128, false, EpiQkvPost>();
    if (e == cudaSuccess) e = tc::configure<256, false, EpiQkvPost>();
    if (e == cudaSuccess) e = tc::configure<64, false, EpiResNorm>();
    if (e == cudaSuccess) e = tc::configure<256, false, EpiResNorm>();
    if (e == cudaSuccess) e = tc::configure<64, false, EpiSwiGLUNorm>();
    if (e == cudaSuccess) e = tc::configure<256, false, EpiSwiGLUNorm>();
    if (e == cudaSuccess) e = tc::configure<256, true, EpiSample>();
    if (e == cudaSuccess) e = tc::configure<64, true, EpiSample>();
    if (e == cudaSuccess) e = tc::configure<256, false, EpiSample>();
    if (e == cudaSuccess) e = tc::configure<64, false, EpiSample>();
    if (e == cudaSuccess) e = configure_attention<128>();
    if (e == cudaSuccess) e = configure_attention<64>();
    return e;
}

// part_out != nullptr: the records are left unmerged and described there (the caller merges them).
template <int HD>
int attention_bf16(pc_ctx* c, cudaStream_t st, const pc::StepDesc* sd, int M, int layer, const AttnPlan& plan, pc::KvArena prompt_arena,
                   pc::KvArena suffix_arena, const __nv_bfloat16* q, __nv_bfloat16* attn,
                   pc::am::PrefixPartial* part_out = nullptr) {
    using namespace pc;
    const pc_model_desc& d = c->d;
    // half_gemm: the attention output is written once, as IEEE half; else as bf16 plus its bf16 rounding remainder
    __nv_bfloat16* attn_lo = d.half_gemm ? nullptr : reinterpret_cast<__nv_bfloat16*>(c->ws + c->cv.attn_lo);
    const RowGeom g = geom(c);
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)d.head_dim);
    const int n_rep = d.n_q_heads / d.n_kv_heads;
    // a group with few query rows keeps few CTAs busy: cut its prompt into ranges so that about one CTA per SM runs
    const int q_tiles = (plan.max_group_rows * n_rep + am::G_QROWS - 1) / am::G_QROWS;
    const int base_ctas = std::max(1, q_tiles * d.n_kv_heads * plan.n_groups);
    // (two of these CTAs fit on an SM)
    const int n_parts = plan.prefill ? 1 : std::max(1, std::min(am::MAX_PREFIX_PARTS, 2 * c->num_sms / base_ctas));
    // the suffix kernel takes one warp per (rollout, KV head, range of the suffix); how the suffixes are cut into ranges
    // is decided on the device for the warps of this grid (the longest suffix of the step is only known there)
    const int items = M * d.n_kv_heads * am::MAX_SUFFIX_CHUNKS;
    const int sgrid = std::min(c->num_sms, (items + am::S_WARPS - 1) / am::S_WARPS);
    am::PrefixPartial part{reinterpret_cast<float*>(c->ws + c->cv.part_m), reinterpret_cast<float*>(c->ws + c->cv.part_l),
                           reinterpret_cast<float*>(c->ws + c->cv.part_o), n_parts, (size_t)std::max(c->max_rows, 1) * d.n_q_heads,
                           d.n_kv_heads, sgrid * am::S_WARPS};
    const dim3 ggrid(q_tiles * n_parts, d.n_kv_heads, plan.n_groups);
    if (plan.prefill) {
        launch_k(am::attn_group_kernel<HD, true>, dim3(ggrid), dim3(am::G_THREADS), am::group_smem_bytes<HD>(), st, 
            c->map_prompt_kv, sd, prompt_arena.n_slots, d.n_q_heads, d.n_kv_heads, layer, q, plan.group_row_start, g, scale_log2,
            part, attn, attn_lo, c->err);
        count_launches(1);
        return PC_OK;
    }
    // The two kernels are independent (both read q, each leaves its own records), so outside profiled steps they are issued
    // on two streams -- a fork and a join inside the captured step -- and share the GPU.
    const bool overlap = c->attn_overlap != 0 && c->prof_active_layer < 0;
    cudaStream_t gst = st;
    if (overlap) {
        if (c->side_stream == nullptr) {
            cudaError_t e = cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
            if (e != cudaSuccess) return cuda_fail(e, "side stream of the attention fork");
        }
        cudaEventRecord(c->ev_fork, st);
        cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0);
        gst = c->side_stream;
    }
    // after the QKV post-processing kernel or the QKV projection (both signal their dependents early); not on the side stream
    // of the fork and not after the persistent kernel
    const bool group_dep = !overlap && part_out == nullptr && dependent_launch(c, DEP_GROUP, M);
    launch_k_dep(group_dep, am::attn_group_kernel<HD, false>, dim3(ggrid), dim3(am::G_THREADS), am::group_smem_bytes<HD>(), gst, 
        c->map_prompt_kv, sd, prompt_arena.n_slots, d.n_q_heads, d.n_kv_heads, layer, q, plan.group_row_start, g, scale_log2, part,
        attn, attn_lo, c->err);
    if (overlap) cudaEventRecord(c->ev_join, gst);
    c->mark(st, layer, PC_MARK_GROUP);
    launch_k(am::attn_suffix_kernel<HD>, dim3(sgrid), dim3(am::S_WARPS * 32), am::suffix_smem_bytes<HD>(), st, 
        c->map_suffix_kv, sd, suffix_arena.n_slots, d.n_q_heads, d.n_kv_heads, layer, q, g, scale_log2, part, c->err);
    if (overlap) cudaStreamWaitEvent(st, c->ev_join, 0);
    c->mark(st, layer, PC_MARK_SUFFIX);
    if (part_out != nullptr) {
        *part_out = part;
        count_launches(2);
        return PC_OK;
    }
    if ((long long)M * d.n_q_heads > 8192)
        launch_k(am::attn_merge_kernel<HD, true>, dim3((M * d.n_q_heads + 7) / 8), dim3(256), 0, st, sd, d.n_q_heads, g, part, attn, attn_lo, c->err);
    else
        launch_k(am::attn_merge_kernel<HD, false>, dim3((M * d.n_q_heads + 7) / 8), dim3(256), 0, st, sd, d.n_q_heads, g, part, attn, attn_lo, c->err);
    c->mark(st, layer, PC_MARK_MERGE);
    count_launches(3);
    return PC_OK;
}

// The decoder layers over the rows whose geometry is already in the workspace; leaves the residual stream in ws.h.
// M is the row count grids and GEMM plans are sized for; the live count (<= M) is read from *sd on the device.
template <typename T>
int run_layers(pc_ctx* c, cudaStream_t st, int M, const pc::StepDesc* sd, pc::KvArena prompt_arena, pc::KvArena suffix_arena,
               const AttnPlan& plan) {
    using namespace pc;
    constexpr bool kF32 = std::is_same<T, float>::value;
    const pc_model_desc& d = c->d;
    char* w = c->ws;
    float* h = reinterpret_cast<float*>(w + c->cv.h);
    T* a = reinterpret_cast<T*>(w + c->cv.a);
    float* qkv = reinterpret_cast<float*>(w + c->cv.qkv);
    T* q = reinterpret_cast<T*>(w + c->cv.q);
    T* attn = reinterpret_cast<T*>(w + c->cv.attn);
    T* act = reinterpret_cast<T*>(w + c->cv.act);
    const bool half_gemm = !kF32 && d.half_gemm != 0;      // every GEMM operand in IEEE half
    // QKV post-processing in the QKV GEMM's epilogue; residual add, operand of the gate/up GEMM and the norm's sum of squares
    // in the output projection's epilogue, its 1/rms applied by the gate/up epilogue (gemm_epilogues.cuh)
    // From three row tiles on: below that the two projections need their K split to keep the SMs busy (measured: unsplit they
    // lose more than the two small kernels cost), and a split GEMM's tile does not hold complete sums.
    const bool fused = half_gemm && d.head_dim == 128 && d.d_model % 64 == 0 && c->fused_epilogues != 0 && M >= (c->fused_epilogues == 1 ? 2 * tc::BM + 1 : c->fused_epilogues);
    float* ssq = reinterpret_cast<float*>(w + c->cv.ssq);
    const int m_stride = std::max(std::max(c->max_rows, c->max_prefill), 1);
    T* a_lo = kF32 || half_gemm ? nullptr : reinterpret_cast<T*>(w + c->cv.a_lo);          // rounding remainders (bf16 operands only)
    float2* rope = reinterpret_cast<float2*>(w + c->cv.rope);
    const RowGeom g = geom(c);
    const int half = d.head_dim / 2;
    const float scale = 1.0f / sqrtf((float)d.head_dim);
    float* res_part = reinterpret_cast<float*>(w + c->cv.res_part);
    const Partials none{nullptr, 0, 0, 0};
    Partials pend = none;
    int n_ssq = 0;
    int n_ssq_attn = 0;          // > 0: the previous layer's down projection left half(h * gain) and sums of squares for this layer's attention norm

    launch_k(rope_table_kernel, dim3((M * half + 255) / 256), dim3(256), 0, st, sd, half, (double)d.rope_theta, g.pos, rope);
    launch_k(embed_rmsnorm_kernel<T>, dim3(M), dim3(NORM_THREADS), 0, st, sd, d.d_model, g.token, reinterpret_cast<const T*>(c->embed), c->attn_norm[0],
                                               d.rms_eps, h, a, a_lo, half_gemm ? 1 : 0, c->err);
    count_launches(2);
    PC_CUDA_CHECK_LAUNCH("embed_rmsnorm");
    for (int l = 0; l < d.n_layers; ++l) {
        c->mark(st, l, PC_MARK_LAYER_BEGIN);
        if (l > 0 && n_ssq_attn == 0) {
            launch_k(rmsnorm_kernel<T>, dim3(M), dim3(NORM_THREADS), 0, st, sd, M, d.d_model, h, nullptr, pend, c->attn_norm[l], d.rms_eps, a, a_lo, half_gemm ? 1 : 0, c->err);
            pend = none;
            count_launches(1);
        }
        c->mark(st, l, PC_MARK_NORM_ATTN);
        const float* bias = d.qkv_bias ? c->bqkv[l] : nullptr;
        Partials qkv_parts{qkv, 1, (size_t)M * c->n_qkv(), c->n_qkv()};
        if constexpr (kF32) {
            launch_gemm_simt<T>(st, sd, a, reinterpret_cast<const T*>(c->wqkv[l]), M, c->n_qkv(), d.d_model,
                                EpiStoreF32{qkv, c->n_qkv(), nullptr});
        } else if (fused) {
            const EpiQkvPost epi{d.n_q_heads, d.n_kv_heads, l, bias, d.qk_norm ? c->q_norm[l] : nullptr, d.qk_norm ? c->k_norm[l] : nullptr,
                                 d.rms_eps, rope, g, prompt_arena, suffix_arena, reinterpret_cast<__half*>(q), c->err, ssq, n_ssq_attn, m_stride, d.d_model};
            n_ssq_attn = 0;
            const bool wide_qkv = c->plan_bn[GEMM_QKV] != 0 ? c->plan_bn[GEMM_QKV] == 256 : wide_tiles_fill_the_gpu(c, M, c->n_qkv());
            const int rc = wide_qkv ? gemm_half_bn<256>(c, st, sd, c->map_a, c->m_wqkv[l], M, epi, DEP_QKV)
                                    : gemm_half_bn<128>(c, st, sd, c->map_a, c->m_wqkv[l], M, epi, DEP_QKV);
            if (rc) return rc;
        } else {
            const GemmPlan gp = plan_gemm(c, GEMM_QKV, c->m_wqkv[l], M, true);
            qkv_parts.n = gp.splits;
            if (int rc = gemm_bf16(c, st, sd, c->map_a, half_gemm ? nullptr : &c->map_a_lo, c->m_wqkv[l], M, gp,
                                   tc::EpiPartial{qkv, c->n_qkv(), qkv_parts.stride}, half_gemm, DEP_QKV))
                return rc;
        }
        c->mark(st, l, PC_MARK_QKV);
        const int post_items = M * (d.n_q_heads + 2 * d.n_kv_heads);
        if (!fused) launch_k(qkv_post_kernel<T>, dim3((post_items + ROW_WARPS - 1) / ROW_WARPS), dim3(ROW_WARPS * 32), 0, st, 
            sd, QkvPostArgs<T>{d.n_q_heads, d.n_kv_heads, d.head_dim, l, qkv_parts, bias, d.qk_norm ? c->q_norm[l] : nullptr,
                               d.qk_norm ? c->k_norm[l] : nullptr, d.rms_eps, rope, g, prompt_arena, suffix_arena, q, c->err});
        count_launches(fused ? 1 : 2);
        c->mark(st, l, PC_MARK_POST);
        if constexpr (kF32) {
            c->mark(st, l, PC_MARK_GROUP);
            if (d.head_dim == 128)
                attn_row_simt_kernel<T, 128><<<dim3(M, d.n_kv_heads), 128, 0, st>>>(sd, d.n_q_heads, d.n_kv_heads, l, q, g,
                                                                                   prompt_arena, suffix_arena, scale, attn);
            else
                attn_row_simt_kernel<T, 64><<<dim3(M, d.n_kv_heads), 128, 0, st>>>(sd, d.n_q_heads, d.n_kv_heads, l, q, g,
                                                                                  prompt_arena, suffix_arena, scale, attn);
            c->mark(st, l, PC_MARK_SUFFIX);
            c->mark(st, l, PC_MARK_MERGE);
            count_launches(1);
            launch_gemm_simt<T>(st, sd, attn, reinterpret_cast<const T*>(c->wo[l]), M, d.d_model, c->q_dim(), EpiResidual{h, d.d_model});
        } else {
            int rc = d.head_dim == 128
                         ? attention_bf16<128>(c, st, sd, M, l, plan, prompt_arena, suffix_arena, q, attn)
                         : attention_bf16<64>(c, st, sd, M, l, plan, prompt_arena, suffix_arena, q, attn);
            if (rc) return rc;
            const GemmPlan gp = plan_gemm(c, GEMM_O, c->m_wo[l], M, true);
            if (fused) {
                const bool wide = c->plan_bn[GEMM_O] != 0 ? c->plan_bn[GEMM_O] == 256 : wide_tiles_fill_the_gpu(c, M, d.d_model);
                n_ssq = (d.d_model + (wide ? 256 : 64) - 1) / (wide ? 256 : 64);
                const EpiResNorm epi{h, d.d_model, c->mlp_norm[l], reinterpret_cast<__half*>(a), ssq, m_stride, c->err};
                const int rc2 = wide ? gemm_half_bn<256>(c, st, sd, c->map_attn, c->m_wo[l], M, epi, DEP_O)
                                     : gemm_half_bn<64>(c, st, sd, c->map_attn, c->m_wo[l], M, epi, DEP_O);
                if (rc2) return rc2;
            } else if (gp.splits == 1) {
                if (int rc2 = gemm_bf16(c, st, sd, c->map_attn, half_gemm ? nullptr : &c->map_attn_lo, c->m_wo[l], M, gp,
                                        tc::EpiResidual{h, d.d_model}, half_gemm, DEP_O))
                    return rc2;
            } else {
                pend = Partials{res_part, gp.splits, (size_t)M * d.d_model, d.d_model};
                if (int rc2 = gemm_bf16(c, st, sd, c->map_attn, half_gemm ? nullptr : &c->map_attn_lo, c->m_wo[l], M, gp,
                                        tc::EpiPartial{res_part, d.d_model, pend.stride}, half_gemm, DEP_O))
                    return rc2;
            }
        }
        c->mark(st, l, PC_MARK_O);
        if (!fused) launch_k(rmsnorm_kernel<T>, dim3(M), dim3(NORM_THREADS), 0, st, sd, M, d.d_model, h, nullptr, pend, c->mlp_norm[l], d.rms_eps, a, nullptr, half_gemm ? 1 : 0, c->err);
        pend = none;
        count_launches(fused ? 1 : 2);
        c->mark(st, l, PC_MARK_NORM_MLP);
        if constexpr (kF32) {
            launch_gemm_simt<T>(st, sd, a, reinterpret_cast<const T*>(c->w_gate_up[l]), M, 2 * d.d_ff, d.d_model,
                                EpiSwiGLU<T>{act, d.d_ff});
            c->mark(st, l, PC_MARK_GATE_UP);
            launch_gemm_simt<T>(st, sd, act, reinterpret_cast<const T*>(c->w_down[l]), M, d.d_model, d.d_ff, EpiResidual{h, d.d_model});
        } else if (fused) {
            const EpiSwiGLUNorm epi{reinterpret_cast<__half*>(act), d.d_ff, ssq, n_ssq, m_stride, d.d_model, d.rms_eps, c->err};
            const int rc = plan_gemm(c, GEMM_GATE_UP, c->m_wgu[l], M, false).wide ? gemm_half_bn<256>(c, st, sd, c->map_a, c->m_wgu[l], M, epi, DEP_GATE_UP)
                                                                                  : gemm_half_bn<64>(c, st, sd, c->map_a, c->m_wgu[l], M, epi, DEP_GATE_UP);
            if (rc) return rc;
            c->mark(st, l, PC_MARK_GATE_UP);
            const GemmPlan gp = plan_gemm(c, GEMM_DOWN, c->m_wdown[l], M, true);
            if (gp.splits == 1 && l + 1 < d.n_layers) {
                // complete sums in every tile: the next layer's attention norm moves into this epilogue and the QKV epilogue
                // (the sums of squares of the MLP norm were consumed by the gate/up projection above)
                n_ssq_attn = (d.d_model + (gp.wide ? 256 : 64) - 1) / (gp.wide ? 256 : 64);
                const EpiResNorm epi2{h, d.d_model, c->attn_norm[l + 1], reinterpret_cast<__half*>(a), ssq, m_stride, c->err};
                const int rc2 = gp.wide ? gemm_half_bn<256>(c, st, sd, c->map_act, c->m_wdown[l], M, epi2, DEP_DOWN)
                                        : gemm_half_bn<64>(c, st, sd, c->map_act, c->m_wdown[l], M, epi2, DEP_DOWN);
                if (rc2) return rc2;
            } else if (gp.splits == 1) {
                if (int rc2 = gemm_bf16(c, st, sd, c->map_act, nullptr, c->m_wdown[l], M, gp, tc::EpiResidual{h, d.d_model}, half_gemm, DEP_DOWN)) return rc2;
            } else {
                pend = Partials{res_part, gp.splits, (size_t)M * d.d_model, d.d_model};
                if (int rc2 = gemm_bf16(c, st, sd, c->map_act, nullptr, c->m_wdown[l], M, gp, tc::EpiPartial{res_part, d.d_model, pend.stride}, half_gemm, DEP_DOWN)) return rc2;
            }
        } else {
            if (int rc = gemm_bf16(c, st, sd, c->map_a, nullptr, c->m_wgu[l], M, plan_gemm(c, GEMM_GATE_UP, c->m_wgu[l], M, false), tc::EpiSwiGLU{act, d.d_ff, half_gemm ? 1 : 0, c->err}, half_gemm, DEP_GATE_UP))
                return rc;
            c->mark(st, l, PC_MARK_GATE_UP);
            const GemmPlan gp = plan_gemm(c, GEMM_DOWN, c->m_wdown[l], M, true);
            if (gp.splits == 1) {
                if (int rc = gemm_bf16(c, st, sd, c->map_act, nullptr, c->m_wdown[l], M, gp, tc::EpiResidual{h, d.d_model}, half_gemm, DEP_DOWN)) return rc;
            } else {
                pend = Partials{res_part, gp.splits, (size_t)M * d.d_model, d.d_model};
                if (int rc = gemm_bf16(c, st, sd, c->map_act, nullptr, c->m_wdown[l], M, gp, tc::EpiPartial{res_part, d.d_model, pend.stride}, half_gemm, DEP_DOWN)) return rc;
            }
        }
        count_launches(2);
        c->mark(st, l, PC_MARK_DOWN);
        PC_CUDA_CHECK_LAUNCH("decoder layer");
    }
    c->pend = pend;        // folded into h by the final norm
    return PC_OK;
}

// logits[n, V] = RMSNorm(h[src[r]]; final_norm) * W_lm^T
template <typename T>
int run_lm_head(pc_ctx* c, cudaStream_t st, int n, const pc::StepDesc* sd, const int32_t* src, float* logits) {
    using namespace pc;
    const pc_model_desc& d = c->d;
    float* h = reinterpret_cast<float*>(c->ws + c->cv.h);
    T* a = reinterpret_cast<T*>(c->ws + c->cv.a);
    const bool half_gemm = !std::is_same<T, float>::value && d.half_gemm != 0;
    T* a_lo = std::is_same<T, float>::value || half_gemm ? nullptr : reinterpret_cast<T*>(c->ws + c->cv.a_lo);
    c->mark(st, -1, PC_MARK_LM_BEGIN);
    launch_k(rmsnorm_kernel<T>, dim3(n), dim3(NORM_THREADS), 0, st, sd, n, d.d_model, h, src, c->pend, c->final_norm, d.rms_eps, a, a_lo, half_gemm ? 1 : 0, c->err);
    c->pend = pc::Partials{nullptr, 0, 0, 0};
    if constexpr (std::is_same<T, float>::value) {
        const T* wlm = reinterpret_cast<const T*>(d.tied_embed ? c->embed : c->lm_head);
        launch_gemm_simt<T>(st, sd, a, wlm, n, d.vocab, d.d_model, EpiStoreF32{logits, d.vocab, nullptr});
    } else {
        if (int rc = gemm_bf16(c, st, sd, c->map_a, half_gemm ? nullptr : &c->map_a_lo, c->m_lm, n, plan_gemm(c, GEMM_LM_HEAD, c->m_lm, n, false),
                               tc::EpiStoreF32{logits, d.vocab, nullptr}, half_gemm, DEP_LM_HEAD))
            return rc;
    }
    count_launches(2);
    c->mark(st, -1, PC_MARK_LM_HEAD);
    PC_CUDA_CHECK_LAUNCH("lm head");
    return PC_OK;
}

// Final norm, LM head and the Gumbel-max draw in the GEMM's epilogue (lm_sample.cuh): the step's logits are not stored.
int run_lm_head_sample(pc_ctx* c, cudaStream_t st, int n, const pc::StepDesc* sd, const pc::RowKeys& keys, const pc::DecodeArgsDev* da) {
    using namespace pc;
    using T = __nv_bfloat16;
    const pc_model_desc& d = c->d;
    float* h = reinterpret_cast<float*>(c->ws + c->cv.h);
    T* a = reinterpret_cast<T*>(c->ws + c->cv.a);
    const bool half_gemm = d.half_gemm != 0;
    T* a_lo = half_gemm ? nullptr : reinterpret_cast<T*>(c->ws + c->cv.a_lo);
    c->mark(st, -1, PC_MARK_LM_BEGIN);
    launch_k(rmsnorm_kernel<T>, dim3(n), dim3(NORM_THREADS), 0, st, sd, n, d.d_model, h, nullptr, c->pend, c->final_norm, d.rms_eps, a, a_lo,
             half_gemm ? 1 : 0, c->err);
    c->pend = pc::Partials{nullptr, 0, 0, 0};
    const GemmPlan gp = plan_gemm(c, GEMM_LM_HEAD, c->m_lm, n, false);
    Top2Rec* rec = reinterpret_cast<Top2Rec*>(c->ws + c->cv.sample_tiles);
    const int m_stride = std::max(c->max_rows, 1);
    if (int rc = gemm_bf16(c, st, sd, c->map_a, half_gemm ? nullptr : &c->map_a_lo, c->m_lm, n, gp,
                           EpiSample{rec, m_stride, keys.key_prompt, keys.rollout, keys.step_key, keys.sample_bound, da}, half_gemm, DEP_LM_HEAD))
        return rc;
    c->mark(st, -1, PC_MARK_LM_HEAD);
    const int bn = gp.wide ? 256 : 64;
    launch_k(sample_tiles_reduce_kernel, dim3(n), dim3(TILES_REDUCE_THREADS), 0, st, sd, 2 * ((d.vocab + bn - 1) / bn), rec, m_stride, keys.out_index, da);
    count_launches(3);
    c->mark(st, -1, PC_MARK_SAMPLE);
    PC_CUDA_CHECK_LAUNCH("lm head with sampler");
    return PC_OK;
}

int check_ready(const pc_ctx* c) {
    if (c == nullptr) return PC_ERR_INVALID_ARG;
    if (c->ws == nullptr) return PC_ERR_NO_WORKSPACE;
    return PC_OK;
}

}  // namespace

extern "C" {

const char* pc_status_string(int status) {
    switch (status) {
        case PC_OK: return "ok";
        case PC_ERR_INVALID_ARG: return "invalid argument";
        case PC_ERR_SHAPE: return "unsupported model shape";
        case PC_ERR_ALIGNMENT: return "misaligned pointer";
        case PC_ERR_CAPACITY: return "workspace capacity exceeded";
        case PC_ERR_UNSUPPORTED: return "unsupported";
        case PC_ERR_CUDA: return "CUDA error";
        case PC_ERR_NO_WORKSPACE: return "workspace not set";
        default: return "unknown status";
    }
}

const char* pc_last_cuda_error(void) { return g_cuda_error.c_str(); }

uint64_t pc_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int pc_set_prompt_keys(pc_ctx* ctx, const int32_t* prompt_key) {
    if (ctx == nullptr) return PC_ERR_INVALID_ARG;
    ctx->prompt_key = prompt_key;
    return PC_OK;
}

int pc_set_gemm_plan(pc_ctx* ctx, const char* spec) {
    if (ctx == nullptr) return PC_ERR_INVALID_ARG;
    int bn[5] = {0, 0, 0, 0, 0}, sp[5] = {0, 0, 0, 0, 0};
    static const char* const names[5] = {"qkv", "o", "gu", "dn", "lm"};
    const char* p = spec ? spec : "";
    while (*p) {
        int kind = -1;
        size_t len = 0;
        for (int k = 0; k < 5; ++k) {
            const size_t n = std::strlen(names[k]);
            if (std::strncmp(p, names[k], n) == 0 && p[n] == '=') { kind = k; len = n + 1; }
        }
        if (kind < 0) return PC_ERR_INVALID_ARG;
        int w = 0, s = 0, used = 0;
        if (std::sscanf(p + len, "%dx%d%n", &w, &s, &used) != 2) return PC_ERR_INVALID_ARG;
        if ((w != 64 && w != 128 && w != 256) || s < 1 || s > kMaxSplits) return PC_ERR_INVALID_ARG;      // 128: fused QKV epilogue only
        bn[kind] = w; sp[kind] = s;
        p += len + used;
        if (*p == ',') ++p;
        else if (*p) return PC_ERR_INVALID_ARG;
    }
    for (int k = 0; k < 5; ++k) { ctx->plan_bn[k] = bn[k]; ctx->plan_splits[k] = sp[k]; }
    ctx->drop_graphs();          // captured steps carry the old choice
    return PC_OK;
}

int pc_set_fused_epilogues(pc_ctx* ctx, int on) {
    if (ctx == nullptr || on < 0) return PC_ERR_INVALID_ARG;
    if (on != ctx->fused_epilogues) ctx->drop_graphs();
    ctx->fused_epilogues = on;
    return PC_OK;
}

int pc_set_fused_sampler(pc_ctx* ctx, int on) {
    if (ctx == nullptr || (on != 0 && on != 1)) return PC_ERR_INVALID_ARG;
    if (on != ctx->fused_sampler) ctx->drop_graphs();
    ctx->fused_sampler = on;
    return PC_OK;
}

int pc_set_dependent_launch(pc_ctx* ctx, int mask) {
    if (ctx == nullptr || mask < 0 || mask > 63) return PC_ERR_INVALID_ARG;
    if (mask != ctx->dep_launch) ctx->drop_graphs();
    ctx->dep_launch = mask;
    return PC_OK;
}

int pc_set_attention_overlap(pc_ctx* ctx, int on) {
    if (ctx == nullptr || (on != 0 && on != 1)) return PC_ERR_INVALID_ARG;
    if (on != ctx->attn_overlap) ctx->drop_graphs();
    ctx->attn_overlap = on;
    return PC_OK;
}

int pc_set_decode_mode(pc_ctx* ctx, int mode) {
    if (ctx == nullptr || (mode != 0 && mode != 1)) return PC_ERR_INVALID_ARG;
    if (mode != ctx->decode_mode) ctx->drop_graphs();          // captured steps carry the old choice
    ctx->decode_mode = mode;
    return PC_OK;
}

int pc_set_chain_trace(pc_ctx* ctx, int64_t* trace, size_t n_words) {
    if (ctx == nullptr) return PC_ERR_INVALID_ARG;
    if (trace != nullptr && n_words < pc_chain_trace_words(ctx)) return PC_ERR_CAPACITY;
    ctx->chain_trace = reinterpret_cast<long long*>(trace);
    ctx->drop_graphs();
    return PC_OK;
}

size_t pc_chain_trace_words(const pc_ctx* ctx) {
    if (ctx == nullptr) return 0;
    return (size_t)(ctx->d.n_layers + 1) * pc::chain::MAX_PHASES * pc::chain::TRACE_CTAS * pc::chain::TRACE_EVENTS;
}

uint64_t pc_capture_count(const pc_ctx* ctx) { return ctx ? ctx->captures : 0; }

int pc_selftest_wait_timeout(void* stream, uint32_t spin_limit, int32_t* dev_error_flag) {
    if (dev_error_flag == nullptr || spin_limit == 0 || spin_limit > (1u << 20)) return PC_ERR_INVALID_ARG;
    pc::tc::wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(spin_limit, dev_error_flag);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("wait self-test");
    return PC_OK;
}

int pc_set_index_bounds(pc_ctx* ctx, int n_prompts, int64_t n_tokens) {
    if (ctx == nullptr || n_prompts < 0 || n_tokens < 0) return PC_ERR_INVALID_ARG;
    ctx->n_prompts_hint = n_prompts;
    ctx->n_tokens_hint = n_tokens;
    return PC_OK;
}

int pc_set_logprob_buffer(pc_ctx* ctx, float* logprobs) {
    if (ctx == nullptr) return PC_ERR_INVALID_ARG;
    ctx->logprobs = logprobs;
    return PC_OK;
}

int pc_token_logprob(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row, float temperature,
                     const int32_t* tokens, const int64_t* tok_index, float* out_logprob, const int64_t* out_index) {
    if (n_rows < 0 || vocab <= 0 || !(temperature > 0.f)) return PC_ERR_INVALID_ARG;
    if (n_rows == 0) return PC_OK;
    if (logits == nullptr || tokens == nullptr || out_logprob == nullptr) return PC_ERR_INVALID_ARG;
    launch_k(pc::token_logprob_kernel, dim3(n_rows), dim3(256), 0, static_cast<cudaStream_t>(stream), nullptr, vocab, logits, logits_row, temperature, tokens,
                                                                                   tok_index, 0, out_logprob, out_index, 0, nullptr);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("token_logprob");
    return PC_OK;
}

int pc_profile_step(pc_ctx* ctx, int layer, void* const* events, int n_events) {
    if (ctx == nullptr || layer < 0 || layer >= ctx->d.n_layers || events == nullptr || n_events != PC_PROFILE_MARKS) return PC_ERR_INVALID_ARG;
    for (int i = 0; i < PC_PROFILE_MARKS; ++i) ctx->prof_ev[i] = static_cast<cudaEvent_t>(events[i]);
    ctx->prof_layer = layer;
    return PC_OK;
}

int pc_create(const pc_model_desc* desc, const pc_weights* wts, pc_ctx** out) {
    if (desc == nullptr || wts == nullptr || out == nullptr) return PC_ERR_INVALID_ARG;
    *out = nullptr;
    const pc_model_desc& d = *desc;
    if (d.dtype != PC_DTYPE_F32 && d.dtype != PC_DTYPE_BF16) return PC_ERR_INVALID_ARG;
    if (d.half_gemm != 0 && (d.half_gemm != 1 || d.dtype != PC_DTYPE_BF16)) return PC_ERR_INVALID_ARG;
    if (d.n_layers <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.d_ff <= 0 || d.vocab <= 0 ||
        !(d.rms_eps >= 0.f) || !(d.rope_theta > 0.f))
        return PC_ERR_INVALID_ARG;
    if (d.head_dim != 64 && d.head_dim != 128) return PC_ERR_SHAPE;
    if (d.n_q_heads % d.n_kv_heads != 0 || d.n_q_heads / d.n_kv_heads > pc::ATTN_MAX_REP) return PC_ERR_SHAPE;
    if (d.d_model % 8 != 0 || d.d_ff % 8 != 0 || d.d_model > 8192) return PC_ERR_SHAPE;
    if (d.dtype == PC_DTYPE_BF16 && (d.d_model % 64 != 0 || d.d_ff % 64 != 0)) return PC_ERR_SHAPE;
    if (wts->embed == nullptr || wts->final_norm == nullptr || ((!d.tied_embed || d.half_gemm) && wts->lm_head == nullptr)) return PC_ERR_INVALID_ARG;
    if (wts->attn_norm == nullptr || wts->wqkv == nullptr || wts->wo == nullptr || wts->mlp_norm == nullptr ||
        wts->w_gate_up == nullptr || wts->w_down == nullptr)
        return PC_ERR_INVALID_ARG;
    if (d.qkv_bias && wts->bqkv == nullptr) return PC_ERR_INVALID_ARG;
    if (d.qk_norm && (wts->q_norm == nullptr || wts->k_norm == nullptr)) return PC_ERR_INVALID_ARG;
    pc_ctx* c = new (std::nothrow) pc_ctx();
    if (c == nullptr) return PC_ERR_INVALID_ARG;
    c->d = d;
    c->embed = wts->embed;
    c->lm_head = wts->lm_head;
    c->final_norm = wts->final_norm;
    if (!aligned(c->embed, 16) || (c->lm_head && !aligned(c->lm_head, 16))) { delete c; return PC_ERR_ALIGNMENT; }
    for (int l = 0; l < d.n_layers; ++l) {
        const void* mats[4] = {wts->wqkv[l], wts->wo[l], wts->w_gate_up[l], wts->w_down[l]};
        for (const void* m : mats) {
            if (m == nullptr) { delete c; return PC_ERR_INVALID_ARG; }
            if (!aligned(m, 16)) { delete c; return PC_ERR_ALIGNMENT; }
        }
        if (wts->attn_norm[l] == nullptr || wts->mlp_norm[l] == nullptr) { delete c; return PC_ERR_INVALID_ARG; }
        if (d.qkv_bias && wts->bqkv[l] == nullptr) { delete c; return PC_ERR_INVALID_ARG; }
        if (d.qk_norm && (wts->q_norm[l] == nullptr || wts->k_norm[l] == nullptr)) { delete c; return PC_ERR_INVALID_ARG; }
        c->attn_norm.push_back(wts->attn_norm[l]);
        c->mlp_norm.push_back(wts->mlp_norm[l]);
        c->bqkv.push_back(d.qkv_bias ? wts->bqkv[l] : nullptr);
        c->q_norm.push_back(d.qk_norm ? wts->q_norm[l] : nullptr);
        c->k_norm.push_back(d.qk_norm ? wts->k_norm[l] : nullptr);
        c->wqkv.push_back(wts->wqkv[l]);
        c->wo.push_back(wts->wo[l]);
        c->w_gate_up.push_back(wts->w_gate_up[l]);
        c->w_down.push_back(wts->w_down[l]);
    }
    if (d.dtype == PC_DTYPE_BF16) {
        if (c->q_dim() % 64 != 0) { delete c; return PC_ERR_SHAPE; }
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
            delete c;
            return cuda_fail(cudaGetLastError(), "no CUDA device for a bf16 model");
        }
        c->num_sms = sms;
        bool ok = true;
        c->m_wqkv.resize(d.n_layers); c->m_wo.resize(d.n_layers); c->m_wgu.resize(d.n_layers); c->m_wdown.resize(d.n_layers);
        for (int l = 0; l < d.n_layers && ok; ++l) {
            ok = make_wmap(&c->m_wqkv[l], c->wqkv[l], c->n_qkv(), d.d_model) && make_wmap(&c->m_wo[l], c->wo[l], d.d_model, c->q_dim()) &&
                 make_wmap(&c->m_wgu[l], c->w_gate_up[l], 2 * d.d_ff, d.d_model) && make_wmap(&c->m_wdown[l], c->w_down[l], d.d_model, d.d_ff);
        }
        ok = ok && make_wmap(&c->m_lm, d.tied_embed && !d.half_gemm ? c->embed : c->lm_head, d.vocab, d.d_model);
        if (!ok) {
            delete c;
            g_cuda_error = "cuTensorMapEncodeTiled failed for a weight matrix";
            return PC_ERR_CUDA;
        }
    }
    *out = c;
    return PC_OK;
}

void pc_destroy(pc_ctx* ctx) { delete ctx; }

int pc_workspace_bytes(const pc_ctx* ctx, int max_rows, int max_prefill_tokens, size_t* out_bytes) {
    if (ctx == nullptr || out_bytes == nullptr || max_rows < 0 || max_prefill_tokens < 0) return PC_ERR_INVALID_ARG;
    *out_bytes = carve(ctx, max_rows, max_prefill_tokens).total;
    return PC_OK;
}

int pc_set_workspace(pc_ctx* ctx, void* dev_ws, size_t bytes, int max_rows, int max_prefill_tokens, int32_t* dev_error_flag) {
    if (ctx == nullptr || dev_ws == nullptr || dev_error_flag == nullptr || max_rows < 0 || max_prefill_tokens < 0)
        return PC_ERR_INVALID_ARG;
    if (!aligned(dev_ws, 256) || !aligned(dev_error_flag, 4)) return PC_ERR_ALIGNMENT;
    const Carve cv = carve(ctx, max_rows, max_prefill_tokens);
    if (bytes < cv.total) return PC_ERR_CAPACITY;
    ctx->ws = static_cast<char*>(dev_ws);
    ctx->ws_bytes = bytes;
    ctx->max_rows = max_rows;
    ctx->max_prefill = max_prefill_tokens;
    ctx->err = dev_error_flag;
    ctx->cv = cv;
    ctx->split_capacity_rows = std::min<size_t>((size_t)std::max(max_rows, max_prefill_tokens), kSplitMaxRows) * kMaxSplits;
    ctx->drop_graphs();
    if (ctx->d.dtype == PC_DTYPE_BF16) {
        cudaError_t ce = configure_kernels();
        if (ce != cudaSuccess) { ctx->ws = nullptr; return cuda_fail(ce, "kernel attributes"); }
        const uint64_t cap = (uint64_t)std::max(std::max(max_rows, max_prefill_tokens), 1);
        char* w = ctx->ws;
        if (!pc::make_bf16_map(&ctx->map_a, w + cv.a, cap, ctx->d.d_model, 128) ||
            !pc::make_bf16_map(&ctx->map_attn, w + cv.attn, cap, ctx->q_dim(), 128) ||
            !pc::make_bf16_map(&ctx->map_act, w + cv.act, cap, ctx->d.d_ff, 128) ||
            !pc::make_bf16_map(&ctx->map_a_lo, w + cv.a_lo, cap, ctx->d.d_model, 128) ||
            !pc::make_bf16_map(&ctx->map_attn_lo, w + cv.attn_lo, cap, ctx->q_dim(), 128)) {
            ctx->ws = nullptr;
            g_cuda_error = "cuTensorMapEncodeTiled failed for an activation buffer";
            return PC_ERR_CUDA;
        }
        ctx->chain_ready = false;
        if (ctx->d.half_gemm) {
            // constants of the persistent decode kernel: per-layer weight descriptors and gain / bias pointers
            const pc_model_desc& d = ctx->d;
            std::vector<pc::chain::LayerTab> tabs((size_t)d.n_layers);
            auto put3 = [](CUtensorMap* dst, const WMap& m) { dst[0] = m.narrow; dst[1] = m.mid; dst[2] = m.wide; };
            for (int l = 0; l < d.n_layers; ++l) {
                pc::chain::LayerTab& t = tabs[(size_t)l];
                std::memset(&t, 0, sizeof(t));
                put3(t.wqkv, ctx->m_wqkv[l]); put3(t.wo, ctx->m_wo[l]); put3(t.wgu, ctx->m_wgu[l]); put3(t.wdown, ctx->m_wdown[l]);
                t.attn_norm = ctx->attn_norm[l]; t.mlp_norm = ctx->mlp_norm[l];
                t.bqkv = d.qkv_bias ? ctx->bqkv[l] : nullptr;
                t.q_norm = d.qk_norm ? ctx->q_norm[l] : nullptr;
                t.k_norm = d.qk_norm ? ctx->k_norm[l] : nullptr;
            }
            pc::chain::GlobalTab gt;
            std::memset(&gt, 0, sizeof(gt));
            gt.a = ctx->map_a; gt.attn = ctx->map_attn; gt.act = ctx->map_act;
            put3(gt.lm, ctx->m_lm);
            gt.final_norm = ctx->final_norm;
            ce = cudaMemcpy(w + cv.chain_layers, tabs.data(), tabs.size() * sizeof(pc::chain::LayerTab), cudaMemcpyHostToDevice);
            if (ce == cudaSuccess) ce = cudaMemcpy(w + cv.chain_glob, &gt, sizeof(gt), cudaMemcpyHostToDevice);
            if (ce == cudaSuccess)
                ce = cudaFuncSetAttribute(pc::chain::decode_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, pc::chain::SMEM_BYTES);
            if (ce != cudaSuccess) { ctx->ws = nullptr; return cuda_fail(ce, "tables of the persistent decode kernel"); }
            ctx->chain_ready = true;
        }
    }
    return PC_OK;
}

int pc_prefill_shared(pc_ctx* ctx, void* stream, int n_prompts, const int32_t* prompt_tokens, const int32_t* prompt_offsets,
                      int total_tokens, int max_prompt_len, void* prompt_kv, int64_t prompt_slots,
                      const int64_t* prompt_kv_start, float* last_logits) {
    if (int rc = check_ready(ctx)) return rc;
    if (n_prompts < 0 || total_tokens < 0 || max_prompt_len < 0 || prompt_slots < 0) return PC_ERR_INVALID_ARG;
    if (n_prompts == 0 || total_tokens == 0) return PC_OK;
    if (prompt_tokens == nullptr || prompt_offsets == nullptr || prompt_kv == nullptr || prompt_kv_start == nullptr ||
        last_logits == nullptr)
        return PC_ERR_INVALID_ARG;
    if (!aligned(prompt_kv, 16) || !aligned(last_logits, 16)) return PC_ERR_ALIGNMENT;
    if (total_tokens > ctx->max_prefill || n_prompts > total_tokens || max_prompt_len > total_tokens) return PC_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const pc::RowGeom g = geom(ctx);
    int32_t* last_row = reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.last_row);
    pc::StepDesc* sd = reinterpret_cast<pc::StepDesc*>(ctx->ws + ctx->cv.step_desc);
    pc::set_step_desc<<<1, pc::STEP_DESC_THREADS, 0, st>>>(sd, total_tokens, n_prompts, max_prompt_len, g.max_slen, nullptr, 0);
    launch_k(pc::prep_prefill_rows, dim3(n_prompts), dim3(256), 0, st, n_prompts, prompt_tokens, prompt_offsets, prompt_kv_start, prompt_slots,
                                                     ctx->d.vocab, g, last_row, ctx->err);
    count_launches(2);
    PC_CUDA_CHECK_LAUNCH("prep_prefill_rows");
    const pc::KvArena pa{prompt_kv, prompt_slots}, sa{prompt_kv, prompt_slots};
    const AttnPlan plan{true, n_prompts, prompt_offsets, max_prompt_len};
    int rc = PC_OK;
    if (ctx->d.dtype == PC_DTYPE_F32) {
        rc = run_layers<float>(ctx, st, total_tokens, sd, pa, sa, plan);
    } else {
        rc = arena_maps(ctx, prompt_kv, prompt_slots, nullptr, 0);
        if (rc == PC_OK) rc = run_layers<__nv_bfloat16>(ctx, st, total_tokens, sd, pa, sa, plan);
    }
    if (rc) return rc;
    // only the last position of every prompt goes through the LM head: its row count is known on the host
    return ctx->d.dtype == PC_DTYPE_F32 ? run_lm_head<float>(ctx, st, n_prompts, nullptr, last_row, last_logits)
                                        : run_lm_head<__nv_bfloat16>(ctx, st, n_prompts, nullptr, last_row, last_logits);
}

}  // extern "C"

namespace {

// Everything a decode step needs besides the step descriptor; constant over a stage.
struct DecodeArgs {
    const int32_t* row_prompt; const int32_t* row_rollout; const int32_t* row_step; const int64_t* row_kv_start;
    int32_t* tokens; const int64_t* row_tok_index; const int32_t* group_row_start; const int32_t* prompt_len;
    const void* prompt_kv; int64_t prompt_slots; const int64_t* prompt_kv_start; void* suffix_kv; int64_t suffix_slots;
    float temperature; uint64_t seed; int sample;
    float* logprobs;      // optional: behaviour log-probability of every sampled token (pc_set_logprob_buffer)
    const int32_t* prompt_key;   // optional: sampling-key id of every prompt (pc_set_prompt_keys)
};
// Zero-filled first (padding included) so that two equal argument sets compare equal byte by byte.
DecodeArgs make_decode_args(const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step, const int64_t* row_kv_start,
                            int32_t* tokens, const int64_t* row_tok_index, const int32_t* group_row_start, const int32_t* prompt_len,
                            const void* prompt_kv, int64_t prompt_slots, const int64_t* prompt_kv_start, void* suffix_kv,
                            int64_t suffix_slots, const pc_sample_params* sample) {
    DecodeArgs a;
    std::memset(&a, 0, sizeof(a));
    a.row_prompt = row_prompt; a.row_rollout = row_rollout; a.row_step = row_step; a.row_kv_start = row_kv_start;
    a.tokens = tokens; a.row_tok_index = row_tok_index; a.group_row_start = group_row_start; a.prompt_len = prompt_len;
    a.prompt_kv = prompt_kv; a.prompt_slots = prompt_slots; a.prompt_kv_start = prompt_kv_start; a.suffix_kv = suffix_kv;
    a.suffix_slots = suffix_slots;
    a.temperature = sample ? sample->temperature : 1.f;
    a.seed = sample ? sample->seed : 0;
    a.sample = sample != nullptr;
    a.logprobs = nullptr;
    a.prompt_key = nullptr;
    return a;
}

pc::RowKeys row_keys(const pc_ctx* c) {
    char* w = c->ws;
    return pc::RowKeys{reinterpret_cast<int32_t*>(w + c->cv.key_prompt), reinterpret_cast<int32_t*>(w + c->cv.key_rollout),
                       reinterpret_cast<int32_t*>(w + c->cv.key_step), reinterpret_cast<int64_t*>(w + c->cv.out_index),
                       reinterpret_cast<int32_t*>(w + c->cv.group_start), reinterpret_cast<int32_t*>(w + c->cv.sample_bound)};
}

// Upper bounds of a step's group geometry, rounded up to classes so that steps of similar shape share a captured graph
// and a step-by-step call picks the same attention plan as a captured one: the number of groups to the next power of
// two, the largest group to the most rows that need the same number of query tiles (neither beyond the row bound).
void canonical_group_bounds(const pc_ctx* c, int n_groups, int max_group_rows, int row_bound, int* groups_bound, int* group_rows_bound) {
    int gb = 1;
    while (gb < n_groups) gb <<= 1;
    *groups_bound = std::min(gb, std::max(row_bound, 1));
    const int n_rep = c->d.n_q_heads / c->d.n_kv_heads;
    const int q_tiles = (std::max(max_group_rows, 1) * n_rep + pc::am::G_QROWS - 1) / pc::am::G_QROWS;
    *group_rows_bound = std::min(q_tiles * pc::am::G_QROWS / n_rep, std::max(row_bound, 1));
}

// Rewrites the device-resident argument block (stream-ordered: work already queued keeps the values it was issued with).
int upload_decode_args(pc_ctx* ctx, cudaStream_t st, const DecodeArgs& a, const pc_step_desc* steps_dev) {
    pc::DecodeArgsDev d;
    std::memset(&d, 0, sizeof(d));
    d.steps = reinterpret_cast<const pc::StepDesc*>(steps_dev);
    d.row_prompt = a.row_prompt; d.row_rollout = a.row_rollout; d.row_step = a.row_step; d.row_kv_start = a.row_kv_start;
    d.tokens = a.tokens; d.row_tok_index = a.row_tok_index; d.group_row_start = a.group_row_start; d.prompt_len = a.prompt_len;
    d.prompt_kv_start = a.prompt_kv_start; d.logprobs = a.logprobs; d.prompt_key = a.prompt_key;
    d.temperature = a.temperature;
    d.k0 = (uint32_t)(a.seed & 0xffffffffu); d.k1 = (uint32_t)(a.seed >> 32);
    d.n_prompts = ctx->n_prompts_hint; d.n_tokens = ctx->n_tokens_hint;
    const cudaError_t e = cudaMemcpyAsync(ctx->ws + ctx->cv.dargs, &d, sizeof(d), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "decode argument block");
    return PC_OK;
}

int check_decode_args(const pc_ctx* ctx, const DecodeArgs& a) {
    if (a.row_prompt == nullptr || a.row_rollout == nullptr || a.row_step == nullptr || a.row_kv_start == nullptr ||
        a.tokens == nullptr || a.row_tok_index == nullptr || a.group_row_start == nullptr || a.prompt_len == nullptr ||
        a.prompt_kv == nullptr || a.prompt_kv_start == nullptr || a.suffix_kv == nullptr)
        return PC_ERR_INVALID_ARG;
    if (a.prompt_slots < 0 || a.suffix_slots < 0) return PC_ERR_INVALID_ARG;
    if (a.sample && !(a.temperature > 0.f)) return PC_ERR_INVALID_ARG;
    if (!aligned(a.prompt_kv, 16) || !aligned(a.suffix_kv, 16)) return PC_ERR_ALIGNMENT;
    (void)ctx;
    return PC_OK;
}

// One segment of the persistent decode kernel (decode_chain.cuh) over the rows described by *sd.
int launch_chain(pc_ctx* c, cudaStream_t st, int M, const pc::StepDesc* sd, int seg, pc::KvArena prompt_arena, pc::KvArena suffix_arena,
                 const pc::am::PrefixPartial* part, float* logits) {
    using namespace pc;
    const pc_model_desc& d = c->d;
    char* w = c->ws;
    chain::ChainParams p;
    std::memset(&p, 0, sizeof(p));
    p.sd = sd; p.M = M; p.seg = seg; p.with_merge = part != nullptr ? 1 : 0;
    p.n_layers = d.n_layers; p.d_model = d.d_model; p.n_qkv = c->n_qkv(); p.q_dim = c->q_dim(); p.d_ff = d.d_ff; p.vocab = d.vocab;
    p.Hq = d.n_q_heads; p.Hkv = d.n_kv_heads; p.hd = d.head_dim; p.eps = d.rms_eps;
    const WMap* maps[5] = {&c->m_wqkv[0], &c->m_wo[0], &c->m_wgu[0], &c->m_wdown[0], &c->m_lm};
    const bool may_split[5] = {true, true, false, true, false};
    int bn_max = 64;
    for (int k = 0; k < 5; ++k) {
        const GemmPlan gp = plan_gemm(c, (GemmKind)k, *maps[k], M, may_split[k]);
        p.bn[k] = gp.wide ? 256 : 64;
        p.splits[k] = gp.splits;
        const bool used = k == GEMM_LM_HEAD ? seg == d.n_layers - 1 : (k == GEMM_QKV ? seg != d.n_layers - 1 : seg >= 0);
        if (used) bn_max = std::max(bn_max, p.bn[k]);
    }
    p.slot_bytes = chain::A_BYTES + bn_max * pc::tc::BK * 2;
    p.slots = std::min(chain::MAX_SLOTS, chain::RING_BYTES / p.slot_bytes);
    auto pick = [](const WMap& m, int bn) -> const CUtensorMap& { return bn == 256 ? m.wide : (bn == 128 ? m.mid : m.narrow); };
    const int l_here = seg < 0 ? 0 : seg;
    p.maps[chain::MAP_A] = c->map_a; p.maps[chain::MAP_ATTN] = c->map_attn; p.maps[chain::MAP_ACT] = c->map_act;
    p.maps[chain::MAP_WO] = pick(c->m_wo[l_here], p.bn[GEMM_O]);
    p.maps[chain::MAP_WGU] = pick(c->m_wgu[l_here], p.bn[GEMM_GATE_UP]);
    p.maps[chain::MAP_WDOWN] = pick(c->m_wdown[l_here], p.bn[GEMM_DOWN]);
    p.maps[chain::MAP_WNEXT] = seg == d.n_layers - 1 ? pick(c->m_lm, p.bn[GEMM_LM_HEAD]) : pick(c->m_wqkv[seg + 1], p.bn[GEMM_QKV]);
    p.layers = reinterpret_cast<const chain::LayerTab*>(w + c->cv.chain_layers);
    p.glob = reinterpret_cast<const chain::GlobalTab*>(w + c->cv.chain_glob);
    p.embed = c->embed;
    p.h = reinterpret_cast<float*>(w + c->cv.h);
    p.a = reinterpret_cast<__nv_bfloat16*>(w + c->cv.a);
    p.qkv = reinterpret_cast<float*>(w + c->cv.qkv);
    p.res_part = reinterpret_cast<float*>(w + c->cv.res_part);
    p.q = reinterpret_cast<__nv_bfloat16*>(w + c->cv.q);
    p.attn = reinterpret_cast<__nv_bfloat16*>(w + c->cv.attn);
    p.act = reinterpret_cast<__nv_bfloat16*>(w + c->cv.act);
    p.logits = logits;
    p.rope = reinterpret_cast<const float2*>(w + c->cv.rope);
    p.g = geom(c);
    p.prompt_arena = prompt_arena; p.suffix_arena = suffix_arena;
    if (part != nullptr) p.part = *part;
    p.bar = reinterpret_cast<int32_t*>(w + c->cv.chain_bar);
    p.err = c->err;
    p.trace = c->chain_trace;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)c->num_sms); cfg.blockDim = dim3(chain::THREADS); cfg.dynamicSmemBytes = chain::SMEM_BYTES; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;       // every CTA must be resident: they wait for one another
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, chain::decode_chain_kernel, p);
    if (e != cudaSuccess) return cuda_fail(e, "persistent decode kernel");
    count_launches(1);
    return PC_OK;
}

// The decoder layers and the LM head of a decode step with the persistent kernel between the attention calls.
int run_decode_chained(pc_ctx* c, cudaStream_t st, int M, const pc::StepDesc* sd, pc::KvArena prompt_arena, pc::KvArena suffix_arena,
                       const AttnPlan& plan, float* logits) {
    using namespace pc;
    const pc_model_desc& d = c->d;
    char* w = c->ws;
    const RowGeom g = geom(c);
    const int half = d.head_dim / 2;
    launch_k(rope_table_kernel, dim3((M * half + 255) / 256), dim3(256), 0, st, sd, half, (double)d.rope_theta, g.pos, reinterpret_cast<float2*>(w + c->cv.rope));
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("rope table");
    if (int rc = launch_chain(c, st, M, sd, -1, prompt_arena, suffix_arena, nullptr, logits)) return rc;
    const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(w + c->cv.q);
    __nv_bfloat16* attn = reinterpret_cast<__nv_bfloat16*>(w + c->cv.attn);
    for (int l = 0; l < d.n_layers; ++l) {
        am::PrefixPartial part;
        int rc = d.head_dim == 128 ? attention_bf16<128>(c, st, sd, M, l, plan, prompt_arena, suffix_arena, q, attn, &part)
                                   : attention_bf16<64>(c, st, sd, M, l, plan, prompt_arena, suffix_arena, q, attn, &part);
        if (rc) return rc;
        if ((rc = launch_chain(c, st, M, sd, l, prompt_arena, suffix_arena, &part, logits))) return rc;
    }
    PC_CUDA_CHECK_LAUNCH("chained decode step");
    return PC_OK;
}

// The kernels of one decode step.  Grids and GEMM plans are sized for (m_bound rows, groups_bound groups of at most
// group_rows_bound rows); the live counts and the offsets into the caller's row arrays are in the step descriptor.
int decode_launches(pc_ctx* ctx, cudaStream_t st, int m_bound, int groups_bound, int group_rows_bound, const DecodeArgs& a,
                    float* logits_out) {
    const pc::RowGeom g = geom(ctx);
    const pc::RowKeys keys = row_keys(ctx);
    const pc::StepDesc* sd = reinterpret_cast<const pc::StepDesc*>(ctx->ws + ctx->cv.step_desc);
    const pc::DecodeArgsDev* da = reinterpret_cast<const pc::DecodeArgsDev*>(ctx->ws + ctx->cv.dargs);
    // a profiling request is served by the first step issued outside a capture (a captured step never carries the events)
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaStreamIsCapturing(st, &cap);
    ctx->prof_active_layer = -1;
    if (cap == cudaStreamCaptureStatusNone && ctx->prof_layer >= 0) { ctx->prof_active_layer = ctx->prof_layer; ctx->prof_layer = -1; }
    struct Disarm { pc_ctx* c; ~Disarm() { c->prof_active_layer = -1; } } disarm{ctx};
    launch_k(pc::prep_decode_rows, dim3((m_bound + 128) / 128), dim3(128), 0, st, sd, da, a.prompt_slots, a.suffix_slots, ctx->d.vocab, g, keys, ctx->err);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("prep_decode_rows");
    const pc::KvArena pa{const_cast<void*>(a.prompt_kv), a.prompt_slots}, sa{a.suffix_kv, a.suffix_slots};
    const bool f32 = ctx->d.dtype == PC_DTYPE_F32;
    const AttnPlan plan{false, groups_bound, keys.group_start, group_rows_bound};
    float* logits = logits_out ? logits_out : reinterpret_cast<float*>(ctx->ws + ctx->cv.logits);
    int rc;
    if (!f32 && ctx->decode_mode == 1 && ctx->chain_ready) {
        rc = run_decode_chained(ctx, st, m_bound, sd, pa, sa, plan, logits);
        if (rc) return rc;
    } else {
        rc = f32 ? run_layers<float>(ctx, st, m_bound, sd, pa, sa, plan) : run_layers<__nv_bfloat16>(ctx, st, m_bound, sd, pa, sa, plan);
        if (rc) return rc;
        if (!f32 && a.sample && logits_out == nullptr && a.logprobs == nullptr && ctx->fused_sampler) {
            // nobody asked for the logits: the draw happens in the LM head's epilogue and they are never stored
            return run_lm_head_sample(ctx, st, m_bound, sd, keys, da);
        }
        rc = f32 ? run_lm_head<float>(ctx, st, m_bound, sd, nullptr, logits) : run_lm_head<__nv_bfloat16>(ctx, st, m_bound, sd, nullptr, logits);
        if (rc) return rc;
    }
    if (a.sample) {
        // keys, output positions, token buffer, temperature and seed come from the workspace copies / the argument block
        const int chunks = pc::sample_chunks(m_bound, ctx->num_sms);
        if (chunks == 1) {
            launch_k(pc::sample_kernel, dim3(m_bound), dim3(256), 0, st, sd, ctx->d.vocab, logits, nullptr, 1.f, 0u, 0u, keys.key_prompt, keys.rollout,
                                                       keys.step_key, 0, nullptr, keys.out_index, 0, nullptr, nullptr, da);
            count_launches(1);
        } else {
            pc::Top2Rec* scratch = reinterpret_cast<pc::Top2Rec*>(ctx->ws + ctx->cv.sample_scratch);
            launch_k(pc::sample_partial_kernel, dim3(dim3(m_bound, chunks)), dim3(256), 0, st, sd, ctx->d.vocab, chunks, logits, nullptr, 1.f, 0u, 0u,
                                                                             keys.key_prompt, keys.rollout, keys.step_key, 0, scratch, nullptr, da);
            launch_k(pc::sample_reduce_kernel, dim3((m_bound + 127) / 128), dim3(128), 0, st, sd, m_bound, chunks, scratch, nullptr, keys.out_index, 0,
                                                                            nullptr, da);
            count_launches(2);
        }
        if (a.logprobs != nullptr) {
            launch_k(pc::token_logprob_kernel, dim3(m_bound), dim3(256), 0, st, sd, ctx->d.vocab, logits, nullptr, 1.f, nullptr, keys.out_index, 0, nullptr,
                                                              keys.out_index, 0, da);
            count_launches(1);
        }
        ctx->mark(st, -1, PC_MARK_SAMPLE);
        PC_CUDA_CHECK_LAUNCH("sample");
    }
    return PC_OK;
}

}  // namespace

extern "C" {

int pc_decode_step(pc_ctx* ctx, void* stream, int n_rows, const int32_t* row_prompt, const int32_t* row_rollout,
                   const int32_t* row_step, const int64_t* row_kv_start, int32_t* tokens, const int64_t* row_tok_index,
                   int n_groups, const int32_t* group_row_start, int max_group_rows, const int32_t* prompt_len,
                   const void* prompt_kv, int64_t prompt_slots, const int64_t* prompt_kv_start, void* suffix_kv,
                   int64_t suffix_slots, float* logits_out, const pc_sample_params* sample) {
    if (int rc = check_ready(ctx)) return rc;
    if (n_rows < 0 || n_groups < 0 || max_group_rows < 0) return PC_ERR_INVALID_ARG;
    if (n_rows == 0) return PC_OK;
    DecodeArgs a = make_decode_args(row_prompt, row_rollout, row_step, row_kv_start, tokens, row_tok_index, group_row_start,
                                          prompt_len, prompt_kv, prompt_slots, prompt_kv_start, suffix_kv, suffix_slots, sample);
    if (int rc = check_decode_args(ctx, a)) return rc;
    a.logprobs = ctx->logprobs;
    a.prompt_key = ctx->prompt_key;
    if (n_groups == 0 || max_group_rows == 0 || max_group_rows > n_rows || n_groups > n_rows) return PC_ERR_INVALID_ARG;
    if (logits_out == nullptr && sample == nullptr) return PC_ERR_INVALID_ARG;
    if (logits_out && !aligned(logits_out, 16)) return PC_ERR_ALIGNMENT;
    if (n_rows > ctx->max_rows) return PC_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->d.dtype == PC_DTYPE_BF16)
        if (int rc = arena_maps(ctx, prompt_kv, prompt_slots, suffix_kv, suffix_slots)) return rc;
    if (int rc = upload_decode_args(ctx, st, a, nullptr)) return rc;
    pc::set_step_desc<<<1, pc::STEP_DESC_THREADS, 0, st>>>(reinterpret_cast<pc::StepDesc*>(ctx->ws + ctx->cv.step_desc), n_rows, n_groups,
                                                           max_group_rows, reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.max_slen),
                                                           reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.chain_bar),
                                                           (int)chain_bar_words(ctx->d.n_layers));
    count_launches(1);
    int groups_bound, group_rows_bound;
    canonical_group_bounds(ctx, n_groups, max_group_rows, n_rows, &groups_bound, &group_rows_bound);
    return decode_launches(ctx, st, n_rows, groups_bound, group_rows_bound, a, logits_out);
}

int pc_decode_run(pc_ctx* ctx, void* stream, int n_steps, const pc_step_desc* steps_host, const pc_step_desc* steps_dev,
                  const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step, const int64_t* row_kv_start,
                  int32_t* tokens, const int64_t* row_tok_index, const int32_t* group_row_start, const int32_t* prompt_len,
                  const void* prompt_kv, int64_t prompt_slots, const int64_t* prompt_kv_start, void* suffix_kv,
                  int64_t suffix_slots, const pc_sample_params* sample) {
    static_assert(sizeof(pc_step_desc) == sizeof(pc::StepDesc), "the public and the device step descriptor must agree");
    if (int rc = check_ready(ctx)) return rc;
    if (n_steps < 0) return PC_ERR_INVALID_ARG;
    if (n_steps == 0) return PC_OK;
    if (steps_host == nullptr || steps_dev == nullptr || sample == nullptr) return PC_ERR_INVALID_ARG;
    DecodeArgs a = make_decode_args(row_prompt, row_rollout, row_step, row_kv_start, tokens, row_tok_index, group_row_start,
                                          prompt_len, prompt_kv, prompt_slots, prompt_kv_start, suffix_kv, suffix_slots, sample);
    if (int rc = check_decode_args(ctx, a)) return rc;
    a.logprobs = ctx->logprobs;
    a.prompt_key = ctx->prompt_key;
    for (int s = 0; s < n_steps; ++s) {
        const pc_step_desc& d = steps_host[s];
        if (d.n_rows < 0 || d.n_rows > ctx->max_rows || d.n_groups < 0 || d.n_groups > d.n_rows || d.max_group_rows < 0 ||
            d.max_group_rows > d.n_rows || d.row_offset < 0 || d.group_offset < 0 || (d.n_rows > 0 && (d.n_groups == 0 || d.max_group_rows == 0)))
            return d.n_rows > ctx->max_rows ? PC_ERR_CAPACITY : PC_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (ctx->d.dtype == PC_DTYPE_BF16)
        if (int rc = arena_maps(ctx, prompt_kv, prompt_slots, suffix_kv, suffix_slots)) return rc;
    int32_t* counter = reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.step_counter);
    pc::StepDesc* sd = reinterpret_cast<pc::StepDesc*>(ctx->ws + ctx->cv.step_desc);
    if (int rc = upload_decode_args(ctx, st, a, steps_dev)) return rc;
    const pc::DecodeArgsDev* da = reinterpret_cast<const pc::DecodeArgsDev*>(ctx->ws + ctx->cv.dargs);
    cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return cuda_fail(e, "reset step counter");
    for (int s = 0; s < n_steps; ++s) {
        if (steps_host[s].n_rows == 0) {          // keep the device counter in step with the host loop
            pc::load_step_desc<<<1, pc::STEP_DESC_THREADS, 0, st>>>(da, counter, sd, reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.max_slen),
                                                                    nullptr, 0);
            count_launches(1);
            continue;
        }
        const int m_bound = std::min(ctx->max_rows, (steps_host[s].n_rows + 127) / 128 * 128);
        int groups_bound, group_rows_bound;
        canonical_group_bounds(ctx, steps_host[s].n_groups, steps_host[s].max_group_rows, m_bound, &groups_bound, &group_rows_bound);
        GraphKey key;
        std::memset(&key, 0, sizeof(key));
        key.m_bound = m_bound; key.groups_bound = groups_bound; key.group_rows_bound = group_rows_bound;
        key.sample = a.sample; key.logprobs = a.logprobs != nullptr; key.decode_mode = ctx->decode_mode;
        key.prompt_kv = a.prompt_kv; key.prompt_slots = a.prompt_slots; key.suffix_kv = a.suffix_kv; key.suffix_slots = a.suffix_slots;
        cudaGraphExec_t exec = nullptr;
        for (auto& ent : ctx->graphs)
            if (std::memcmp(&ent.key, &key, sizeof(key)) == 0) { exec = ent.exec; break; }
        if (exec == nullptr) {
            if (ctx->graphs.size() >= 64) ctx->drop_graphs();
            cudaGraph_t graph = nullptr;
            if (ctx->capture_stream == nullptr) {
                e = cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking);
                if (e != cudaSuccess) return cuda_fail(e, "create capture stream");
            }
            cudaStream_t cs = ctx->capture_stream;
            e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
            if (e != cudaSuccess) return cuda_fail(e, "begin graph capture");
            g_capture_launches = 0;                // launches are recorded into the graph, not run
            pc::load_step_desc<<<1, pc::STEP_DESC_THREADS, 0, cs>>>(da, counter, sd,
                                                                    reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.max_slen),
                                                                    reinterpret_cast<int32_t*>(ctx->ws + ctx->cv.chain_bar),
                                                                    (int)chain_bar_words(ctx->d.n_layers));
            count_launches(1);
            const int rc = decode_launches(ctx, cs, m_bound, groups_bound, group_rows_bound, a, nullptr);
            e = cudaStreamEndCapture(cs, &graph);
            const int captured = (int)g_capture_launches;
            g_capture_launches = -1;
            if (rc != PC_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
            if (e != cudaSuccess) return cuda_fail(e, "end graph capture");
            e = cudaGraphInstantiate(&exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) return cuda_fail(e, "graph instantiate");
            GraphEntry ent;
            ent.key = key; ent.exec = exec; ent.launches = captured;
            ++ctx->captures;
            ctx->graphs.push_back(ent);
        }
        e = cudaGraphLaunch(exec, st);
        if (e != cudaSuccess) return cuda_fail(e, "graph launch");
        for (auto& ent : ctx->graphs)
            if (ent.exec == exec) { count_launches(ent.launches); break; }
    }
    return PC_OK;
}

int pc_sample(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row, float temperature,
              uint64_t seed, const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step,
              int32_t* out_tokens, const int64_t* out_index, float* out_top2_gap, void* scratch, size_t scratch_bytes) {
    if (n_rows < 0 || vocab <= 0 || !(temperature > 0.f)) return PC_ERR_INVALID_ARG;
    if (n_rows == 0) return PC_OK;
    if (logits == nullptr || row_prompt == nullptr || row_rollout == nullptr || row_step == nullptr || out_tokens == nullptr)
        return PC_ERR_INVALID_ARG;
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (scratch != nullptr && !aligned(scratch, 16)) return PC_ERR_ALIGNMENT;
    int chunks = 1;
    if (scratch != nullptr) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess)
            chunks = pc::sample_chunks(n_rows, sms);
        while (chunks > 1 && (size_t)n_rows * chunks * sizeof(pc::Top2Rec) > scratch_bytes) --chunks;    // use what fits
    }
    if (chunks == 1) {
        launch_k(pc::sample_kernel, dim3(n_rows), dim3(256), 0, st, nullptr, vocab, logits, logits_row, temperature, k0, k1, row_prompt, row_rollout,
                                                  row_step, 0, out_tokens, out_index, 0, out_top2_gap, nullptr, nullptr);
        count_launches(1);
    } else {
        pc::Top2Rec* rec = static_cast<pc::Top2Rec*>(scratch);
        launch_k(pc::sample_partial_kernel, dim3(dim3(n_rows, chunks)), dim3(256), 0, st, nullptr, vocab, chunks, logits, logits_row, temperature, k0, k1,
                                                                        row_prompt, row_rollout, row_step, 0, rec, nullptr, nullptr);
        launch_k(pc::sample_reduce_kernel, dim3((n_rows + 127) / 128), dim3(128), 0, st, nullptr, n_rows, chunks, rec, out_tokens, out_index, 0,
                                                                       out_top2_gap, nullptr);
        count_launches(2);
    }
    PC_CUDA_CHECK_LAUNCH("sample");
    return PC_OK;
}

int pc_reward_last_token(void* stream, int n, const int32_t* tokens, const int64_t* last_index, const int32_t* threshold,
                         float* reward) {
    if (n < 0) return PC_ERR_INVALID_ARG;
    if (n == 0) return PC_OK;
    if (tokens == nullptr || last_index == nullptr || threshold == nullptr || reward == nullptr) return PC_ERR_INVALID_ARG;
    pc::reward_last_token_kernel<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(n, tokens, last_index, threshold,
                                                                                                reward);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("reward");
    return PC_OK;
}

int pc_group_stats(void* stream, int n_groups, const float* rewards, const int32_t* group_start, const int32_t* group_count,
                   int32_t* n, int32_t* n_success, float* mean, float* var) {
    if (n_groups < 0) return PC_ERR_INVALID_ARG;
    if (n_groups == 0) return PC_OK;
    if (rewards == nullptr || group_start == nullptr || group_count == nullptr || n == nullptr || n_success == nullptr ||
        mean == nullptr || var == nullptr)
        return PC_ERR_INVALID_ARG;
    const int threads = 128, groups_per_block = threads / 32;
    pc::group_stats_kernel<<<(n_groups + groups_per_block - 1) / groups_per_block, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        n_groups, rewards, group_start, group_count, n, n_success, mean, var);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("group_stats");
    return PC_OK;
}

int pc_allocate(void* stream, int n_prompts, const int32_t* pilot_success, const int32_t* pilot_n, const pc_alloc_params* params,
                int32_t* status, int32_t* extra_rollouts, int32_t* evict, int32_t* n_selected, int64_t* total_rollouts) {
    if (n_prompts < 0 || params == nullptr || n_selected == nullptr || total_rollouts == nullptr) return PC_ERR_INVALID_ARG;
    if (params->n_commit < 0 || params->b_t < 0 || !(params->p_lower <= params->p_upper)) return PC_ERR_INVALID_ARG;
    if (n_prompts > 0 && (pilot_success == nullptr || pilot_n == nullptr || status == nullptr || extra_rollouts == nullptr ||
                          evict == nullptr))
        return PC_ERR_INVALID_ARG;
    pc::allocate_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
        n_prompts, pilot_success, pilot_n, nullptr, 0.0, params->p_lower, params->p_upper, params->p_solve, params->n_commit, params->b_t,
        status, extra_rollouts, evict, n_selected, reinterpret_cast<long long*>(total_rollouts));
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("allocate");
    return PC_OK;
}

int pc_allocate_variance(void* stream, int n_prompts, const float* pilot_var, const int32_t* pilot_n, double var_min, int n_commit,
                         int b_t, int32_t* status, int32_t* extra_rollouts, int32_t* n_selected, int64_t* total_rollouts) {
    if (n_prompts < 0 || n_commit < 0 || b_t < 0 || !(var_min >= 0.0) || n_selected == nullptr || total_rollouts == nullptr)
        return PC_ERR_INVALID_ARG;
    if (n_prompts > 0 && (pilot_var == nullptr || pilot_n == nullptr || status == nullptr || extra_rollouts == nullptr)) return PC_ERR_INVALID_ARG;
    pc::allocate_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
        n_prompts, nullptr, pilot_n, pilot_var, var_min, 0.0, 0.0, 0.0, n_commit, b_t, status, extra_rollouts, nullptr, n_selected,
        reinterpret_cast<long long*>(total_rollouts));
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("allocate (variance filter)");
    return PC_OK;
}

int pc_grpo_advantage(void* stream, int n_groups, const float* rewards, const int32_t* group_start, const int32_t* group_count,
                      const int32_t* status, float* adv) {
    if (n_groups < 0) return PC_ERR_INVALID_ARG;
    if (n_groups == 0) return PC_OK;
    if (rewards == nullptr || group_start == nullptr || group_count == nullptr || adv == nullptr) return PC_ERR_INVALID_ARG;
    const int threads = 128, groups_per_block = threads / 32;
    pc::grpo_advantage_kernel<<<(n_groups + groups_per_block - 1) / groups_per_block, threads, 0, static_cast<cudaStream_t>(stream)>>>(
        n_groups, rewards, group_start, group_count, status, adv);
    count_launches(1);
    PC_CUDA_CHECK_LAUNCH("grpo_advantage");
    return PC_OK;
}


// ---------------------------------------------------------------------------------------------------------------
// pc_sample_static: the two-pass sampler with its scratch inside the library image.
// ---------------------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

constexpr int kStaticSampleMaxRows = 4096;
// One record per (row, vocabulary range).  The array lives in the device image of the library: every GPU that loads
// libpc.so holds these 2 MiB until the process exits.  Its name is only a host-side handle here; kernels are given
// the device address that cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_sample_scratch[(size_t)kStaticSampleMaxRows * pc::SAMPLE_MAX_CHUNKS *
                                                                       sizeof(pc::Top2Rec)];

constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};      // device address of the array, per device ordinal
int g_static_scratch_sms[kMaxDevices] = {};

}  // namespace

extern "C" {

int pc_sample_static(void* stream, int n_rows, int vocab, const float* logits, const int32_t* logits_row, float temperature,
                     uint64_t seed, const int32_t* row_prompt, const int32_t* row_rollout, const int32_t* row_step,
                     int32_t* out_tokens, const int64_t* out_index, float* out_top2_gap) {
    if (n_rows < 0 || vocab <= 0 || !(temperature > 0.f)) return PC_ERR_INVALID_ARG;
    if (n_rows > kStaticSampleMaxRows) {
        g_cuda_error = "pc_sample_static: n_rows exceeds the built-in scratch (4096 rows)";
        return PC_ERR_CAPACITY;
    }
    if (n_rows == 0) return PC_OK;
    if (logits == nullptr || row_prompt == nullptr || row_rollout == nullptr || row_step == nullptr || out_tokens == nullptr)
        return PC_ERR_INVALID_ARG;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return PC_ERR_UNSUPPORTED;
    if (g_static_scratch_addr[dev] == nullptr) {
        // first call on this device: resolve the array's device address (the device is current)
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_sample_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static sampler scratch)");
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        g_static_scratch_sms[dev] = sms;
        g_static_scratch_addr[dev] = p;
    }
    pc::Top2Rec* rec = static_cast<pc::Top2Rec*>(g_static_scratch_addr[dev]);
    const int chunks = pc::sample_chunks(n_rows, g_static_scratch_sms[dev]);
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // every record the second kernel reads is written by the first one in this same call: nothing has to start at zero
    launch_k(pc::sample_partial_kernel, dim3(dim3(n_rows, chunks)), dim3(256), 0, st, nullptr, vocab, chunks, logits, logits_row, temperature, k0, k1,
                                                                    row_prompt, row_rollout, row_step, 0, rec, nullptr, nullptr);
    launch_k(pc::sample_reduce_kernel, dim3((n_rows + 127) / 128), dim3(128), 0, st, nullptr, n_rows, chunks, rec, out_tokens, out_index, 0, out_top2_gap, nullptr);
    count_launches(2);
    PC_CUDA_CHECK_LAUNCH("sample (static scratch)");
    return PC_OK;
}

}  // extern "C"
