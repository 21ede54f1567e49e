// Host side of the C ABI declared in include/kimad.h: context, static planner (candidate table,
// chunk table, workspace layout) and the per-step launch sequence.  No device memory is allocated
// here; the caller's workspace is carved into the regions listed in `Layout`.
#include <cmath>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "kimad_select.cuh"
#include "kimad_receiver.cuh"

using namespace kimad;

namespace {

constexpr int kGroups = 2; // groups of workers in flight at a time (see kimad_ctx::gstream)
constexpr size_t kAlign = 256;
constexpr int kCanaryByte = 0xA5; // checked build: fill of the guard words between workspace regions
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
    // static tables
    size_t dbuf, chunks, layers, ktab, ktab_dyn, reg_layers, tiny_layers, reg_index, runs;
    // zeroed at set_workspace and kept clean by the kernels
    size_t zero_from, h1_cnt, h1_ss, h23_cnt, h23_ss, bh_cnt, bh_sum, low_hist, recount, recount_bytes, fb, r2, flags;
    // scratch without initial-state requirements
    size_t cell_tab, cell_win, bin_lo, meta, cands, slots, err, tau, keep_eq, shift, sel, chunk_cnt, jobs, csel,
        fb_chunks, fb_layers, r2_chunks, r2_layers, rf, rf_chunks, rf_layers, pd, total;
};

} // namespace

struct kimad_ctx {
    uint32_t L = 0, W = 0, K = 0, D = 1000;
    uint32_t value_dtype = 0, check_finite = 0;
    uint64_t N = 0, stride = 0, dstride = 0, cap = 0, full_bytes = 0;
    uint32_t bpe = 8;
    std::vector<uint64_t> layer_sizes, ktab;
    std::vector<double> grid;
    std::vector<Chunk> chunks;
    std::vector<LayerDesc> layers;
    std::vector<uint32_t> reg_layers, tiny_layers, reg_index; // layers above / up to kTinyMax elements
    std::vector<SweepRun> runs;                               // the sweep's CTAs: static runs of chunks, balanced by elements
    std::vector<unsigned char> static_image;                  // the static tables as they lie in the workspace, one block
    std::vector<size_t> guards;                               // checked build: offsets of the canary words between regions
    uint32_t curve_mode = 0;
    uint32_t policy = 0, cost_model = 0;
    size_t sample_smem = 0, pass_a_smem = 0, tiny_smem = 0;
    Layout lay{};
    unsigned char* ws = nullptr;
    DpPlan dp_plan{};
    size_t dp_smem = 0;
    uint64_t launches = 0;
    kimad_packed last_out{};
    bool have_last = false;
    bool timing = false;
    cudaEvent_t ev[KIMAD_N_STAGES + 1] = {};
    // the tiny layers' exact curves depend on the step's inputs only: they run on a stream of their own, forked
    // from and joined to the caller's stream with events
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // two groups of workers are taken through the stages after the sample on streams of their own, the first with
    // the higher priority: while one group is in its latency-bound stages (curves, DP, offsets) the other one streams
    // (every group has a stream for its sweeps, of low priority, and one for its short kernels, of high priority, so
    // that a DP or an offset scan is not queued behind another group's sweep; events hand the group over between
    // the two)
    cudaStream_t gstream[kGroups] = {}, gshort[kGroups] = {}, glist[kGroups] = {};
    cudaEvent_t ev_go = nullptr, ev_done[kGroups] = {}, ev_hand[kGroups][4] = {}, ev_list[kGroups][2] = {};
    int pipeline_mode = 0; // 0: two groups when the step is large enough, 1: whenever W >= 2, 2: never
    bool have_ev = false;
    template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace {

void plan_layout(kimad_ctx* c) {
    Layout& y = c->lay;
    size_t o = 0;
    c->guards.clear();
    auto take = [&](size_t bytes) {
        size_t at = o;
        o = align_up(o + bytes);
#ifdef KIMAD_CHECKED
        c->guards.push_back(o); // a canary of kAlign bytes behind every region
        o += kAlign;
#endif
        return at;
    };
    const size_t WL = (size_t)c->W * c->L, WLK = WL * c->K, WR = (size_t)c->W * c->reg_layers.size();
    const size_t nch = c->chunks.size();
    y.dbuf = take((size_t)c->W * c->dstride * sizeof(uint8_t));
    y.chunks = take(nch * sizeof(Chunk));
    y.layers = take(c->layers.size() * sizeof(LayerDesc));
    y.ktab = take(c->ktab.size() * sizeof(uint64_t));
    y.ktab_dyn = take(c->policy == 3 ? (size_t)c->W * c->L * sizeof(uint64_t) : 0); // per-worker rows of the fitted ratio
    y.reg_layers = take(c->reg_layers.size() * sizeof(uint32_t));
    y.tiny_layers = take(c->tiny_layers.size() * sizeof(uint32_t));
    y.reg_index = take(c->reg_index.size() * sizeof(uint32_t));
    y.runs = take(c->runs.size() * sizeof(SweepRun));
    y.zero_from = o;
    y.h1_cnt = take(WL * kL1Bins * sizeof(uint32_t));
    y.h1_ss = take(WL * kL1Bins * sizeof(uint64_t));
    y.h23_cnt = take(WLK * kL23Bins * sizeof(uint32_t));
    y.h23_ss = take(WLK * kL23Bins * sizeof(uint64_t));
    y.bh_cnt = take(WR * kMaxBins * sizeof(uint32_t));
    y.bh_sum = take(WR * kMaxBins * sizeof(uint64_t));
    y.low_hist = take(WL * kLowBins * sizeof(uint32_t));
    // work lists, one set per group of workers
    y.recount_bytes = align_up(256 + (size_t)2 * c->W * nch * sizeof(uint2));
    y.recount = take(kGroups * y.recount_bytes);
    y.fb = take(kGroups * align_up(sizeof(FbList)));
    y.r2 = take(kGroups * align_up(sizeof(Round2)));
    y.flags = take((size_t)c->W * sizeof(uint32_t));
    y.cell_tab = take(WR * kCellTab * sizeof(uint32_t));
    y.cell_win = take(WR * sizeof(int4));
    y.bin_lo = take(WR * (kMaxBins + 1) * sizeof(uint32_t));
    y.meta = take(WR * sizeof(BandMeta));
    y.cands = take(WLK * sizeof(Cand));
    y.slots = take(WL * sizeof(SlotTab));
    y.err = take(WLK * sizeof(float));
    y.tau = take(WLK * sizeof(uint32_t));
    y.keep_eq = take(WLK * sizeof(uint32_t));
    y.shift = take(WLK * sizeof(uint32_t));
    y.sel = take(WL * sizeof(Sel));
    y.chunk_cnt = take((size_t)c->W * nch * sizeof(uint2));
    y.jobs = take((size_t)c->W * nch * sizeof(ChunkJob));
    y.csel = take((size_t)c->W * nch * sizeof(ChunkSel));
    y.fb_chunks = take(kGroups * align_up((size_t)c->W * nch * sizeof(uint2)));
    y.fb_layers = take(kGroups * align_up(WL * sizeof(uint2)));
    y.r2_chunks = take(kGroups * align_up((size_t)c->W * nch * sizeof(uint2)));
    y.r2_layers = take(kGroups * align_up(WL * sizeof(uint2)));
    y.rf = take(WLK * sizeof(RefineCand));
    y.rf_chunks = take(kGroups * align_up((size_t)c->W * nch * sizeof(uint2)));
    y.rf_layers = take(kGroups * align_up(WL * sizeof(uint2)));
    y.pd = take(c->dp_plan.pd_in_smem ? 0 : (size_t)c->W * c->L * c->dp_plan.pd_row_bytes);
    y.total = o;
}

#define CUDA_TRY(x)                                  \
    do {                                             \
        if ((x) != cudaSuccess) return KIMAD_ERR_CUDA; \
    } while (0)

constexpr size_t kDpSmemMax = 225 * 1024; // dynamic shared memory the DP kernel may ask for
constexpr uint64_t kSweepRunElems = 4ull << 20; // elements a CTA of the sweep takes at most (as long as four waves suffice)
constexpr uint64_t kPipelineMinElems = 1ull << 25; // W N from which a step is run as two groups of workers

// Kernels are loaded on their first launch; loading one takes about a millisecond.  Touching every kernel a
// step can launch (the rarely taken ones included) when the workspace is attached keeps that out of the steps.
static int preload_kernels() {
    cudaFuncAttributes a;
#define KIMAD_PRELOAD(f) CUDA_TRY(cudaFuncGetAttributes(&a, f))
    KIMAD_PRELOAD(k_sample); KIMAD_PRELOAD(k_pass_a<true>); KIMAD_PRELOAD(k_pass_a<false>); KIMAD_PRELOAD(k_resolve_a);
    KIMAD_PRELOAD(k_refine_hist); KIMAD_PRELOAD(k_refine_resolve);
    KIMAD_PRELOAD(k_tiny_exact); KIMAD_PRELOAD(k_fb_hist1); KIMAD_PRELOAD(k_fb_hist23<2>); KIMAD_PRELOAD(k_fb_hist23<3>);
    KIMAD_PRELOAD(k_resolve1); KIMAD_PRELOAD(k_resolve23<2>); KIMAD_PRELOAD(k_resolve23<3>); KIMAD_PRELOAD(k_rebuild_slots);
    KIMAD_PRELOAD(k_dp); KIMAD_PRELOAD(k_fit_ratio); KIMAD_PRELOAD(k_sel_count); KIMAD_PRELOAD(k_sel_count_r2); KIMAD_PRELOAD(k_sel_resolve);
    KIMAD_PRELOAD(k_sel_resolve_r2); KIMAD_PRELOAD(k_sel_recount); KIMAD_PRELOAD(k_sel_slices); KIMAD_PRELOAD(k_sel_scan);
    KIMAD_PRELOAD((k_sel_write<false, false>)); KIMAD_PRELOAD((k_sel_write<false, true>));
    KIMAD_PRELOAD((k_sel_write<true, false>)); KIMAD_PRELOAD((k_sel_write<true, true>));
    KIMAD_PRELOAD(k_apply_packed<false>); KIMAD_PRELOAD(k_apply_packed<true>);
    KIMAD_PRELOAD(k_aggregate<false>); KIMAD_PRELOAD(k_aggregate<true>);
#undef KIMAD_PRELOAD
    return KIMAD_OK;
}

// Launch trace (kimad_debug_trace_step): while a traced step is being issued every launch is bracketed by a pair of
// CUDA events on its stream.  One traced step at a time per process (a development aid, not thread-safe).
struct LaunchRec { const char* name; cudaStream_t s; cudaEvent_t a, b; };
static std::vector<LaunchRec>* g_launch_trace = nullptr;

// Launch with programmatic stream serialisation (the kernel must start with pdl_wait()).
template <typename... KArgs, typename... Args>
static cudaError_t launch_named(const char* name, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                Args... args) {
    LaunchRec rec{name, s, nullptr, nullptr};
    if (g_launch_trace) {
        if (cudaEventCreate(&rec.a) != cudaSuccess || cudaEventCreate(&rec.b) != cudaSuccess) return cudaErrorUnknown;
        cudaEventRecord(rec.a, s);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
    if (g_launch_trace) {
        cudaEventRecord(rec.b, s);
        g_launch_trace->push_back(rec);
    }
    return e;
}
#define launch_pdl(kern, ...) launch_named(#kern, kern, __VA_ARGS__)

static int ensure_side_stream(kimad_ctx* c) {
    if (c->side) return KIMAD_OK;
    CUDA_TRY(cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking));
    CUDA_TRY(cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming));
    int prio_least = 0, prio_greatest = 0;
    CUDA_TRY(cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
    for (int g = 0; g < kGroups; ++g) {
        CUDA_TRY(cudaStreamCreateWithPriority(&c->gstream[g], cudaStreamNonBlocking, prio_least));
        CUDA_TRY(cudaStreamCreateWithPriority(&c->gshort[g], cudaStreamNonBlocking, prio_greatest));
        CUDA_TRY(cudaStreamCreateWithPriority(&c->glist[g], cudaStreamNonBlocking, prio_greatest));
        for (cudaEvent_t& e : c->ev_list[g]) CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&c->ev_done[g], cudaEventDisableTiming));
        for (cudaEvent_t& e : c->ev_hand[g]) CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    }
    CUDA_TRY(cudaEventCreateWithFlags(&c->ev_go, cudaEventDisableTiming));
    return KIMAD_OK;
}

// Once per device and process: shared-memory limits of the kernels (a property of the function, shared by all
// contexts: the limits do not depend on the context) and the kernel preload.  Per context: its side stream.
static int prepare_device(kimad_ctx* c) {
    static bool ready[KIMAD_BUILTIN_MAX_DEVICES] = {};
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= KIMAD_BUILTIN_MAX_DEVICES) return KIMAD_ERR_INVALID_ARG;
    if (!ready[dev]) {
        CUDA_TRY(cudaFuncSetAttribute(k_dp, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDpSmemMax));
        CUDA_TRY(cudaFuncSetAttribute(k_sample, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->sample_smem));
        CUDA_TRY(cudaFuncSetAttribute(k_pass_a<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->pass_a_smem));
        CUDA_TRY(cudaFuncSetAttribute(k_pass_a<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->pass_a_smem));
        CUDA_TRY(cudaFuncSetAttribute(k_tiny_exact, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->tiny_smem));
        { const int rc_pre = preload_kernels(); if (rc_pre != KIMAD_OK) return rc_pre; }
        ready[dev] = true;
    }
    return ensure_side_stream(c);
}

// Checked build: (re)writes the canaries of a workspace, in stream order.  A no-op otherwise (no guards are planned).
static int fill_guards(const kimad_ctx* c, unsigned char* ws, cudaStream_t s) {
    for (size_t g : c->guards) CUDA_TRY(cudaMemsetAsync(ws + g, kCanaryByte, kAlign, s));
    return KIMAD_OK;
}

enum StepMode { kNormal = 0, kInjectErr = 1, kGivenJ = 2 };

int run_step(kimad_ctx* c, const float* grads, float* state, const double* bw, double t, const kimad_packed* out,
             void* stream_v, StepMode mode, const float* err_dev, const uint32_t* j_dev) {
    if (!c || !grads || !state || !bw || !out || !out->idx || !out->val || !out->offs || !out->k || !out->j ||
        !out->stats)
        return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    if (!(t >= 0.0)) return KIMAD_ERR_INVALID_ARG;
    if (mode == kInjectErr && !err_dev) return KIMAD_ERR_INVALID_ARG;
    if (mode == kGivenJ && !j_dev) return KIMAD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream_v);
    const uint32_t L = c->L, W = c->W, K = c->K;
    const uint32_t nch = (uint32_t)c->chunks.size();
    const bool vec = ((uintptr_t)grads % 16 == 0) && ((uintptr_t)state % 16 == 0) && (c->stride % 4 == 0);

    const Layout& y = c->lay;
    // one code byte per element, u8 [W][dstride]; exact values are recomputed from grads and state
    const DSource dbuf{c->at<uint8_t>(y.dbuf), grads, state, c->stride};
    const Chunk* chunks = c->at<Chunk>(y.chunks);
    const LayerDesc* layers = c->at<LayerDesc>(y.layers);
    // candidates: the grid's table for every worker, or (policy 3) each worker's row of the ratio fitted to its budget
    const KTab ktab = c->policy == 3 && mode != kGivenJ ? KTab{c->at<uint64_t>(y.ktab_dyn), (uint64_t)c->L * c->K}
                                                        : KTab{c->at<uint64_t>(y.ktab), 0};
    const uint32_t* reg_layers = c->at<uint32_t>(y.reg_layers);
    const uint32_t* tiny_layers = c->at<uint32_t>(y.tiny_layers);
    const uint32_t* reg_index = c->at<uint32_t>(y.reg_index);
    uint32_t* h1c = c->at<uint32_t>(y.h1_cnt);
    unsigned long long* h1s = c->at<unsigned long long>(y.h1_ss);
    uint32_t* h23c = c->at<uint32_t>(y.h23_cnt);
    unsigned long long* h23s = c->at<unsigned long long>(y.h23_ss);
    uint32_t* bhc = c->at<uint32_t>(y.bh_cnt);
    unsigned long long* bhs = c->at<unsigned long long>(y.bh_sum);
    uint32_t* cell_tab = c->at<uint32_t>(y.cell_tab);
    int4* cell_win = c->at<int4>(y.cell_win);
    uint32_t* binlo = c->at<uint32_t>(y.bin_lo);
    BandMeta* meta = c->at<BandMeta>(y.meta);
    Cand* cands = c->at<Cand>(y.cands);
    SlotTab* slots = c->at<SlotTab>(y.slots);
    float* err = c->at<float>(y.err);
    uint32_t* tau = c->at<uint32_t>(y.tau);
    uint32_t* keq = c->at<uint32_t>(y.keep_eq);
    uint32_t* shf = c->at<uint32_t>(y.shift);
    Sel* sel = c->at<Sel>(y.sel);
    uint2* ccnt = c->at<uint2>(y.chunk_cnt);
    ChunkJob* jobs = c->at<ChunkJob>(y.jobs);
    ChunkSel* csel = c->at<ChunkSel>(y.csel);
    uint32_t* lowh = c->at<uint32_t>(y.low_hist);
    uint32_t* flags = c->at<uint32_t>(y.flags);
    uint8_t* pd = c->at<uint8_t>(y.pd);
    const SweepRun* runs = c->at<SweepRun>(y.runs);

    const uint32_t R = (uint32_t)c->reg_layers.size(), T = (uint32_t)c->tiny_layers.size();
    const dim3 blk(kThreads);
    const uint32_t list_cap = W * nch; // entries of every chunk list (twice that for the recount list)
    int stage = 0;
    auto mark = [&](cudaStream_t st) { if (c->timing) cudaEventRecord(c->ev[stage++], st); };
    auto budgets_of = [&](uint32_t w0, uint32_t nw) {
        DpBudgets b{};
        for (uint32_t i = 0; i < nw; ++i) {
            double cb = std::floor(bw[w0 + i] * t);
            b.c[i] = !(cb > 0.0) ? 0ull : (cb >= 18446744073709551615.0 ? ~0ull : (uint64_t)cb);
        }
        return b;
    };
    // Two groups of workers (none when the stages are being timed, or for small steps, where it gains nothing)
    const bool two = !c->timing && W >= 2 && c->pipeline_mode != 2 &&
                     (c->pipeline_mode == 1 || (uint64_t)W * c->N >= kPipelineMinElems);
    const uint32_t n_groups = two ? 2u : 1u;

    mark(s);
    if (c->policy == 3 && mode != kGivenJ) { // Section 3.1: the one ratio sized to each worker's budget
        for (uint32_t w0 = 0; w0 < W; w0 += kDpWorkersPerLaunch) {
            const uint32_t nw = std::min<uint32_t>(kDpWorkersPerLaunch, W - w0);
            CUDA_TRY(launch_pdl(k_fit_ratio, nw, blk, 0, s, budgets_of(w0, nw), w0, W, L, c->bpe, c->N, layers,
                                c->at<uint64_t>(y.ktab_dyn)));
            c->launches += 1;
        }
    }
    if (T) CUDA_TRY(cudaEventRecord(c->ev_fork, s)); // fork point of the tiny layers' kernel: the step's start
    // (a) + (b): sample -> bands, all workers
    if (R) {
        CUDA_TRY(launch_pdl(k_sample, dim3(R, W), kBigThreads, c->sample_smem, s, grads, state, c->stride, layers, reg_layers, R,
                            ktab, K, c->curve_mode == 1 ? 1u : 0u, cell_tab, cell_win, binlo, meta));
        c->launches += 1;
    }
    if (T) { // tiny layers: sorted in shared memory on the side stream, beside the sample kernel (its CTAs fill what
             // that kernel leaves idle); joined before the sweep, whose CTAs take most of an SM's shared memory and
             // could not start on an SM that still holds CTAs of another kernel
        CUDA_TRY(cudaStreamWaitEvent(c->side, c->ev_fork, 0));
        CUDA_TRY(launch_pdl(k_tiny_exact, dim3(T, W), blk, c->tiny_smem, c->side, grads, state, c->stride, layers, tiny_layers, L,
                            ktab, K, err, tau, keq, shf, flags));
        CUDA_TRY(cudaEventRecord(c->ev_join, c->side));
        CUDA_TRY(cudaStreamWaitEvent(s, c->ev_join, 0));
        c->launches += 1;
    }
    mark(s);
    if (two) CUDA_TRY(cudaEventRecord(c->ev_go, s));
    // budget share kept, from the host's view of the budgets: picks the tuning of the write sweep
    double kept = 0.0;
    for (uint32_t i = 0; i < W; ++i) kept = std::max(kept, std::floor(bw[i] * t) / ((double)c->bpe * (double)c->N));
    const bool dense_write = kept >= 0.04;

    for (uint32_t g = 0; g < n_groups; ++g) {
        // workers [w0, w0 + nw) on stream gs; every group has work lists of its own
        const uint32_t w0 = two ? (g == 0 ? 0u : W / 2) : 0u, nw = two ? (g == 0 ? W / 2 : W - W / 2) : W;
        cudaStream_t big = two ? c->gstream[g] : s, small = two ? c->gshort[g] : s; // sweeps / short kernels
        if (two) CUDA_TRY(cudaStreamWaitEvent(big, c->ev_go, 0));
        int hand = 0;
        auto hand_over = [&](cudaStream_t from, cudaStream_t to) -> cudaError_t { // `to` continues where `from` stands
            if (!two) return cudaSuccess;
            cudaError_t e = cudaEventRecord(c->ev_hand[g][hand], from);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(to, c->ev_hand[g][hand], 0);
            ++hand;
            return e;
        };
        uint32_t* recount_n = c->at<uint32_t>(y.recount + g * y.recount_bytes);
        uint2* recount_list = c->at<uint2>(y.recount + g * y.recount_bytes + 256);
        FbList* fb = c->at<FbList>(y.fb + g * align_up(sizeof(FbList)));
        Round2* r2 = c->at<Round2>(y.r2 + g * align_up(sizeof(Round2)));
        uint2* fb_chunks = c->at<uint2>(y.fb_chunks + g * align_up((size_t)W * nch * sizeof(uint2)));
        uint2* r2_chunks = c->at<uint2>(y.r2_chunks + g * align_up((size_t)W * nch * sizeof(uint2)));
        uint2* fb_layers = c->at<uint2>(y.fb_layers + g * align_up((size_t)W * L * sizeof(uint2)));
        RefineCand* rf = c->at<RefineCand>(y.rf);
        uint2* rf_chunks = c->at<uint2>(y.rf_chunks + g * align_up((size_t)W * nch * sizeof(uint2)));
        uint2* rf_layers = c->at<uint2>(y.rf_layers + g * align_up((size_t)W * L * sizeof(uint2)));
        uint2* r2_layers = c->at<uint2>(y.r2_layers + g * align_up((size_t)W * L * sizeof(uint2)));
        const dim3 gch(nch, nw), glw(L, nw);
        // the group's runs of the sweep: the run table is sorted by worker
        uint32_t run0 = 0, run1 = 0;
        for (uint32_t i = 0; i < (uint32_t)c->runs.size(); ++i) {
            if (c->runs[i].w < w0) run0 = i + 1;
            if (c->runs[i].w < w0 + nw) run1 = i + 1;
        }
        if (vec)
            CUDA_TRY(launch_pdl(k_pass_a<true>, run1 - run0, kBigThreads, c->pass_a_smem, big, grads, state, dbuf.code, chunks, runs + run0,
                                c->stride, c->dstride, reg_index, R, cell_tab, cell_win, meta, bhc, bhs));
        else
            CUDA_TRY(launch_pdl(k_pass_a<false>, run1 - run0, kBigThreads, c->pass_a_smem, big, grads, state, dbuf.code, chunks, runs + run0,
                                c->stride, c->dstride, reg_index, R, cell_tab, cell_win, meta, bhc, bhs));
        c->launches += 1;
        mark(big);
        CUDA_TRY(hand_over(big, small));
        if (R) {
            CUDA_TRY(launch_pdl(k_resolve_a, dim3(R, nw), kBigThreads, 0, small, layers, reg_layers, R, L, ktab, K, meta, binlo, bhc, bhs,
                                err, tau, keq, shf, flags, fb, fb_chunks, fb_layers, rf, rf_chunks, rf_layers, list_cap, w0));
            c->launches += 1;
        }
        mark(small);
        // (c) as a launch sequence on stream st; `when`: 0 always, 1 only if no layer is listed for the refinement or
        // the exact path, 2 only if one is
        auto launch_dp = [&](cudaStream_t st, uint32_t when) -> int {
            for (uint32_t wa = w0; wa < w0 + nw; wa += kDpWorkersPerLaunch) {
                const uint32_t nwa = std::min<uint32_t>(kDpWorkersPerLaunch, w0 + nw - wa);
                const int dp_mode = mode == kGivenJ ? 1 : (c->policy == 1 ? 2 : (c->policy == 2 ? 3 : (c->policy == 3 ? 4 : 0)));
                CUDA_TRY(launch_pdl(k_dp, nwa, kDpThreads, c->dp_smem, st, budgets_of(wa, nwa), wa, W, L, K, c->D, c->bpe, c->full_bytes,
                                    c->cap, c->check_finite, dp_mode, c->cost_model, c->dp_plan, layers,
                                    ktab, mode == kInjectErr ? err_dev : err, tau, keq, shf, j_dev, flags, pd, sel, out->k, out->j,
                                    out->offs, out->stats, out->dense, CodeSpace{reg_index, meta, cell_tab, cell_win, R}, when, fb));
                c->launches += 1;
            }
            return KIMAD_OK;
        };
        // refinement and exact radix select for the layers listed by k_resolve_a (the lists are usually empty)
        auto launch_lists = [&](cudaStream_t st) -> int {
            // small grids: the lists are usually empty, and every kernel of the chain then costs only its launch; the
            // histogram kernels get four CTAs per SM, enough to stream a large handed-over layer
            const uint32_t gfb = 4 * 148, glay = std::min<uint32_t>(nw * R, 32u);
            const dim3 gslot(glay, 1, K);
            // candidates with a loose bound first (they may still end on the exact path's lists)
            CUDA_TRY(launch_pdl(k_refine_hist, 6 * 148, blk, 0, st, dbuf, chunks, c->dstride, L, K, fb, rf_chunks, rf,
                                CodeSpace{reg_index, meta, cell_tab, cell_win, R}, h23c, h23s));
            CUDA_TRY(launch_pdl(k_refine_resolve, glay, blk, 0, st, layers, L, K, fb, rf_layers, rf, h23c, h23s, err, tau, keq, shf,
                                fb_chunks, fb_layers, list_cap));
            CUDA_TRY(launch_pdl(k_fb_hist1, gfb, blk, 0, st, dbuf, chunks, c->dstride, L, fb, fb_chunks, h1c, h1s, flags));
            CUDA_TRY(launch_pdl(k_resolve1, glay, blk, 0, st, fb, fb_layers, h1c, h1s, ktab, L, K, cands, slots));
            CUDA_TRY(launch_pdl(k_fb_hist23<2>, gfb, blk, 0, st, dbuf, chunks, c->dstride, L, K, fb, fb_chunks, slots, h23c, h23s));
            CUDA_TRY(launch_pdl(k_resolve23<2>, gslot, blk, 0, st, fb, fb_layers, h23c, h23s, L, K, cands, slots, err, tau, keq, shf));
            CUDA_TRY(launch_pdl(k_rebuild_slots, (nw * R + kThreads - 1) / kThreads, blk, 0, st, fb, fb_layers, L, K, cands, slots));
            CUDA_TRY(launch_pdl(k_fb_hist23<3>, gfb, blk, 0, st, dbuf, chunks, c->dstride, L, K, fb, fb_chunks, slots, h23c, h23s));
            CUDA_TRY(launch_pdl(k_resolve23<3>, gslot, blk, 0, st, fb, fb_layers, h23c, h23s, L, K, cands, slots, err, tau, keq, shf));
            c->launches += 9;
            return KIMAD_OK;
        };
        if (R && !c->timing) {
            // The lists are usually empty, so the DP is launched at once and goes ahead only if they are; the nine
            // list-driven kernels run beside it on a stream of their own, followed by a second launch of the DP that
            // goes ahead only if something was listed.  Their launch latencies leave the step's critical path.
            cudaStream_t lst = c->glist[g];
            CUDA_TRY(cudaEventRecord(c->ev_list[g][0], small));
            CUDA_TRY(cudaStreamWaitEvent(lst, c->ev_list[g][0], 0));
            { const int rc = launch_dp(small, 1); if (rc != KIMAD_OK) return rc; }
            { const int rc = launch_lists(lst); if (rc != KIMAD_OK) return rc; }
            { const int rc = launch_dp(lst, 2); if (rc != KIMAD_OK) return rc; }
            CUDA_TRY(cudaEventRecord(c->ev_list[g][1], lst));
            CUDA_TRY(cudaStreamWaitEvent(small, c->ev_list[g][1], 0));
        } else {
            if (R) { const int rc = launch_lists(small); if (rc != KIMAD_OK) return rc; }
            mark(small);
            { const int rc = launch_dp(small, 0); if (rc != KIMAD_OK) return rc; }
        }
        mark(small);
        CUDA_TRY(hand_over(small, big));
        // (d), (e), (f)
        CUDA_TRY(launch_pdl(k_sel_count, gch, blk, 0, big, dbuf, chunks, nch, c->dstride, L, sel, layers, csel, lowh, recount_n,
                            recount_list, 2 * list_cap, w0));
        mark(big);
        CUDA_TRY(hand_over(big, small));
        CUDA_TRY(launch_pdl(k_sel_resolve, glw, blk, 0, small, L, layers, nch, csel, lowh, sel, r2, r2_layers, r2_chunks, w0));
        CUDA_TRY(launch_pdl(k_sel_count_r2, 148, blk, 0, small, dbuf, chunks, nch, c->dstride, L, sel, layers, csel, lowh, recount_n,
                            recount_list, 2 * list_cap, r2, r2_chunks));
        CUDA_TRY(launch_pdl(k_sel_resolve_r2, std::min<uint32_t>(nw * L, 32u), blk, 0, small, L, layers, nch, csel, lowh, sel, r2,
                            r2_layers, r2_chunks));
        CUDA_TRY(launch_pdl(k_sel_recount, 148, blk, 0, small, dbuf, chunks, nch, c->dstride, L, sel, recount_n, recount_list, csel));
        CUDA_TRY(launch_pdl(k_sel_slices, (uint32_t)(((uint64_t)nw * nch + 7) / 8), blk, 0, small, chunks, nch, w0, nw, L, sel, csel, ccnt));
        CUDA_TRY(launch_pdl(k_sel_scan, glw, blk, 0, small, layers, chunks, nch, L, sel, ccnt, jobs, recount_n, fb, r2, w0));
        mark(small);
        CUDA_TRY(hand_over(small, big));
        {
            auto launch = [&](auto kern) {
                return launch_named("k_sel_write", kern, gch, blk, 0, big, grads, state, chunks, nch, c->dstride, c->stride, csel,
                                    jobs, c->cap, out->idx, out->val, w0);
            };
            if (c->value_dtype == 1) CUDA_TRY(dense_write ? launch(k_sel_write<true, true>) : launch(k_sel_write<true, false>));
            else CUDA_TRY(dense_write ? launch(k_sel_write<false, true>) : launch(k_sel_write<false, false>));
        }
        mark(big);
        c->launches += 8;
        if (two) CUDA_TRY(cudaEventRecord(c->ev_done[g], big));
    }
    if (two)
        for (uint32_t g = 0; g < n_groups; ++g) CUDA_TRY(cudaStreamWaitEvent(s, c->ev_done[g], 0));
    CUDA_TRY(cudaGetLastError());
    c->last_out = *out;
    c->have_last = true;
    return KIMAD_OK;
}

} // namespace

extern "C" {

int kimad_create(kimad_ctx** out, const uint64_t* layer_sizes, uint32_t n_layers, uint32_t n_workers,
                 const double* ratio_grid, uint32_t n_ratios, const kimad_options* opt) {
    if (!out) return KIMAD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!layer_sizes || !ratio_grid || n_layers == 0 || n_workers == 0 || n_ratios == 0 ||
        n_ratios > KIMAD_MAX_RATIOS)
        return KIMAD_ERR_INVALID_ARG;
    kimad_options o{};
    if (opt) o = *opt;
    if (o.D == 0) o.D = 1000;
    if (o.D > KIMAD_MAX_D || o.D < n_layers || o.value_dtype > 1 || o.infeasible_policy != 0 || o.curve_mode > 1 ||
        o.policy > 3 || o.cost_model > 1)
        return KIMAD_ERR_INVALID_ARG;
    if (o.cost_model == 1 && o.policy >= 2) return KIMAD_ERR_INVALID_ARG;               // dense fallback: policies 0 and 1
    if (o.policy == 3 && (n_ratios != 1 || ratio_grid[0] != 1.0)) return KIMAD_ERR_INVALID_ARG; // the ratio is fitted, not listed
    for (uint32_t j = 0; j < n_ratios; ++j) {
        if (!(ratio_grid[j] > 0.0) || ratio_grid[j] > 1.0) return KIMAD_ERR_INVALID_ARG;
        if (j && !(ratio_grid[j] > ratio_grid[j - 1])) return KIMAD_ERR_INVALID_ARG;
    }
    kimad_ctx* c = new (std::nothrow) kimad_ctx();
    if (!c) return KIMAD_ERR_NOMEM;
    try {
        c->L = n_layers; c->W = n_workers; c->K = n_ratios; c->D = o.D;
        c->value_dtype = o.value_dtype; c->check_finite = o.check_finite;
        c->bpe = o.value_dtype == 0 ? 8 : 6;
        c->layer_sizes.assign(layer_sizes, layer_sizes + n_layers);
        c->grid.assign(ratio_grid, ratio_grid + n_ratios);
        c->ktab.resize((size_t)n_layers * n_ratios);
        uint64_t N = 0;
        for (uint32_t l = 0; l < n_layers; ++l) {
            const uint64_t n = layer_sizes[l];
            if (n == 0 || n > 0xffffffffull) { delete c; return KIMAD_ERR_INVALID_ARG; }
            for (uint32_t j = 0; j < n_ratios; ++j) { // candidate k: ratio of the layer, at least one entry
                uint64_t k = (uint64_t)std::ceil(ratio_grid[j] * (double)n);
                if (k < 1) k = 1;
                if (k > n) k = n;
                c->ktab[(size_t)l * n_ratios + j] = k;
            }
            c->full_bytes += candidate_bytes(n, c->ktab[(size_t)l * n_ratios + n_ratios - 1], c->bpe, o.cost_model, nullptr);
            // chunk table: aligned windows of the flat vector intersected with this layer
            LayerDesc ld{N, n, (uint32_t)c->chunks.size(), 0};
            for (uint64_t p = N; p < N + n;) {
                const uint64_t e = std::min(N + n, (p / kChunkElems + 1) * kChunkElems);
                c->chunks.push_back(Chunk{l, 0, p, e});
                p = e;
            }
            ld.n_chunks = (uint32_t)c->chunks.size() - ld.first_chunk;
            c->layers.push_back(ld);
            if (n <= (uint64_t)kTinyMax) {
                c->reg_index.push_back(0xffffffffu);
                c->tiny_layers.push_back(l);
            } else {
                c->reg_index.push_back((uint32_t)c->reg_layers.size());
                c->reg_layers.push_back(l);
            }
            N += n;
        }
        c->N = N;
        c->stride = o.worker_stride ? o.worker_stride : N;
        c->cap = o.max_packed_elems ? o.max_packed_elems : N;
        if (c->stride < N || c->chunks.size() > 0x7fffffffull) { delete c; return KIMAD_ERR_INVALID_ARG; }
        c->dstride = (N + 15) / 16 * 16; // every worker's code plane starts on a 16-byte boundary
        // shared-memory plan of the DP kernel
        const size_t Kp = (c->K + 3) & ~(size_t)3;
        const size_t dp_base = ((size_t)2 * (2 * c->D + 3) + c->L) * 4 + 16; // + alignment slack of the candidate tables
        const size_t tab_all = (size_t)c->L * (Kp * 8 + 4), tab_one = Kp * 8 + 4;
        c->dp_plan.pd_nibble = c->K <= 16 ? 1u : 0u;
        c->dp_plan.pd_row_bytes = c->dp_plan.pd_nibble ? (c->D + 2) / 2 : (c->D + 1);
        const size_t pd_bytes = (size_t)c->L * c->dp_plan.pd_row_bytes;
        if (dp_base + tab_one > kDpSmemMax) { delete c; return KIMAD_ERR_INVALID_ARG; }
        c->dp_plan.tab_in_smem = dp_base + tab_all <= kDpSmemMax ? 1u : 0u;
        size_t used = dp_base + (c->dp_plan.tab_in_smem ? tab_all : tab_one);
        c->dp_plan.pd_in_smem = used + pd_bytes <= kDpSmemMax ? 1u : 0u;
        if (c->dp_plan.pd_in_smem) used += pd_bytes;
        c->dp_smem = used;
        c->curve_mode = o.curve_mode;
        c->policy = o.policy;
        c->cost_model = o.cost_model;
        if (c->policy == 2 && !c->dp_plan.tab_in_smem) { delete c; return KIMAD_ERR_INVALID_ARG; }
        c->sample_smem = (size_t)(2 * (1024 + 32) + 32768 + 1024 + 2 * kMaxGaps + 32 + 3 * 128) * 4;
        c->pass_a_smem = (size_t)(2 * kMaxBins + kCellTab) * 4;
        { // the sweep's runs, one CTA each: every worker's chunk list is cut into pieces of about equal element counts.
          // The sweep of a group of workers ((W + 1) / 2 of them) is one wave of CTAs (148 SMs, one CTA resident per
          // SM), or up to four waves when a run would otherwise exceed kSweepRunElems: long static runs end
          // unevenly, and later waves even that out.
            const uint32_t nch = (uint32_t)c->chunks.size();
            const uint32_t gw = (c->W + 1) / 2; // workers in the larger group (1 for a single worker)
            const uint64_t waves = std::min<uint64_t>(4, std::max<uint64_t>(1, (N * gw + 148ull * kSweepRunElems - 1) / (148ull * kSweepRunElems)));
            const uint32_t per_w = std::max<uint32_t>(1u, std::min<uint32_t>(nch, (uint32_t)((waves * 148u + gw - 1) / gw)));
            for (uint32_t w = 0; w < c->W; ++w) {
                uint64_t acc = 0;
                uint32_t g = 0, start = 0;
                for (uint32_t f = 0; f < nch; ++f) {
                    if (g + 1 < per_w && f > start && acc >= (N * (uint64_t)(g + 1)) / per_w) { c->runs.push_back(SweepRun{w, start, f}); start = f; ++g; }
                    acc += c->chunks[f].end - c->chunks[f].begin;
                }
                c->runs.push_back(SweepRun{w, start, nch});
            }
        }
        c->tiny_smem = (size_t)kTinyMax * (8 + 4);
        plan_layout(c);
        { // host image of the static tables [chunks, zero_from): attached workspaces get it in one copy
            const Layout& y = c->lay;
            c->static_image.assign(y.zero_from - y.chunks, 0);
            unsigned char* im = c->static_image.data() - y.chunks;
            std::memcpy(im + y.chunks, c->chunks.data(), c->chunks.size() * sizeof(Chunk));
            std::memcpy(im + y.layers, c->layers.data(), c->layers.size() * sizeof(LayerDesc));
            std::memcpy(im + y.ktab, c->ktab.data(), c->ktab.size() * sizeof(uint64_t));
            if (!c->reg_layers.empty()) std::memcpy(im + y.reg_layers, c->reg_layers.data(), c->reg_layers.size() * 4);
            if (!c->tiny_layers.empty()) std::memcpy(im + y.tiny_layers, c->tiny_layers.data(), c->tiny_layers.size() * 4);
            std::memcpy(im + y.reg_index, c->reg_index.data(), c->reg_index.size() * 4);
            std::memcpy(im + y.runs, c->runs.data(), c->runs.size() * sizeof(SweepRun));
            for (size_t g : c->guards)
                if (g >= y.chunks && g + kAlign <= y.zero_from) std::memset(im + g, kCanaryByte, kAlign);
        }
    } catch (const std::bad_alloc&) {
        delete c;
        return KIMAD_ERR_NOMEM;
    }
    *out = c;
    return KIMAD_OK;
}

void kimad_destroy(kimad_ctx* ctx) {
    if (ctx && ctx->have_ev)
        for (cudaEvent_t e : ctx->ev) cudaEventDestroy(e);
    if (ctx && ctx->side) {
        cudaStreamSynchronize(ctx->side);
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
        cudaStreamDestroy(ctx->side);
        for (int g = 0; g < kGroups; ++g) {
            if (ctx->gstream[g]) { cudaStreamSynchronize(ctx->gstream[g]); cudaStreamDestroy(ctx->gstream[g]); }
            if (ctx->gshort[g]) { cudaStreamSynchronize(ctx->gshort[g]); cudaStreamDestroy(ctx->gshort[g]); }
            if (ctx->glist[g]) { cudaStreamSynchronize(ctx->glist[g]); cudaStreamDestroy(ctx->glist[g]); }
            for (cudaEvent_t e : ctx->ev_list[g]) if (e) cudaEventDestroy(e);
            if (ctx->ev_done[g]) cudaEventDestroy(ctx->ev_done[g]);
            for (cudaEvent_t e : ctx->ev_hand[g]) if (e) cudaEventDestroy(e);
        }
        if (ctx->ev_go) cudaEventDestroy(ctx->ev_go);
    }
    delete ctx;
}

int kimad_debug_enable_stage_timing(kimad_ctx* c, int enable) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    if (enable && !c->have_ev) {
        for (cudaEvent_t& e : c->ev) CUDA_TRY(cudaEventCreate(&e));
        c->have_ev = true;
    }
    c->timing = enable != 0;
    return KIMAD_OK;
}

int kimad_debug_trace_step(kimad_ctx* c, const float* grads_dev, float* state_dev, const double* bandwidth_bytes_per_s,
                           double t_target_s, const kimad_packed* out, void* cuda_stream, char* text, size_t text_len) {
    if (!text || text_len == 0) return KIMAD_ERR_INVALID_ARG;
    text[0] = 0;
    if (g_launch_trace) return KIMAD_ERR_INVALID_ARG; // another traced step is being issued
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    std::vector<LaunchRec> recs;
    cudaEvent_t start = nullptr;
    CUDA_TRY(cudaEventCreate(&start));
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaEventRecord(start, s));
    g_launch_trace = &recs;
    const int rc = run_step(c, grads_dev, state_dev, bandwidth_bytes_per_s, t_target_s, out, cuda_stream, kNormal, nullptr, nullptr);
    g_launch_trace = nullptr;
    const cudaError_t sync = cudaDeviceSynchronize();
    std::vector<cudaStream_t> streams; // ordinal of a stream = order of its first launch
    size_t at = 0;
    for (const LaunchRec& r : recs) {
        float t0 = 0.f, t1 = 0.f;
        if (sync == cudaSuccess && rc == KIMAD_OK) {
            cudaEventElapsedTime(&t0, start, r.a);
            cudaEventElapsedTime(&t1, start, r.b);
            size_t si = 0;
            while (si < streams.size() && streams[si] != r.s) ++si;
            if (si == streams.size()) streams.push_back(r.s);
            if (at < text_len) {
                const int n = snprintf(text + at, text_len - at, "%-28s stream %zu  %8.3f -> %8.3f ms\n", r.name, si, t0, t1);
                if (n > 0) at += (size_t)n;
            }
        }
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    cudaEventDestroy(start);
    text[text_len - 1] = 0;
    if (sync != cudaSuccess) return KIMAD_ERR_CUDA;
    return rc;
}

int kimad_debug_set_schedule(kimad_ctx* c, int mode) {
    if (!c || mode < 0 || mode > 2) return KIMAD_ERR_INVALID_ARG;
    c->pipeline_mode = mode;
    return KIMAD_OK;
}

int kimad_debug_stage_times(kimad_ctx* c, float* host_ms) {
    if (!c || !host_ms || !c->have_ev || !c->have_last) return KIMAD_ERR_INVALID_ARG;
    CUDA_TRY(cudaDeviceSynchronize());
    for (int i = 0; i < KIMAD_N_STAGES; ++i) CUDA_TRY(cudaEventElapsedTime(&host_ms[i], c->ev[i], c->ev[i + 1]));
    return KIMAD_OK;
}

size_t kimad_workspace_bytes(const kimad_ctx* ctx) { return ctx ? ctx->lay.total : 0; }

int kimad_set_workspace(kimad_ctx* c, void* dev_ptr, size_t bytes) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    if (!dev_ptr || bytes < c->lay.total || (uintptr_t)dev_ptr % kAlign) return KIMAD_ERR_WORKSPACE;
    c->ws = static_cast<unsigned char*>(dev_ptr);
    const Layout& y = c->lay;
    CUDA_TRY(cudaMemcpy(c->ws + y.chunks, c->static_image.data(), c->static_image.size(), cudaMemcpyHostToDevice));
    // histograms, work lists and flags start at zero and are kept clean by the kernels that consume them
    CUDA_TRY(cudaMemset(c->ws + y.zero_from, 0, y.cell_tab - y.zero_from));
    { const int rc_g = fill_guards(c, c->ws, nullptr); if (rc_g != KIMAD_OK) return rc_g; }
    { const int rc_dev = prepare_device(c); if (rc_dev != KIMAD_OK) return rc_dev; }
    CUDA_TRY(cudaDeviceSynchronize());
    return KIMAD_OK;
}

int kimad_step(kimad_ctx* ctx, const float* grads_dev, float* state_dev, const double* bandwidth_bytes_per_s,
               double t_target_s, const kimad_packed* out, void* cuda_stream) {
    return run_step(ctx, grads_dev, state_dev, bandwidth_bytes_per_s, t_target_s, out, cuda_stream, kNormal, nullptr,
                    nullptr);
}

int kimad_debug_step_with_err(kimad_ctx* ctx, const float* grads_dev, float* state_dev,
                              const double* bandwidth_bytes_per_s, double t_target_s, const kimad_packed* out,
                              void* cuda_stream, const float* err_dev) {
    return run_step(ctx, grads_dev, state_dev, bandwidth_bytes_per_s, t_target_s, out, cuda_stream, kInjectErr, err_dev,
                    nullptr);
}

int kimad_debug_step_with_j(kimad_ctx* ctx, const float* grads_dev, float* state_dev,
                            const double* bandwidth_bytes_per_s, double t_target_s, const kimad_packed* out,
                            void* cuda_stream, const uint32_t* j_dev) {
    return run_step(ctx, grads_dev, state_dev, bandwidth_bytes_per_s, t_target_s, out, cuda_stream, kGivenJ, nullptr,
                    j_dev);
}

int kimad_apply_packed(const kimad_ctx* c, const kimad_packed* msg, float* est_dev, void* cuda_stream) {
    if (!c || !msg || !msg->idx || !msg->val || !msg->offs || !est_dev) return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const LayerDesc* layers = reinterpret_cast<const LayerDesc*>(c->ws + c->lay.layers);
    const dim3 grid(148 * 4, c->W);
    if (c->value_dtype == 1)
        k_apply_packed<true><<<grid, kThreads, 0, s>>>(msg->idx, msg->val, msg->offs, layers, c->L, c->cap, c->stride, est_dev);
    else
        k_apply_packed<false><<<grid, kThreads, 0, s>>>(msg->idx, msg->val, msg->offs, layers, c->L, c->cap, c->stride, est_dev);
    CUDA_TRY(cudaGetLastError());
    return KIMAD_OK;
}

int kimad_aggregate(float* x_dev, const float* est_dev, uint64_t stride, uint32_t n_workers, uint64_t n,
                    const float* weights, float gamma, void* cuda_stream) {
    if (!x_dev || !est_dev || !weights || n_workers == 0 || n_workers > KIMAD_MAX_AGG_WORKERS || stride < n)
        return KIMAD_ERR_INVALID_ARG;
    if (n == 0) return KIMAD_OK;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    AggWeights wt{};
    for (uint32_t m = 0; m < n_workers; ++m) wt.w[m] = weights[m];
    const bool vec = (reinterpret_cast<uintptr_t>(x_dev) % 16 == 0) && (reinterpret_cast<uintptr_t>(est_dev) % 16 == 0) &&
                     (stride % 4 == 0);
    const uint64_t units = vec ? (n + 3) / 4 : n;
    const uint32_t grid = (uint32_t)std::min<uint64_t>((units + kThreads - 1) / kThreads, 148ull * 16);
    if (vec)
        k_aggregate<true><<<grid, kThreads, 0, s>>>(x_dev, est_dev, stride, n_workers, n, wt, gamma);
    else
        k_aggregate<false><<<grid, kThreads, 0, s>>>(x_dev, est_dev, stride, n_workers, n, wt, gamma);
    CUDA_TRY(cudaGetLastError());
    return KIMAD_OK;
}

int kimad_get_k(kimad_ctx* c, uint32_t* host_k, void* cuda_stream) {
    if (!c || !c->have_last) return KIMAD_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    std::vector<kimad_stats> st(c->W);
    if (host_k)
        CUDA_TRY(cudaMemcpyAsync(host_k, c->last_out.k, (size_t)c->W * c->L * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaMemcpyAsync(st.data(), c->last_out.stats, c->W * sizeof(kimad_stats), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    int worst_err = 0, worst_soft = 0;
    for (const kimad_stats& x : st) {
        if (x.status < worst_err) worst_err = x.status;
        if (x.status > worst_soft) worst_soft = x.status;
    }
    return worst_err < 0 ? worst_err : worst_soft;
}

int kimad_get_k_table(const kimad_ctx* c, uint64_t* host_k_table) {
    if (!c || !host_k_table) return KIMAD_ERR_INVALID_ARG;
    std::memcpy(host_k_table, c->ktab.data(), c->ktab.size() * sizeof(uint64_t));
    return KIMAD_OK;
}

int kimad_plan_budget(const kimad_ctx* c, double bandwidth_bytes_per_s, double t_target_s, uint64_t* budget_bytes,
                      uint64_t* cells) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    const double cb = std::floor(bandwidth_bytes_per_s * t_target_s);
    const uint64_t cc = !(cb > 0.0) ? 0ull : (cb >= 18446744073709551615.0 ? ~0ull : (uint64_t)cb);
    if (budget_bytes) *budget_bytes = cc;
    if (cc >= c->full_bytes) return KIMAD_STATUS_PLATEAU;
    if (cc == 0) return KIMAD_STATUS_INFEASIBLE;
    if (cells)
        for (size_t i = 0; i < c->ktab.size(); ++i)
            cells[i] = budget_cells(candidate_bytes(c->layer_sizes[i / c->K], c->ktab[i], c->bpe, c->cost_model, nullptr), c->D, cc);
    return KIMAD_OK;
}

int kimad_debug_get_curve(kimad_ctx* c, float* host_err, uint32_t* host_tau, uint32_t* host_keep_eq,
                          uint32_t* host_shift) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    const size_t n = (size_t)c->W * c->L * c->K;
    CUDA_TRY(cudaDeviceSynchronize());
    if (host_err) CUDA_TRY(cudaMemcpy(host_err, c->ws + c->lay.err, n * 4, cudaMemcpyDeviceToHost));
    if (host_tau) CUDA_TRY(cudaMemcpy(host_tau, c->ws + c->lay.tau, n * 4, cudaMemcpyDeviceToHost));
    if (host_keep_eq) CUDA_TRY(cudaMemcpy(host_keep_eq, c->ws + c->lay.keep_eq, n * 4, cudaMemcpyDeviceToHost));
    if (host_shift) CUDA_TRY(cudaMemcpy(host_shift, c->ws + c->lay.shift, n * 4, cudaMemcpyDeviceToHost));
    return KIMAD_OK;
}

int kimad_debug_get_selection(kimad_ctx* c, uint32_t* host_tau, uint32_t* host_keep_eq) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    const size_t n = (size_t)c->W * c->L;
    std::vector<Sel> sel(n);
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(sel.data(), c->ws + c->lay.sel, n * sizeof(Sel), cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < n; ++i) {
        if (host_tau) host_tau[i] = sel[i].tau;
        if (host_keep_eq) host_keep_eq[i] = sel[i].keep_eq;
    }
    return KIMAD_OK;
}

int kimad_debug_get_band_meta(kimad_ctx* c, uint32_t* host_meta) {
    if (!c || !host_meta) return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    CUDA_TRY(cudaDeviceSynchronize());
    CUDA_TRY(cudaMemcpy(host_meta, c->ws + c->lay.meta, (size_t)c->W * c->reg_layers.size() * sizeof(BandMeta),
                        cudaMemcpyDeviceToHost));
    return KIMAD_OK;
}

int kimad_debug_exact_path_layers(kimad_ctx* c, uint64_t* host_count) {
    if (!c || !host_count) return KIMAD_ERR_INVALID_ARG;
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    CUDA_TRY(cudaDeviceSynchronize());
    for (uint32_t i = 0; i < 6 + c->K; ++i) host_count[i] = 0;
    for (int g = 0; g < kGroups; ++g) { // every group of workers keeps counters of its own
        FbList f{};
        CUDA_TRY(cudaMemcpy(&f, c->ws + c->lay.fb + g * align_up(sizeof(FbList)), sizeof(FbList), cudaMemcpyDeviceToHost));
        host_count[0] += f.total_layers;
        for (int i = 0; i < 4; ++i) host_count[1 + i] += f.why[i];
        host_count[5] += f.refined;
        for (uint32_t j = 0; j < c->K; ++j) host_count[6 + j] += f.loose_j[j];
    }
    return KIMAD_OK;
}

int kimad_debug_check(kimad_ctx* c, uint32_t* failed_checks, uint32_t* damaged_canaries) {
    if (!c) return KIMAD_ERR_INVALID_ARG;
    if (failed_checks) *failed_checks = 0;
    if (damaged_canaries) *damaged_canaries = 0;
#ifdef KIMAD_CHECKED
    if (!c->ws) return KIMAD_ERR_WORKSPACE;
    CUDA_TRY(cudaDeviceSynchronize());
    unsigned int word = 0;
    CUDA_TRY(cudaMemcpyFromSymbol(&word, g_kimad_check_word, sizeof(word)));
    if (failed_checks) *failed_checks = word;
    uint32_t bad = 0;
    unsigned char buf[kAlign];
    for (size_t g : c->guards) {
        CUDA_TRY(cudaMemcpy(buf, c->ws + g, kAlign, cudaMemcpyDeviceToHost));
        for (size_t i = 0; i < kAlign; ++i)
            if (buf[i] != (unsigned char)kCanaryByte) { ++bad; break; }
    }
    if (damaged_canaries) *damaged_canaries = bad;
    return 1;
#else
    return 0;
#endif
}

uint64_t kimad_launch_count(const kimad_ctx* ctx) { return ctx ? ctx->launches : 0; }

// ---------------------------------------------------------------------------------------------------
// Bandwidth monitor: windowed throughput of the reported transfers with exponential smoothing (host only)
// ---------------------------------------------------------------------------------------------------
} // extern "C"
struct kimad_monitor {
    std::vector<uint64_t> bytes;
    std::vector<double> secs;
    uint32_t window = 1, head = 0, filled = 0;
    double alpha = 1.0, est = 0.0;
    bool any = false;
};
extern "C" {

int kimad_monitor_create(kimad_monitor** out, uint32_t window, double alpha) {
    if (!out) return KIMAD_ERR_INVALID_ARG;
    *out = nullptr;
    if (window == 0 || window > 65536 || !(alpha > 0.0) || !(alpha <= 1.0)) return KIMAD_ERR_INVALID_ARG;
    kimad_monitor* m = new (std::nothrow) kimad_monitor();
    if (!m) return KIMAD_ERR_NOMEM;
    try {
        m->bytes.assign(window, 0);
        m->secs.assign(window, 0.0);
    } catch (const std::bad_alloc&) {
        delete m;
        return KIMAD_ERR_NOMEM;
    }
    m->window = window;
    m->alpha = alpha;
    *out = m;
    return KIMAD_OK;
}

void kimad_monitor_destroy(kimad_monitor* m) { delete m; }

int kimad_monitor_observe(kimad_monitor* m, uint64_t bytes, double seconds) {
    if (!m || !(seconds > 0.0) || !std::isfinite(seconds)) return KIMAD_ERR_INVALID_ARG;
    m->bytes[m->head] = bytes;
    m->secs[m->head] = seconds;
    m->head = (m->head + 1) % m->window;
    if (m->filled < m->window) ++m->filled;
    // sums are taken afresh over the window, oldest entry first: no drift from adding and removing terms
    double sb = 0.0, ss = 0.0;
    const uint32_t first = (m->head + m->window - m->filled) % m->window;
    for (uint32_t i = 0; i < m->filled; ++i) {
        const uint32_t at = (first + i) % m->window;
        sb += (double)m->bytes[at];
        ss += m->secs[at];
    }
    const double windowed = sb / ss;
    m->est = m->any ? m->alpha * windowed + (1.0 - m->alpha) * m->est : windowed;
    m->any = true;
    return KIMAD_OK;
}

double kimad_monitor_estimate(const kimad_monitor* m) { return m && m->any ? m->est : 0.0; }

// ---------------------------------------------------------------------------------------------------
// Allocation-free variant of kimad_step: the scratch is a fixed array inside the library's device image.
// ---------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_builtin_scratch[KIMAD_BUILTIN_SCRATCH_BYTES];
// Host code may not pass the symbol itself to a kernel: its device address is looked up once per device.
static unsigned char* g_builtin_ptr[KIMAD_BUILTIN_MAX_DEVICES] = {};

int kimad_step_builtin_scratch(kimad_ctx* c, const float* grads_dev, float* state_dev, const double* bandwidth_bytes_per_s,
                               double t_target_s, const kimad_packed* out, void* cuda_stream) {
    // arguments first: nothing of the shared array is touched by a call that is going to be refused
    if (!c || !grads_dev || !state_dev || !bandwidth_bytes_per_s || !out || !out->idx || !out->val || !out->offs || !out->k ||
        !out->j || !out->stats || !(t_target_s >= 0.0))
        return KIMAD_ERR_INVALID_ARG;
    if (c->lay.total > (size_t)KIMAD_BUILTIN_SCRATCH_BYTES) return KIMAD_ERR_TOO_LARGE;
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= KIMAD_BUILTIN_MAX_DEVICES) return KIMAD_ERR_INVALID_ARG;
    if (!g_builtin_ptr[dev]) { // first call on this device (it is the current one)
        void* p = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&p, g_builtin_scratch));
        g_builtin_ptr[dev] = static_cast<unsigned char*>(p);
    }
    { const int rc_dev = prepare_device(c); if (rc_dev != KIMAD_OK) return rc_dev; } // once per device / per context
    unsigned char* ws = g_builtin_ptr[dev];
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call (of any context) left: bring in this context's tables (one block)
    // and clear everything that has to start at zero, in stream order before the kernels.
    const Layout& y = c->lay;
    CUDA_TRY(cudaMemcpyAsync(ws + y.chunks, c->static_image.data(), c->static_image.size(), cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaMemsetAsync(ws + y.zero_from, 0, y.cell_tab - y.zero_from, s));
    { const int rc_g = fill_guards(c, ws, s); if (rc_g != KIMAD_OK) return rc_g; }
    unsigned char* caller_ws = c->ws; // the context's own workspace (if any) is left untouched
    c->ws = ws;
    const int rc = run_step(c, grads_dev, state_dev, bandwidth_bytes_per_s, t_target_s, out, cuda_stream, kNormal, nullptr,
                            nullptr);
    c->ws = caller_ws;
    return rc;
}

const char* kimad_strerror(int code) {
    switch (code) {
        case KIMAD_OK: return "ok";
        case KIMAD_STATUS_INFEASIBLE: return "budget below the smallest candidates: candidate 0 taken everywhere";
        case KIMAD_STATUS_PLATEAU: return "budget covers the largest candidate of every layer";
        case KIMAD_ERR_INVALID_ARG: return "invalid argument";
        case KIMAD_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
        case KIMAD_ERR_CAPACITY: return "selected entries exceed max_packed_elems";
        case KIMAD_ERR_NONFINITE: return "non-finite value in grad - state";
        case KIMAD_ERR_TIMEOUT: return "device wait timed out";
        case KIMAD_ERR_CUDA: return "CUDA runtime error";
        case KIMAD_ERR_NOMEM: return "host allocation failed";
        case KIMAD_ERR_TOO_LARGE: return "problem needs more scratch than the built-in array of kimad_step_builtin_scratch";
        default: return "unknown code";
    }
}

} // extern "C"
