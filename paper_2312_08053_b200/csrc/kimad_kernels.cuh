// Device code of the Kimad+ compression pass for sm_100a: helpers shared by all stages, the exact radix
// resolve kernels and the knapsack DP.
//
// Stage map of one step (letters as in include/kimad.h; file in brackets):
//   k_sample        (a)+(b) per (worker, layer): stratified sample of |grad - g| -> for every candidate k_j the
//                   band of 16-bit key prefixes that can hold its threshold -> bins and the cell table [kimad_curve.cuh]
//   k_pass_a        (a)+(b) the sweep: d = grad - g (Section 3 footnote, Eq. 6), bin = table(key(d)), count and
//                   exact integer sum of squares per bin in shared memory; one byte per element (a monotone code
//                   of its bin) goes to scratch, d itself is never stored                         [kimad_curve.cuh]
//   k_resolve_a     (b) Eq. 4 / the "Errors" matrix of Algorithm 3: err_l(k_j) from the bins, certified to the
//                   curve tolerance; layers that fail the certificate are handed to the exact path [kimad_curve.cuh]
//   k_tiny_exact    (b) layers of at most 4096 elements, sorted in shared memory                 [kimad_curve.cuh]
//   k_refine_hist, k_refine_resolve
//                   (b) candidates whose certified bound is too loose: one more look at their bin (usually none)
//   k_fb_hist1, k_fb_hist23<2|3>, k_resolve1, k_resolve23<2|3>, k_rebuild_slots
//                   (b) exact 11+10+10-bit radix select over the handed-over layers (usually none)
//                                                                          [kimad_curve.cuh, this file]
//   k_dp            (c) Algorithm 3 on the budget axis (Eq. 2, Eq. 3, Section 3.2), one CTA per worker; also the
//                   uniform-ratio policies and the error-axis reading                            [this file]
//   k_sel_count, k_sel_resolve(_r2), k_sel_count_r2, k_sel_recount, k_sel_slices, k_sel_scan
//                   (d) exact threshold and per-slice output offsets at the chosen k             [kimad_select.cuh]
//   k_sel_write     (e)+(f) ordered (index, value) pack and g += C(d) (Algorithm 1, Eq. 6)       [kimad_select.cuh]
//   k_apply_packed, k_aggregate   receiving side and model step (Algorithm 1, server lines)      [kimad_receiver.cuh]
//
// Nothing here is a dense contraction, so there is no tensor-core path.  The sweep runs at 83-90 % of the measured HBM
// copy rate on its 9 bytes per element (one shared-memory table read and two shared-memory atomics per element keep it
// from the rest); the counting and write sweeps are bound by HBM on large layers and by load latency on small ones.
// After the sample kernel the workers go through the stages as two groups on streams of their own (kimad_api.cu).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kimad_common.h"

namespace kimad {

constexpr int kThreads = 256;
constexpr int kL1Bins = 2048;  // 8 exponent bits + 3 mantissa bits
constexpr int kL23Bins = 1024; // 10 bits each

__device__ __forceinline__ uint32_t key_of(float d) { return __float_as_uint(d) & 0x7fffffffu; }

// Kernels launched with programmatic stream serialisation may be scheduled before their predecessor in the
// stream has finished (which hides their launch latency); they wait here, before touching anything it wrote.
// A no-op for an ordinary launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Aligned view of a chunk for 128-bit loads of the inputs (quads of elements) and of the code plane (sixteen
// codes): units start at a0 = begin & ~15; only the first and the last ones can be partial.  All offsets are
// 32-bit and relative to a0.
struct ChunkView {
    uint64_t a0;
    uint32_t first, len; // valid element offsets are [first, len)
    __device__ __forceinline__ explicit ChunkView(const Chunk& ch)
        : a0(ch.begin & ~15ull), first((uint32_t)(ch.begin - (ch.begin & ~15ull))), len((uint32_t)(ch.end - (ch.begin & ~15ull))) {}
    __device__ __forceinline__ uint32_t quads() const { return (len + 3) >> 2; }
    __device__ __forceinline__ bool quad_full(uint32_t q) const { return 4 * q >= first && 4 * q + 4 <= len; }
};

// The difference vector d = grad - g is never stored.  The sweep leaves one BYTE per element (u8 [W][dstride]): a
// 7-bit code that never decreases with the magnitude key inside a layer -- the element's histogram bin divided by
// a power of two for layers swept with a histogram, the upper seven bits of the key otherwise (code_of_key).  The
// counting sweep of the select stage classifies an entry as above or below the threshold by its code and needs the
// exact value only for the entries whose code equals the threshold's; whoever needs an exact d recomputes the one
// subtraction from the inputs (the estimator is not written before the write sweep, and there every element is
// read before it is updated).
struct DSource {
    uint8_t* code;
    const float* grads;
    const float* state;
    uint64_t stride; // elements between workers in grads / state
};
struct DView { // one worker's data at a chunk's aligned start
    const uint8_t* code;
    const float* gr;
    const float* st;
    __device__ __forceinline__ DView(const DSource& p, uint32_t w, uint64_t dstride, uint64_t a0)
        : code(p.code + (size_t)w * dstride + a0), gr(p.grads + (size_t)w * p.stride + a0), st(p.state + (size_t)w * p.stride + a0) {}
    __device__ __forceinline__ float at(uint32_t e) const { return __fsub_rn(gr[e], st[e]); }
};
// code of layers without a histogram: the upper seven bits of the 31-bit key
__device__ __forceinline__ uint32_t code_of_key(uint32_t key) { return key >> 24; }
// the lowest bytes of four words as one word (element 0 in the lowest byte)
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}
// the codes of a quad of keys of a layer without a histogram (the highest byte of every key)
__device__ __forceinline__ uint32_t pack_key_codes(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
    return __byte_perm(__byte_perm(k0, k1, 0x0073), __byte_perm(k2, k3, 0x0073), 0x5410);
}

// ------------------------------------------------------------------------------------------------
// block-wide exclusive scans (256 threads), result valid in every thread; `total` optional
// ------------------------------------------------------------------------------------------------
template <typename T, int NT = kThreads>
__device__ __forceinline__ T block_excl_scan(T v, T* s_warp /* [NT / 32] */, T* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    T x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    __syncthreads(); // s_warp may still be read from a previous call
    if (lane == 31) s_warp[wid] = x;
    __syncthreads();
    T base = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < NT / 32; ++i) {
        T t = s_warp[i];
        if (i < wid) base += t;
        tot += t;
    }
    if (total) *total = tot;
    // the lane's exclusive value is taken from its left neighbour, not as inclusive - own: a subtraction would
    // cancel the small terms of a floating-point scan whose values span many orders of magnitude
    T ex = __shfl_up_sync(0xffffffffu, x, 1);
    if (lane == 0) ex = 0;
    return base + ex;
}

// ------------------------------------------------------------------------------------------------
// (a) difference + level-1 histogram
// ------------------------------------------------------------------------------------------------
// Squares are accumulated as exact integers.  Every histogram bin holds keys of one exponent e, so
// value^2 = M^2 * 4^(max(e,1)-150) with M the 24-bit significand (no hidden bit for subnormals);
// bins sum (M^2 >> 16), a 32-bit quantity (truncation <= 2^-30 relative).  Integer adds commute, so
// the sums -- and with them the error curve -- do not depend on the order the atomics land in.
__device__ __forceinline__ uint64_t sq_fixed(uint32_t key) {
    const uint32_t e = key >> 23, mant = key & 0x7fffffu;
    const uint32_t M = e ? (mant | 0x800000u) : mant;
    return ((uint64_t)M * (uint64_t)M) >> 16;
}
// scale that turns a bin's integer sum back into a sum of squared values; e = exponent field of the bin
__device__ __forceinline__ double sq_scale(uint32_t e) { // 2^(2 (max(e,1) - 150) + 16), always a normal double
    const int x = 2 * ((int)(e ? e : 1u) - 150) + 16;
    return __longlong_as_double((long long)(x + 1023) << 52);
}

// ------------------------------------------------------------------------------------------------
// (b) resolve: candidates -> bins.  One CTA per (worker, layer).
// ------------------------------------------------------------------------------------------------
// In-place: on return s_incl[p] (p = position counted from the TOP bin, p = NB-1-bin) holds the
// inclusive count of keys in bins >= that bin; s_below[bin] holds the sum of ss over bins < bin.
template <int NB>
__device__ __forceinline__ void scan_bins(uint32_t* s_incl /* in: counts by position */, double* s_below /* in: ss by bin */,
                                          uint32_t* s_w32, double* s_w64) {
    constexpr int PER = NB / kThreads;
    static_assert(PER % 4 == 0, "16-byte shared-memory accesses");
    uint32_t loc[PER];
    uint32_t sum = 0;
    uint4* v4 = reinterpret_cast<uint4*>(s_incl + threadIdx.x * PER);
#pragma unroll
    for (int i = 0; i < PER / 4; ++i) {
        const uint4 t = v4[i];
        loc[4 * i] = t.x; loc[4 * i + 1] = t.y; loc[4 * i + 2] = t.z; loc[4 * i + 3] = t.w;
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) sum += loc[i];
    uint32_t ex = block_excl_scan<uint32_t>(sum, s_w32, nullptr);
#pragma unroll
    for (int i = 0; i < PER; ++i) { ex += loc[i]; loc[i] = ex; }
#pragma unroll
    for (int i = 0; i < PER / 4; ++i) v4[i] = make_uint4(loc[4 * i], loc[4 * i + 1], loc[4 * i + 2], loc[4 * i + 3]);
    if (s_below) {
        double dl[PER];
        double ds = 0.0;
        double2* d2 = reinterpret_cast<double2*>(s_below + threadIdx.x * PER);
#pragma unroll
        for (int i = 0; i < PER / 2; ++i) { const double2 t = d2[i]; dl[2 * i] = t.x; dl[2 * i + 1] = t.y; }
#pragma unroll
        for (int i = 0; i < PER; ++i) ds += dl[i];
        double de = block_excl_scan<double>(ds, s_w64, nullptr);
#pragma unroll
        for (int i = 0; i < PER; ++i) { const double t = dl[i]; dl[i] = de; de += t; }
#pragma unroll
        for (int i = 0; i < PER / 2; ++i) d2[i] = make_double2(dl[2 * i], dl[2 * i + 1]);
    }
    __syncthreads();
}

// first position p (0 = top bin) whose inclusive count reaches `rank` (1-based)
template <int NB>
__device__ __forceinline__ int find_pos(const uint32_t* s_incl, uint32_t rank) {
    int lo = 0, hi = NB - 1;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_incl[mid] >= rank) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// The exact radix kernels below run over the list of layers handed over in this step (usually empty).
struct FbList { // layers handed to the exact radix path in this step, and their chunks
    uint32_t n_chunks;
    uint32_t n_layers;
    uint32_t total_layers; // never reset: how many layers were handed over since the workspace was attached
    uint32_t why[5];       // never reset: ... because 0: forced, 1: bands too wide for the tables, 2: threshold
                           // outside its band, 3: error bound too loose
    uint32_t loose_j[KIMAD_MAX_RATIOS + 1]; // never reset: which candidate's bound was too loose
    // layers whose only defect is a loose bound are refined instead: one more look at the entries of the bins that
    // hold the loose candidates' thresholds (k_refine_hist, k_refine_resolve)
    uint32_t rf_chunks;
    uint32_t rf_layers;
    uint32_t refined; // never reset: layers that took the refinement
};
// A candidate of a refined layer: its threshold lies in the bin [klo, klo + 2^shift), which holds cb entries of which
// the `drop` smallest are not kept; `below` = the squares of everything below the bin.  shift = kNoRefine: this
// candidate's curve entry is final.
struct RefineCand {
    uint32_t klo, shift, cb, drop;
    double below;
};
constexpr uint32_t kNoRefine = 0xffffffffu;

__global__ void __launch_bounds__(kThreads)
k_resolve1(const FbList* __restrict__ fb, const uint2* __restrict__ fb_layers, uint32_t* __restrict__ g_cnt,
           unsigned long long* __restrict__ g_ss, const KTab ktab, uint32_t L, uint32_t K,
           Cand* __restrict__ cands, SlotTab* __restrict__ slots) {
    pdl_wait();
    __shared__ __align__(16) uint32_t s_incl[kL1Bins];
    __shared__ __align__(16) double s_below[kL1Bins];
    __shared__ uint32_t s_w32[8];
    __shared__ double s_w64[8];
  for (uint32_t it = blockIdx.x; it < fb->n_layers; it += gridDim.x) {
    const uint32_t l = fb_layers[it].y, w = fb_layers[it].x;
    const size_t wl = (size_t)w * L + l;
    uint32_t* gc = g_cnt + wl * kL1Bins;
    unsigned long long* gs = g_ss + wl * kL1Bins;
    {
        constexpr int PER = kL1Bins / kThreads;
        uint32_t c[PER];
        unsigned long long g[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) { c[i] = gc[threadIdx.x + i * kThreads]; g[i] = gs[threadIdx.x + i * kThreads]; }
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int b = threadIdx.x + i * kThreads;
            s_incl[kL1Bins - 1 - b] = c[i];
            s_below[b] = (double)g[i] * sq_scale((uint32_t)b >> 3);
            gc[b] = 0; // leave the histogram clean for the next step
            gs[b] = 0ull;
        }
    }
    __syncthreads();
    scan_bins<kL1Bins>(s_incl, s_below, s_w32, s_w64);
    Cand* cd = cands + wl * K;
    for (uint32_t j = threadIdx.x; j < K; j += kThreads) {
        const uint32_t k = (uint32_t)ktab.at(w, (size_t)l * K + j);
        const int p = find_pos<kL1Bins>(s_incl, k);
        const uint32_t above = p ? s_incl[p - 1] : 0u;
        Cand c;
        c.prefix = (uint32_t)(kL1Bins - 1 - p);
        c.rank = k - above;
        c.gt = above;
        c.err_low = s_below[kL1Bins - 1 - p];
        c.slot = 0;
        cd[j] = c;
    }
    __syncthreads();
    if (threadIdx.x == 0) { // distinct prefixes, in candidate order (prefix is non-increasing in j)
        SlotTab& stab = slots[wl];
        uint32_t ns = 0;
        for (uint32_t j = 0; j < K; ++j) {
            if (ns == 0 || stab.prefix[ns - 1] != cd[j].prefix) stab.prefix[ns++] = cd[j].prefix;
            cd[j].slot = ns - 1;
        }
        stab.n = ns;
    }
    __syncthreads();
  }
}

// LEVEL 2: refine inside a level-1 bin; LEVEL 3: inside a (level-1, level-2) bin.
// One CTA per (layer, worker, slot).
template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_resolve23(const FbList* __restrict__ fb, const uint2* __restrict__ fb_layers, uint32_t* __restrict__ g_cnt,
            unsigned long long* __restrict__ g_ss, uint32_t L, uint32_t K, Cand* __restrict__ cands,
            const SlotTab* __restrict__ slots, float* __restrict__ err_out, uint32_t* __restrict__ tau_out,
            uint32_t* __restrict__ keep_eq_out, uint32_t* __restrict__ shift_out) {
    pdl_wait();
    __shared__ __align__(16) uint32_t s_incl[kL23Bins];
    __shared__ __align__(16) double s_below[kL23Bins];
    __shared__ uint32_t s_w32[8];
    __shared__ double s_w64[8];
  for (uint32_t it = blockIdx.x; it < fb->n_layers; it += gridDim.x) {
    const uint32_t l = fb_layers[it].y, w = fb_layers[it].x, s = blockIdx.z;
    const size_t wl = (size_t)w * L + l;
    const SlotTab& stab = slots[wl];
    if (s >= stab.n) continue;
    Cand* cd = cands + wl * K;
    uint32_t* gc = g_cnt + (wl * K + s) * kL23Bins;
    unsigned long long* gs = g_ss + (wl * K + s) * kL23Bins;
    const uint32_t prefix = stab.prefix[s];
    {
        constexpr int PER = kL23Bins / kThreads;
        uint32_t cc[PER];
        unsigned long long g[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            cc[i] = gc[threadIdx.x + i * kThreads];
            g[i] = LEVEL == 2 ? gs[threadIdx.x + i * kThreads] : 0ull;
        }
        const double scale = sq_scale(prefix >> 3); // LEVEL 2: prefix = level-1 bin (8 exponent + 3 mantissa bits)
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            const int b = threadIdx.x + i * kThreads;
            s_incl[kL23Bins - 1 - b] = cc[i];
            gc[b] = 0;
            if (LEVEL == 2) {
                s_below[b] = (double)g[i] * scale;
                gs[b] = 0ull;
            } else { // all 31 bits known: the bin's sum of squares is count * value^2
                const double v = (double)__uint_as_float((prefix << 10) | (uint32_t)b);
                s_below[b] = (double)cc[i] * v * v;
            }
        }
    }
    __syncthreads();
    scan_bins<kL23Bins>(s_incl, s_below, s_w32, s_w64);
    for (uint32_t j = threadIdx.x; j < K; j += kThreads) {
        Cand c = cd[j];
        if (c.slot != s) continue;
        const int p = find_pos<kL23Bins>(s_incl, c.rank);
        const uint32_t above = p ? s_incl[p - 1] : 0u;
        const uint32_t bin = (uint32_t)(kL23Bins - 1 - p);
        c.prefix = (prefix << 10) | bin;
        c.gt += above;
        c.err_low += s_below[bin];
        if (LEVEL == 2) {
            c.rank -= above;
            cd[j] = c;
        } else {
            const uint32_t eq = s_incl[p] - above;
            const uint32_t keep = c.rank - above; // 1 <= keep <= eq
            const double v = (double)__uint_as_float(c.prefix);
            const double e = c.err_low + (double)(eq - keep) * v * v;
            err_out[wl * K + j] = (float)e;
            tau_out[wl * K + j] = c.prefix;
            keep_eq_out[wl * K + j] = keep;
            shift_out[wl * K + j] = 0;
        }
    }
    __syncthreads();
  }
}

// After digit 2: new slots = distinct 21-bit prefixes (non-increasing in j).  One thread per (worker, layer).
__global__ void __launch_bounds__(kThreads)
k_rebuild_slots(const FbList* __restrict__ fb, const uint2* __restrict__ fb_layers, uint32_t L, uint32_t K,
                Cand* __restrict__ cands, SlotTab* __restrict__ slots) {
    pdl_wait();
    const uint32_t it = blockIdx.x * kThreads + threadIdx.x;
    if (it >= fb->n_layers) return;
    const size_t wl = (size_t)fb_layers[it].x * L + fb_layers[it].y;
    Cand* cd = cands + (size_t)wl * K;
    SlotTab& stab = slots[wl];
    uint32_t n2 = 0;
    for (uint32_t j = 0; j < K; ++j) {
        const uint32_t pfx = cd[j].prefix;
        if (n2 == 0 || stab.prefix[n2 - 1] != pfx) stab.prefix[n2++] = pfx;
        cd[j].slot = n2 - 1;
    }
    stab.n = n2;
}

// ------------------------------------------------------------------------------------------------
// What the sample kernel leaves per (worker, regular layer) for the sweep (details in kimad_curve.cuh)
// ------------------------------------------------------------------------------------------------
constexpr int kCellTab = 4096; // entries of the cell table: the window of cells from the lowest to the highest band
                               // and one entry on either side
struct BandMeta {
    uint32_t n_bins;
    uint32_t n_cells; // entries of the cell table in use
    uint32_t flagged; // != 0: this layer takes the exact radix path in this step (and is swept without a histogram)
    uint32_t n_gaps;  // gap regions (when flagged: detail of the misfit)
};
// entry of the cell table: base << 5 | shift (base signed): the bin of a key is base + (key >> shift).
// window of a layer: {cell of the first entry, cell of the last entry, log2 of the keys per entry, log2 of the bins
// per code of the byte plane (bits 0..4) | 256 when the sweep leaves the layer's exact zeros out of its histogram}
struct CodeSpace { // how the sweep coded the elements of one (worker, layer)
    const uint32_t* reg_index; // [L], 0xffffffff: tiny layer
    const BandMeta* meta;      // [W][R]
    const uint32_t* cell_tab;  // [W][R][kCellTab]
    const int4* cell_win;      // [W][R]
    uint32_t R;
    // code of a key of layer l of worker w, as the sweep wrote it for every element of that layer
    __device__ __forceinline__ uint32_t code(uint32_t w, uint32_t l, uint32_t key) const {
        const uint32_t r = reg_index[l];
        if (r == 0xffffffffu) return key >> 24;
        const size_t wr = (size_t)w * R + r;
        if (meta[wr].flagged) return key >> 24;
        const int4 win = cell_win[wr];
        const uint32_t e = cell_tab[wr * kCellTab + (size_t)(min(max((int)(key >> win.z), win.x), win.y) - win.x)];
        return (uint32_t)(((int)e >> 5) + (int)(key >> (e & 31u))) >> (win.w & 31);
    }
};

// ------------------------------------------------------------------------------------------------
// (c) knapsack DP over the budget axis, one CTA per worker
// ------------------------------------------------------------------------------------------------
struct DpBudgets { uint64_t c[kDpWorkersPerLaunch]; };

constexpr int kDpThreads = 512;
constexpr int kDpCells = 2; // budget cells per thread
constexpr int kDpMaxChain = 16;                // layers carried through one barrier interval
constexpr uint32_t kDpSameCells = 0x80000000u; // flags kept beside a layer's usable-candidate count
constexpr uint32_t kDpChain = 0x40000000u;     // same cells, finite errors that do not increase with j
constexpr uint32_t kDpInner = 0x20000000u;     // layer of a chained run that is not the run's last

// Shared-memory plan of k_dp (host computes the same sizes):
//   two rows of (D+2) +inf followed by D+1 values, f32 | j[L] u32 | usable[L or 1] u32 |
//   units[(L or 1) * Kp] u32, err[(L or 1) * Kp] f32, Kp = K rounded up to 4 | PD
// The +inf margin in front of each row lets prev[b - u] be read without a bounds test for every u <= D+1
// (an unusable candidate has u = D+1).  PD holds the winning candidate of every (layer, cell): a nibble
// when K <= 16, else a byte; it lives in shared memory when it fits, else in the caller's workspace.
struct DpPlan {
    uint32_t tab_in_smem; // candidate tables preloaded for all layers (else one layer at a time)
    uint32_t pd_in_smem;
    uint32_t pd_nibble;
    uint32_t pd_row_bytes;
};

// mode 0: DP (Kimad+); mode 1: candidates given (j_in); mode 2: one candidate index for all layers, the
// largest whose total size fits the budget (Kimad on the grid, Section 3.1); mode 3: Algorithm 3 read with the
// discretised error as the axis and the size as the value (needs plan.tab_in_smem); mode 4: the table holds, per
// worker, the single candidate of the ratio fitted to the budget (k_fit_ratio): nothing to search.
// cost_model 1: a candidate whose sparse size reaches the layer's dense size is sent densely (candidate_bytes).
__global__ void __launch_bounds__(kDpThreads)
k_dp(DpBudgets budgets, uint32_t w_base, uint32_t W, uint32_t L, uint32_t K, uint32_t D, uint32_t bpe,
     uint64_t full_bytes, uint64_t cap, uint32_t check_finite, int mode, uint32_t cost_model, DpPlan plan,
     const LayerDesc* __restrict__ layers, const KTab ktab, const float* __restrict__ err, const uint32_t* __restrict__ tau,
     const uint32_t* __restrict__ keep_eq, const uint32_t* __restrict__ shift /* may be null: all exact */,
     const uint32_t* __restrict__ j_in, uint32_t* __restrict__ flags,
     uint8_t* __restrict__ pd_global, Sel* __restrict__ sel, uint32_t* __restrict__ out_k,
     uint32_t* __restrict__ out_j, uint64_t* __restrict__ out_offs, kimad_stats* __restrict__ out_stats,
     uint32_t* __restrict__ out_dense /* may be null */, const CodeSpace codes,
     uint32_t when /* 0: always; 1: only if no layer is listed for refinement or the exact path; 2: only if one is */,
     const FbList* __restrict__ lists) {
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const uint32_t w = w_base + blockIdx.x;
    if (w >= W) return;
    if (when) {
        // a layer listed for refinement may move on to the exact path's list while this kernel runs, but then the
        // refinement's list alone decides
        const bool listed = lists->rf_layers != 0u || lists->n_layers != 0u;
        if (listed != (when == 2u)) return;
    }
    const uint64_t c = budgets.c[blockIdx.x];
    const uint32_t row = D + 1, pad = D + 2, rowp = row + pad, Kp = (K + 3) & ~3u;
    const float kInf = __int_as_float(0x7f800000);
    float* rows = reinterpret_cast<float*>(smem_raw);
    float* prev = rows + pad;          // prev[-pad .. -1] = +inf
    float* cur = rows + rowp + pad;
    uint32_t* s_j = reinterpret_cast<uint32_t*>(rows + 2 * rowp); // [L]
    const uint32_t ltab = plan.tab_in_smem ? L : 1;
    uint32_t* s_usable = s_j + L;                                 // [ltab] candidates that fit into D cells
    uint32_t* s_units = s_usable + ltab;                          // [ltab * Kp], 16-byte aligned (read four at a time)
    s_units += (4u - ((2u * rowp + L + ltab) & 3u)) & 3u;
    float* s_err = reinterpret_cast<float*>(s_units + ltab * Kp); // [ltab * Kp]
    uint8_t* pd = plan.pd_in_smem ? reinterpret_cast<uint8_t*>(s_err + ltab * Kp)
                                  : pd_global + (size_t)w * L * plan.pd_row_bytes;
    __shared__ float s_redv[32];
    __shared__ uint32_t s_redb[32];
    __shared__ int s_status;

    const float* e_w = err + (size_t)w * L * K;
    const uint32_t fl = flags[w];
    int status = KIMAD_OK;
    if (check_finite && (fl & 1u)) status = KIMAD_ERR_NONFINITE;

    if (status == KIMAD_OK) {
        if (mode == 1) {
            for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = min(j_in[(size_t)w * L + l], K - 1);
        } else if (c >= full_bytes) {
            status = KIMAD_STATUS_PLATEAU;
            for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = K - 1;
        } else if (c == 0) {
            status = KIMAD_STATUS_INFEASIBLE;
            for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = 0;
        } else if (mode == 2) {
            // total size of candidate j over the layers, one thread per j; sizes ascend with j
            __shared__ uint32_t s_fit; // number of candidates that fit
            if (threadIdx.x == 0) s_fit = 0;
            __syncthreads();
            for (uint32_t j = threadIdx.x; j < K; j += blockDim.x) {
                uint64_t bytes = 0;
                for (uint32_t l = 0; l < L; ++l) bytes += candidate_bytes(layers[l].n, ktab.at(w, (size_t)l * K + j), bpe, cost_model, nullptr);
                if (bytes <= c) atomicMax(&s_fit, j + 1);
            }
            __syncthreads();
            const uint32_t fit = s_fit;
            if (fit == 0) status = KIMAD_STATUS_INFEASIBLE;
            for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = fit ? fit - 1 : 0;
        } else if (mode == 4) {
            for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = 0; // feasibility is decided on the totals below
        } else if (mode == 3) {
            // Error axis: E_max = sum_l err_{l,0} (binary64, layers in order), cells e_{l,j} = floor(err D / E_max),
            // value = fewest kept entries for a total of exactly e cells; answer = lowest e whose value fits c.
            __shared__ double s_emax;
            __shared__ uint32_t s_best;
            uint32_t* prow = reinterpret_cast<uint32_t*>(rows);
            uint32_t* pv = prow + pad;
            uint32_t* cu = prow + rowp + pad;
            uint32_t* s_kk = reinterpret_cast<uint32_t*>(s_err);
            const uint32_t kNone = 0xffffffffu;
            if (threadIdx.x == 0) {
                double e = 0.0;
                for (uint32_t l = 0; l < L; ++l) e = __dadd_rn(e, (double)e_w[(size_t)l * K]);
                s_emax = e;
                s_best = kNone;
            }
            __syncthreads();
            const double emax = s_emax;
            for (uint32_t i = threadIdx.x; i < L * Kp; i += blockDim.x) {
                const uint32_t l = i / Kp, j = i % Kp;
                uint32_t u = D + 1, kk = 0; // padding reads the margin
                if (j < K) {
                    const double q = emax > 0.0 ? floor(__ddiv_rn(__dmul_rn((double)e_w[(size_t)l * K + j], (double)D), emax)) : 0.0;
                    u = q > (double)D ? D : (uint32_t)q;
                    kk = (uint32_t)ktab.at(w, (size_t)l * K + j);
                }
                s_units[i] = u;
                s_kk[i] = kk;
            }
            for (uint32_t i = threadIdx.x; i < 2 * rowp; i += blockDim.x) prow[i] = kNone;
            __syncthreads();
            if (threadIdx.x == 0) pv[0] = 0;
            for (uint32_t l = 0; l < L; ++l) {
                __syncthreads();
                const uint32_t* un = s_units + l * Kp;
                const uint32_t* kk = s_kk + l * Kp;
                uint8_t* pdl = pd + (size_t)l * plan.pd_row_bytes;
                for (uint32_t bb = 0; bb < row; bb += kDpCells * blockDim.x) {
#pragma unroll
                    for (int q = 0; q < kDpCells; ++q) {
                        const uint32_t b = bb + threadIdx.x + q * blockDim.x;
                        const uint32_t bc = min(b, row - 1);
                        uint32_t best = kNone, bj = 0;
                        for (uint32_t j = 0; j < K; ++j) {
                            const uint32_t p = pv[(int)bc - (int)un[j]];
                            const uint32_t t = p > kNone - kk[j] ? kNone : p + kk[j];
                            if (t < best) { best = t; bj = j; }
                        }
                        if (b < row) cu[b] = best;
                        if (plan.pd_nibble) {
                            const uint32_t nb = __shfl_down_sync(0xffffffffu, bj, 1);
                            if (!(threadIdx.x & 1) && b < row) pdl[b >> 1] = (uint8_t)(bj | (nb << 4));
                        } else if (b < row) {
                            pdl[b] = (uint8_t)bj;
                        }
                    }
                }
                uint32_t* sw = pv; pv = cu; cu = sw;
            }
            __syncthreads();
            const uint64_t cap_k = c / bpe;
            for (uint32_t b = threadIdx.x; b < row; b += blockDim.x)
                if (pv[b] != kNone && (uint64_t)pv[b] <= cap_k) atomicMin(&s_best, b);
            __syncthreads();
            if (threadIdx.x == 0) {
                if (s_best == kNone) {
                    s_status = KIMAD_STATUS_INFEASIBLE;
                } else {
                    s_status = KIMAD_OK;
                    uint32_t b = s_best;
                    for (uint32_t l = L; l-- > 0;) {
                        const uint8_t* pdl = pd + (size_t)l * plan.pd_row_bytes;
                        const uint32_t j = plan.pd_nibble ? ((pdl[b >> 1] >> (4 * (b & 1))) & 15u) : pdl[b];
                        s_j[l] = j;
                        b -= s_units[l * Kp + j];
                    }
                }
            }
            __syncthreads();
            status = s_status;
            if (status == KIMAD_STATUS_INFEASIBLE)
                for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = 0;
        } else {
            // candidate (l, j) -> smem slot; units above D become D+1 (reads the +inf margin), padding likewise
            auto load_tab = [&](uint32_t l, uint32_t j, uint32_t slot_l) {
                uint32_t u = D + 1;
                float e = 0.f;
                if (j < K) {
                    bool dense;
                    const uint64_t uu = budget_cells(candidate_bytes(layers[l].n, ktab.at(w, (size_t)l * K + j), bpe, cost_model, &dense), D, c);
                    u = uu > D ? D + 1 : (uint32_t)uu;
                    e = dense ? 0.f : e_w[(size_t)l * K + j]; // a layer sent densely loses nothing
                }
                s_units[slot_l * Kp + j] = u;
                s_err[slot_l * Kp + j] = e;
            };
            auto count_usable = [&](uint32_t slot_l) { // sizes ascend with j, so the usable candidates come first
                uint32_t nu = 0;
                bool same = true; // all usable candidates take the same number of cells (small layers under a coarse cell)
                bool mono = true; // ... and their errors are finite and do not increase with j
                while (nu < K && s_units[slot_l * Kp + nu] <= D) {
                    same &= s_units[slot_l * Kp + nu] == s_units[slot_l * Kp];
                    const float e = s_err[slot_l * Kp + nu];
                    mono &= e < kInf && e >= 0.f && (nu == 0 || e <= s_err[slot_l * Kp + nu - 1]);
                    ++nu;
                }
                s_usable[slot_l] = nu | (same && nu > 1 ? kDpSameCells : 0u) | (same && nu >= 1 && mono ? kDpChain : 0u);
            };
            if (plan.tab_in_smem) {
                for (uint32_t i = threadIdx.x; i < L * Kp; i += blockDim.x) load_tab(i / Kp, i % Kp, i / Kp);
                __syncthreads();
                for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) count_usable(l);
            }
            for (uint32_t i = threadIdx.x; i < 2 * rowp; i += blockDim.x) rows[i] = kInf;
            __syncthreads();
            if (threadIdx.x == 0) prev[0] = 0.f;
            for (uint32_t l = 0; l < L; ++l) {
                __syncthreads();
                if (!plan.tab_in_smem) {
                    if (threadIdx.x < Kp) load_tab(l, threadIdx.x, 0);
                    __syncthreads();
                    if (threadIdx.x == 0) count_usable(0);
                    __syncthreads();
                }
                if (plan.tab_in_smem && (s_usable[l] & kDpChain)) {
                    // A run of consecutive layers whose usable candidates all take the same number of cells (small
                    // layers under a coarse cell).  Such a layer shifts the row by its cells and adds, per cell, the
                    // smallest fl(p + e_j); with e non-increasing in j the candidates attaining it are the last ones,
                    // and the first of them (the one a strict `<` over ascending j keeps) is found by bisection (when
                    // the running sum dwarfs the layer's errors they all tie and candidate 0 is kept).  The shifts of
                    // a run add up, so a thread carries its cells through the whole run by itself: one barrier per
                    // run, and the back-pointers of the run's layers are stored at the cell the run ENDS in (the
                    // backtracking below reads them there).
                    uint32_t m = 1, U = s_units[l * Kp];
                    while (l + m < L && m < (uint32_t)kDpMaxChain && (s_usable[l + m] & kDpChain)) { U += s_units[(l + m) * Kp]; ++m; }
                    float v[kDpCells];
                    for (uint32_t bb = 0; bb < row; bb += kDpCells * blockDim.x) {
                        const uint32_t b0 = bb + threadIdx.x;
#pragma unroll
                        for (int q = 0; q < kDpCells; ++q) {
                            const uint32_t b = b0 + q * blockDim.x;
                            v[q] = (b < row && b >= U) ? prev[b - U] : kInf;
                        }
                        for (uint32_t i = 0; i < m; ++i) {
                            const float* er = s_err + (l + i) * Kp;
                            const uint32_t nu = s_usable[l + i] & 0xffffu;
                            const float emin = er[nu - 1];
                            uint8_t* pdl = pd + (size_t)(l + i) * plan.pd_row_bytes;
                            // first j with fl(p + e_j) == fl(p + e_min): bisection in a fixed number of steps, the
                            // thread's cells side by side (p = +inf compares equal everywhere and ends at j = 0, the
                            // value an untouched cell holds)
                            const int steps = nu > 1 ? 32 - __clz(nu - 1) : 0;
                            float t[kDpCells];
                            uint32_t lo[kDpCells], hi[kDpCells];
#pragma unroll
                            for (int q = 0; q < kDpCells; ++q) { t[q] = __fadd_rn(v[q], emin); lo[q] = 0; hi[q] = nu - 1; }
                            for (int s = 0; s < steps; ++s) {
#pragma unroll
                                for (int q = 0; q < kDpCells; ++q) {
                                    const uint32_t mid = (lo[q] + hi[q]) >> 1;
                                    const bool eq = __fadd_rn(v[q], er[mid]) == t[q];
                                    hi[q] = eq ? mid : hi[q];
                                    lo[q] = eq ? lo[q] : min(mid + 1, hi[q]);
                                }
                            }
#pragma unroll
                            for (int q = 0; q < kDpCells; ++q) {
                                const uint32_t b = b0 + q * blockDim.x;
                                const uint32_t bj = lo[q];
                                v[q] = t[q];
                                if (plan.pd_nibble) {
                                    const uint32_t nb = __shfl_down_sync(0xffffffffu, bj, 1);
                                    if (!(threadIdx.x & 1) && b < row) pdl[b >> 1] = (uint8_t)(bj | (nb << 4));
                                } else if (b < row) {
                                    pdl[b] = (uint8_t)bj;
                                }
                            }
                        }
#pragma unroll
                        for (int q = 0; q < kDpCells; ++q) {
                            const uint32_t b = b0 + q * blockDim.x;
                            if (b < row) cur[b] = v[q];
                        }
                    }
                    if (threadIdx.x == 0)
                        for (uint32_t i = 0; i + 1 < m; ++i) s_usable[l + i] |= kDpInner; // not the run's last layer
                    float* sw = prev; prev = cur; cur = sw;
                    l += m - 1;
                    continue;
                }
                const uint32_t sl = plan.tab_in_smem ? l : 0;
                const uint32_t* un = s_units + sl * Kp;
                const float* er = s_err + sl * Kp;
                const uint32_t nu = s_usable[sl] & 0xffffu;
                const bool same_cells = (s_usable[sl] & kDpSameCells) != 0;
                uint8_t* pdl = pd + (size_t)l * plan.pd_row_bytes;
                // each thread owns the cells t, t + T, ... (consecutive threads read consecutive words of
                // prev[]: no bank conflicts); candidates four at a time so that the prev[] reads of a batch are
                // independent loads and a candidate's (cells, error) pair is fetched once for all cells of the thread
                for (uint32_t bb = 0; bb < row; bb += kDpCells * blockDim.x) {
                    const uint32_t b0 = bb + threadIdx.x;
                    float best[kDpCells];
                    uint32_t bj[kDpCells];
#pragma unroll
                    for (int q = 0; q < kDpCells; ++q) { best[q] = kInf; bj[q] = 0; }
                    if (same_cells) { // one read of prev[] serves all candidates; same adds, same order, same ties
                        const int u0 = (int)un[0];
                        float p0[kDpCells];
#pragma unroll
                        for (int q = 0; q < kDpCells; ++q) p0[q] = prev[(int)min(b0 + q * blockDim.x, row - 1) - u0];
                        for (uint32_t j = 0; j < nu; ++j) {
                            const float ej = er[j];
#pragma unroll
                            for (int q = 0; q < kDpCells; ++q) {
                                const float t = __fadd_rn(p0[q], ej);
                                if (t < best[q]) { best[q] = t; bj[q] = j; }
                            }
                        }
                    } else
                    for (uint32_t j0 = 0; j0 < nu; j0 += 4) {
                        float p[4][kDpCells];
                        const uint4 u4 = *reinterpret_cast<const uint4*>(un + j0);
                        const float4 e4 = *reinterpret_cast<const float4*>(er + j0);
                        const uint32_t u[4] = {u4.x, u4.y, u4.z, u4.w};
                        const float e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int q = 0; q < kDpCells; ++q) {
                                // cells beyond the row (last pass only) read the row itself: harmless, never stored
                                const uint32_t b = min(b0 + q * blockDim.x, row - 1);
                                p[i][q] = KIMAD_CHECK((int)b - (int)u[i] >= -(int)pad, 5) ? prev[(int)b - (int)u[i]] : kInf;
                            }
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int q = 0; q < kDpCells; ++q) {
                                const float t = __fadd_rn(p[i][q], e[i]); // +inf when the candidate does not fit
                                if (t < best[q]) { best[q] = t; bj[q] = j0 + i; }
                            }
                    }
#pragma unroll
                    for (int q = 0; q < kDpCells; ++q) {
                        const uint32_t b = b0 + q * blockDim.x;
                        if (b < row) cur[b] = best[q];
                        if (plan.pd_nibble) { // even threads store their own nibble and their right neighbour's
                            const uint32_t nb = __shfl_down_sync(0xffffffffu, bj[q], 1);
                            if (!(threadIdx.x & 1) && b < row) pdl[b >> 1] = (uint8_t)(bj[q] | (nb << 4));
                        } else if (b < row) {
                            pdl[b] = (uint8_t)bj[q];
                        }
                    }
                }
                float* sw = prev; prev = cur; cur = sw;
            }
            __syncthreads();
            // lowest cell attaining the minimum: lexicographic (value, cell) min-reduction
            float bv = kInf;
            uint32_t bb = 0xffffffffu;
            for (uint32_t b = threadIdx.x; b < row; b += blockDim.x) {
                const float v = prev[b];
                if (v < bv || (v == bv && b < bb)) { bv = v; bb = b; }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const uint32_t ob = __shfl_xor_sync(0xffffffffu, bb, o);
                if (ov < bv || (ov == bv && ob < bb)) { bv = ov; bb = ob; }
            }
            if ((threadIdx.x & 31) == 0) { s_redv[threadIdx.x >> 5] = bv; s_redb[threadIdx.x >> 5] = bb; }
            __syncthreads();
            if (threadIdx.x == 0) {
                for (uint32_t i = 1; i < blockDim.x / 32; ++i) {
                    const float ov = s_redv[i];
                    const uint32_t ob = s_redb[i];
                    if (ov < bv || (ov == bv && ob < bb)) { bv = ov; bb = ob; }
                }
                if (!(bv < kInf)) {
                    s_status = KIMAD_STATUS_INFEASIBLE;
                } else {
                    s_status = KIMAD_OK;
                    uint32_t b = bb, b_at = bb;
                    for (uint32_t l = L; l-- > 0;) { // walk the back-pointers
                        const uint8_t* pdl = pd + (size_t)l * plan.pd_row_bytes;
                        if (!plan.tab_in_smem || !(s_usable[l] & kDpInner)) b_at = b; // inner layers of a run: the run's end cell
                        const uint32_t j = plan.pd_nibble ? ((pdl[b_at >> 1] >> (4 * (b_at & 1))) & 15u) : pdl[b_at];
                        s_j[l] = j;
                        b -= plan.tab_in_smem ? s_units[l * Kp + j]
                                              : (uint32_t)budget_cells(candidate_bytes(layers[l].n, ktab.at(w, (size_t)l * K + j), bpe, cost_model, nullptr), D, c);
                    }
                }
            }
            __syncthreads();
            status = s_status;
            if (status == KIMAD_STATUS_INFEASIBLE)
                for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) s_j[l] = 0;
        }
    }
    __syncthreads();

    // totals, capacity check and outputs (prev/cur are free now: k_l and err_l of the chosen candidates are staged
    // there; L <= D < the rows' size).  Entries kept and bytes are order-free integer sums; the error is added left
    // to right in binary32.
    uint32_t* s_k = reinterpret_cast<uint32_t*>(smem_raw);
    float* s_e = reinterpret_cast<float*>(smem_raw) + rowp;
    __shared__ unsigned long long s_nsel, s_used;
    if (threadIdx.x == 0) { s_nsel = 0; s_used = 0; }
    __syncthreads();
    if (status >= 0) {
        unsigned long long my_n = 0, my_b = 0;
        for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) {
            const uint64_t n = layers[l].n, k = ktab.at(w, (size_t)l * K + s_j[l]);
            bool dense;
            my_b += candidate_bytes(n, k, bpe, cost_model, &dense);
            const uint32_t k_eff = (uint32_t)(dense ? n : k);
            my_n += k_eff;
            s_k[l] = k_eff;
            s_e[l] = dense ? 0.f : e_w[(size_t)l * K + s_j[l]];
            if (out_dense) out_dense[(size_t)w * L + l] = dense ? 1u : 0u;
        }
        atomicAdd(&s_nsel, my_n);
        atomicAdd(&s_used, my_b);
    } else if (out_dense) {
        for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) out_dense[(size_t)w * L + l] = 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint64_t nsel = s_nsel;
        float tot = 0.f;
        if (status >= 0)
            for (uint32_t l = 0; l < L; ++l) tot = __fadd_rn(tot, s_e[l]);
        if (status == KIMAD_OK && mode == 4 && s_used > c) status = KIMAD_STATUS_INFEASIBLE; // not even one entry per layer fits
        if (status >= 0 && nsel > cap) status = KIMAD_ERR_CAPACITY;
        kimad_stats s;
        s.budget_bytes = c;
        s.n_selected = status >= 0 ? nsel : 0;
        s.used_bytes = status >= 0 ? s_used : 0;
        s.total_err = status >= 0 ? tot : 0.f;
        s.status = status;
        out_stats[w] = s;
        uint64_t run = 0;
        for (uint32_t l = 0; l < L; ++l) {
            out_offs[(size_t)w * (L + 1) + l] = run;
            if (status >= 0) run += s_k[l];
        }
        out_offs[(size_t)w * (L + 1) + L] = run;
        s_status = status;
        flags[w] = 0; // consumed
    }
    __syncthreads();
    status = s_status;
    for (uint32_t l = threadIdx.x; l < L; l += blockDim.x) {
        const size_t wl = (size_t)w * L + l;
        Sel s;
        if (status >= 0) {
            const uint32_t j = s_j[l];
            s.tau = tau[wl * K + j];
            s.keep_eq = keep_eq[wl * K + j];
            s.k = s_k[l];
            s.shift = shift ? shift[wl * K + j] : 0u;
            s.base = out_offs[(size_t)w * (L + 1) + l];
            s.code = codes.code(w, l, s.tau); // the whole interval lies in one bin, hence has one code
            out_k[wl] = s_k[l];
            out_j[wl] = j;
        } else {
            s.tau = 0; s.keep_eq = 0; s.k = 0; s.shift = 0; s.base = 0; s.code = 0;
            out_k[wl] = 0;
            out_j[wl] = 0;
        }
        s.tau_low = 0;
        sel[wl] = s;
    }
}

// The ratio of Section 3.1 sized to the budget: r = q / 2^32 with the largest q whose entries
// sum_l min(n_l, max(1, floor(q n_l / 2^32))) fit floor(c / (4 + vb)); the worker's table row gets those k_l.
// One CTA per worker; the sum is an order-free integer reduction, q is found by bisection (33 steps).
__global__ void __launch_bounds__(kThreads)
k_fit_ratio(DpBudgets budgets, uint32_t w_base, uint32_t W, uint32_t L, uint32_t bpe, uint64_t N,
            const LayerDesc* __restrict__ layers, uint64_t* __restrict__ ktab_w /* [W][L] */) {
    pdl_wait();
    const uint32_t w = w_base + blockIdx.x;
    if (w >= W) return;
    __shared__ unsigned long long s_sum;
    const uint64_t entries = budgets.c[blockIdx.x] / bpe;
    auto k_of = [&](uint64_t q, uint64_t n) {
        uint64_t k = q >= 4294967296ull ? n : (q * n) >> 32;
        k = k < 1 ? 1 : k;
        return k > n ? n : k;
    };
    uint64_t q;
    if (entries < (uint64_t)L) q = 0;
    else if (entries >= N) q = 4294967296ull;
    else {
        uint64_t lo = 0, hi = 4294967296ull; // sum(lo) <= entries < sum(hi)
        while (hi - lo > 1) {
            const uint64_t mid = lo + (hi - lo) / 2;
            if (threadIdx.x == 0) s_sum = 0;
            __syncthreads();
            unsigned long long mine = 0;
            for (uint32_t l = threadIdx.x; l < L; l += kThreads) mine += k_of(mid, layers[l].n);
#pragma unroll
            for (int o = 16; o; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
            if ((threadIdx.x & 31) == 0) atomicAdd(&s_sum, mine);
            __syncthreads();
            if (s_sum <= entries) lo = mid; else hi = mid;
            __syncthreads();
        }
        q = lo;
    }
    for (uint32_t l = threadIdx.x; l < L; l += kThreads) ktab_w[(size_t)w * L + l] = k_of(q, layers[l].n);
}

} // namespace kimad
