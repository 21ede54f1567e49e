// Stage (a)+(b), fast path: EF21 difference fused with a banded histogram that yields the error curve of
// every candidate in ONE sweep over the gradients.
//
//   k_sample     per (worker, layer): histogram of a stratified sample of |d| over 16-bit key prefixes
//                ("cells"); for every candidate k_j the cells that can contain the k_j-th largest key
//                (sample rank +- 6 sigma) form a band.  Band cells are cut into fine bins of 2^shift
//                keys, everything else into coarse "gap" bins.  Every region (a gap, or a group of bands with
//                one bin width) maps a key to its bin as base + (key >> shift); which region a key lies in is
//                read from a table over the window of cells between the lowest and the highest band.
//                A mass of exact zeros in the sample (a sparse gradient) is counted apart: such a layer's zeros
//                stay out of the sweep's histogram, candidates whose rank lies among them need no band, and
//                sigma grows by what the spread of the zeros over the sampled units says about their clustering.
//   k_pass_a     the sweep: d = grad - g (one code byte per element goes to scratch), bin = base + (key >> shift)
//                with (base, shift) = table(cell(key)), two u32 shared-memory atomics per element: the count, and
//                the exact integer sum of squares in a u32 word whose (rare) carries go straight to the 64-bit sum
//                in global memory.  CTAs own static runs of chunks balanced by elements.
//   k_resolve_a  per (worker, layer): totals of every group of 32 bins, a scan over the groups, then a warp per
//                candidate finds the group and the bin that hold its threshold (zeros left out by the sweep = the
//                layer's size minus the counted entries) and the squares below it.  The candidate's error is certified to 5e-6 relative from the bin's width.  A
//                threshold in a gap bin (the sample mispredicted) sends the layer to the exact radix path; a bound
//                that is too loose sends the candidate to the refinement.
//   k_refine_hist, k_refine_resolve
//                loose candidates: the entries of the threshold's bin, found by their code byte, are counted in
//                1024 pieces of the bin; error and interval from the pieces (still loose: exact path).
//   k_tiny_exact layers of at most kTinyMax elements are sorted in shared memory instead.
//   k_fb_*       exact three-digit radix select over the chunks of the layers handed over (rare).
#pragma once
#include "kimad_kernels.cuh"
#include <type_traits>

namespace kimad {

constexpr int kTinyMax = 4096;
#ifndef KIMAD_FINE_BINS
#define KIMAD_FINE_BINS 12288
#endif
constexpr int kFineBins = KIMAD_FINE_BINS;          // fine bins per (worker, layer)
constexpr int kMaxGaps = KIMAD_MAX_RATIOS + 2;      // gap regions: below / between / above the band groups, + non-finite keys
constexpr int kMaxBins = kFineBins + kL1Bins + 2 * kMaxGaps; // fine bins + gap regions cut at every 11-bit prefix
constexpr int kMaxShift = 15;                       // a fine bin is 2^shift keys wide, at most a whole cell
constexpr int kSampleUnit = 32;                     // consecutive elements read together (128 bytes, one warp)
constexpr int kSampleUnits = 2047;                  // units of a sample (<= 65504 elements: the u16 cell counters cannot overflow)
constexpr int kBigThreads = 1024;
constexpr uint32_t kGapBit = 1u;                    // bin_lo entries carry this bit when the bin is a gap bin


__device__ __forceinline__ uint32_t hash_u32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

// ------------------------------------------------------------------------------------------------
// k_sample: one CTA per (regular layer, worker)
// ------------------------------------------------------------------------------------------------
// (48 registers: a CTA of the tiny layers' kernel, which runs beside this one, then fits on the same SM)
__global__ void __maxnreg__(48)
k_sample(const float* __restrict__ grads, const float* __restrict__ state, uint64_t stride,
         const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ reg_layers, uint32_t R,
         const KTab ktab, uint32_t K, uint32_t force_exact, uint32_t* __restrict__ cell_tab,
         int4* __restrict__ cell_win, uint32_t* __restrict__ bin_lo, BandMeta* __restrict__ meta) {
    pdl_wait();
    extern __shared__ __align__(16) uint32_t sh[];
    double* s_sq = reinterpret_cast<double*>(sh); // [1024] squares (cell midpoints) below each thread segment
    double* s_wd = s_sq + 1024;                   // [32]
    uint32_t* h32 = sh + 2 * (1024 + 32);         // [32768] two u16 cell counters per word
    uint32_t* s_pre = h32 + 32768;                // [1024] inclusive sample count of the thread segments, from the top
    uint32_t* s_base = s_pre + 1024;              // [2 kMaxGaps] first bin id of every gap region, of every group
    uint32_t* s_w = s_base + 2 * kMaxGaps;        // [32]
    uint32_t* s_cb = s_w + 32;                    // [128] per candidate, then per merged group: lowest cell,
    uint32_t* s_ct = s_cb + 128;                  // [128] highest cell,
    uint32_t* s_cs = s_ct + 128;                  // [128] shift
    __shared__ uint32_t s_m, s_flag, s_ng, s_cg, s_z;
    __shared__ unsigned long long s_zz;
    const uint32_t r = blockIdx.x, w = blockIdx.y;
    const uint32_t l = reg_layers[r];
    const size_t wr = (size_t)w * R + r;
    BandMeta* mt = meta + wr;
    if (force_exact) {
        if (threadIdx.x == 0) *mt = BandMeta{0, 0, 1, 0};
        return;
    }
    const LayerDesc ld = layers[l];
    const uint32_t n = (uint32_t)ld.n;
    for (int i = threadIdx.x; i < 32768 / 4; i += kBigThreads) reinterpret_cast<uint4*>(h32)[i] = make_uint4(0u, 0u, 0u, 0u);
    if (threadIdx.x == 0) { s_m = 0; s_flag = 0; s_ng = 0; s_cg = 0; s_z = 0; s_zz = 0ull; }
    __syncthreads();

    // ---- stratified sample of |grad - g|.  Exact zeros (the untouched rows of a sparse gradient) are counted apart:
    // they sit below every other key, add nothing to any error, and the sweep leaves them out of its histogram.
    const float* gr = grads + (size_t)w * stride + ld.begin;
    const float* st = state + (size_t)w * stride + ld.begin;
    const uint32_t n_units = n / kSampleUnit + ((n % kSampleUnit) != 0); // n may be as large as 2^32 - 1
    const uint32_t m_units = min(n_units, (uint32_t)kSampleUnits);
    const bool whole = m_units == n_units;
    const uint32_t sq_ = n / (uint32_t)kSampleUnits, sr_ = n % (uint32_t)kSampleUnits; // used when sampled: m_units = kSampleUnits
    uint32_t mine = 0;
    // a warp reads one unit (128 bytes); eight units per thread are in flight before their keys are counted
    for (uint32_t ib = threadIdx.x / kSampleUnit; ib < m_units; ib += 8 * (kBigThreads / kSampleUnit)) {
        float a[8], b[8];
        bool ok[8];
        // where the round's eight units start is the same for all lanes: lane u (mod 8) works out unit u's start
        // and the others fetch it with a shuffle
        uint32_t my_start;
        {
            const uint32_t i = ib + (threadIdx.x & 7u) * (kBigThreads / kSampleUnit);
            my_start = kSampleUnit * i;
            if (!whole && i < m_units) { // unit i somewhere inside stratum i = [i q + i r / m, (i+1) q + (i+1) r / m)
                const uint32_t s0 = i * sq_ + (i * sr_) / (uint32_t)kSampleUnits;
                const uint32_t s1 = (i + 1) * sq_ + ((i + 1) * sr_) / (uint32_t)kSampleUnits;
                const uint32_t room = s1 > s0 + kSampleUnit ? s1 - s0 - kSampleUnit : 0;
                my_start = s0 + __umulhi(hash_u32(i * 0x9e3779b9u + l * 0x85ebca6bu + 1u), room + 1);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t i = ib + u * (kBigThreads / kSampleUnit);
            const uint32_t p = __shfl_sync(0xffffffffu, my_start, u) + (threadIdx.x % kSampleUnit);
            ok[u] = i < m_units && p < n;
            a[u] = ok[u] ? gr[p] : 0.f;
            b[u] = ok[u] ? st[p] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t key = ok[u] ? key_of(__fsub_rn(a[u], b[u])) : 1u;
            if ((u & 3) == 0) { // every fourth unit: its exact zeros, for the spread of the zeros over the units
                const uint32_t zu = __popc(__ballot_sync(0xffffffffu, key == 0u));
                if (zu && (threadIdx.x & 31) == 0) { atomicAdd(&s_z, zu); atomicAdd(&s_zz, (unsigned long long)(zu * zu)); }
            }
            if (ok[u]) {
                if (key) atomicAdd(&h32[key >> 16], 1u << (16 * ((key >> 15) & 1)));
                ++mine;
            }
        }
    }
    atomicAdd(&s_m, mine);
    __syncthreads();
    const uint32_t m = s_m; // sample size, exact zeros included
    auto cell_count = [&](uint32_t cell) { return (h32[cell >> 1] >> (16 * (cell & 1))) & 0xffffu; };
    auto cell_sq = [&](uint32_t cell) { // square of the cell's middle value (planning only: float range is enough)
        const float v = __uint_as_float((cell << 15) | 0x4000u);
        return (double)(v * v);
    };

    // ---- per thread segment (cells 65535 - 64 t - (0..63)): sample count and squares; the reads of a warp are
    // rotated so that the lanes of a quarter warp hit different banks
    uint32_t mz; // sample entries in the histogram: all but the exact zeros
    {
        uint32_t sum = 0;
        double sq = 0.0;
        // the segment is 32 words (two cells each), read four at a time; most words are empty
        const uint32_t w0 = 32736u - 32u * threadIdx.x; // first word of the segment: cells 2 w0 .. 2 w0 + 63
        for (uint32_t q0 = 0; q0 < 8; ++q0) {
            const uint32_t q = (q0 + threadIdx.x) & 7u;
            const uint4 x4 = reinterpret_cast<const uint4*>(h32)[(w0 >> 2) + q];
            const uint32_t x[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (x[i]) {
                    const uint32_t cell = 2u * (w0 + 4u * q + (uint32_t)i), c0 = x[i] & 0xffffu, c1 = x[i] >> 16;
                    sum += c0 + c1;
                    if (c0) sq += (double)c0 * cell_sq(cell);
                    if (c1) sq += (double)c1 * cell_sq(cell + 1u);
                }
        }
        double totd;
        const uint32_t ex = block_excl_scan<uint32_t, kBigThreads>(sum, s_w, &mz);
        const double exd = block_excl_scan<double, kBigThreads>(sq, s_wd, &totd);
        s_pre[threadIdx.x] = ex + sum;
        s_sq[threadIdx.x] = totd - exd - sq; // squares in the segments below this one (higher thread index)
    }
    __syncthreads();
    const uint32_t z = m - mz; // the sample's exact zeros
    // Variance of the sample's zero count, from the spread of the zero counts of the units looked at (the units i with
    // i mod 128 < 32): zeros that come in runs (whole rows) make the sample's share of zeros, and with it the sample
    // rank of every threshold among the other keys, far less certain than independent draws would.
    double var_z = 0.0;
    if (z && !whole) {
        const double ns = (double)((m_units / 128u) * 32u + min(m_units % 128u, 32u)), zs = (double)s_z;
        var_z = fmax(0.0, ((double)s_zz - zs * zs / ns) / ns) * (double)m_units;
    }
    // cell holding sample rank rk (1-based, from the top); the whole warp takes part
    const uint32_t lane = threadIdx.x & 31;
    auto cell_of_rank = [&](uint32_t rk) {
        int lo = 0, hi = kBigThreads - 1;
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_pre[mid] >= rk) hi = mid; else lo = mid + 1; }
        const uint32_t before = lo ? s_pre[lo - 1] : 0u;
        const uint32_t top = 65535u - 64u * lo;
        // lanes take cells top - 2 lane and top - 2 lane - 1; inclusive counts along the lanes
        const uint32_t c0 = cell_count(top - 2 * lane), c1 = cell_count(top - 2 * lane - 1);
        uint32_t incl = c0 + c1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= (uint32_t)o) incl += y;
        }
        const uint32_t upto0 = before + incl - c1; // entries in the cells top .. top - 2 lane
        const uint32_t hit0 = __ballot_sync(0xffffffffu, upto0 >= rk);
        const uint32_t hit1 = __ballot_sync(0xffffffffu, before + incl >= rk);
        if (!hit1) return top - 63u;
        const uint32_t l1 = __ffs(hit1) - 1;
        return (hit0 >> l1) & 1u ? top - 2 * l1 : top - 2 * l1 - 1;
    };

    // ---- bands: the cells that can hold the k_j-th largest key, and how finely to cut them (one warp per candidate)
    for (uint32_t j = threadIdx.x >> 5; j < K; j += kBigThreads / 32) {
        const uint64_t k = ktab.at(w, (size_t)l * K + j);
        uint32_t o_cb = 1, o_ct = 0, o_cs = 15; // k == n keeps everything: no threshold, no band
        if (k < n) {
            uint32_t r_lo, r_hi;
            if (whole) {
                r_lo = r_hi = (uint32_t)k;
            } else {
                const double p = (double)k / (double)n;
                const double rho = p * (double)m, rel = mz ? rho / (double)mz : 0.0;
                const double sg = sqrt((double)m * p * (1.0 - p) + rel * rel * var_z);
                const double a = floor(rho - 6.0 * sg - 2.0), b = ceil(rho + 6.0 * sg + 2.0);
                r_lo = a < 1.0 ? 0u : (uint32_t)a;
                r_hi = b > (double)m ? 0u : (uint32_t)b;
            }
            // a rank window wholly among the zeros: the threshold is 0 unless the sample misleads, no band (the curve
            // stage knows the exact number of zeros); a window that reaches into the zeros ends at the lowest cell
            // the sample saw, a quarter octave further down
            const bool zero_cand = z && (mz == 0 || r_lo > mz);
            const bool clip_bot = z && !zero_cand && (r_hi == 0 || r_hi > mz);
            if (zero_cand) {
                if (lane == 0) { s_cb[j] = o_cb; s_ct[j] = o_ct; s_cs[j] = o_cs; }
                continue;
            }
            // rank window clipped at the top: the threshold may lie above the largest sample, so the band goes a
            // quarter octave further up; clipped at the bottom: no bound from the sample, exact path
            // bands stay among the finite keys (a sample with non-finite values is reported by the curve stage)
            uint32_t c_top = min(cell_of_rank(max(r_lo, 1u)), 65279u);
            if (r_lo == 0) c_top = min(c_top + 64u, 65279u);
            if (r_hi == 0 && !z && lane == 0) s_flag = 1;
            uint32_t c_bot = cell_of_rank(clip_bot ? mz : max(r_hi, 1u));
            if (clip_bot) c_bot = c_bot > 64u ? c_bot - 64u : 0u;
            c_bot = min(c_bot, c_top);
            const uint32_t ncell = c_top - c_bot + 1;
            if (ncell > (uint32_t)kFineBins) {
                if (lane == 0) s_flag = 2;
            } else {
                // sample entries in each quarter of the band (a tail band is much denser at its bottom)
                const uint32_t nq = (ncell + 3) / 4;
                uint32_t inq[4] = {0, 0, 0, 0};
                for (uint32_t c = c_bot + lane; c <= c_top; c += 32) {
                    const uint32_t cc = cell_count(c), qi = (c - c_bot) / nq;
#pragma unroll
                    for (int i = 0; i < 4; ++i) inq[i] += qi == (uint32_t)i ? cc : 0u;
                }
                // estimate of this candidate's error: squares of everything below the band
                const uint32_t seg = (65535u - c_bot) >> 6;
                double below = 0.0;
                for (uint32_t c = 65535u - 64u * seg - 63u + lane; c < c_bot; c += 32) {
                    const uint32_t cc = cell_count(c);
                    if (cc) below += (double)cc * cell_sq(c);
                }
#pragma unroll
                for (int o = 16; o; o >>= 1) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) inq[i] += __shfl_xor_sync(0xffffffffu, inq[i], o);
                    below += __shfl_xor_sync(0xffffffffu, below, o);
                }
                below += s_sq[seg];
                const double scale = (double)n / (double)m;
                // bins per cell: at most ~2048 entries per bin (what the select stage collects and sorts), and
                // narrow enough that the uncertainty of the bin holding the threshold (its entries times its
                // spread of squares, 2^-7 of v^2 for a whole cell) stays below ~3e-6 of the error; entries per
                // cell and v^2 are taken quarter by quarter
                double dens = 0.0, load = 0.0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t qtop = min(c_top, c_bot + (uint32_t)(i + 1) * nq - 1);
                    const double per_cell = (double)(inq[i] + 1) / (double)nq * scale; // + 1: never plan on an empty sample
                    dens = per_cell > dens ? per_cell : dens;
                    const double ld = per_cell * cell_sq(qtop);
                    load = ld > load ? ld : load;
                }
                double bins = dens / 2048.0;
                const double e_est = below * scale;
                const double cert = e_est > 0.0 ? sqrt(load * 0.0078125 / (3e-6 * e_est)) : 1024.0;
                if (cert > bins) bins = cert;
                uint32_t sh_j = 15;
                while (sh_j > 5 && (double)(1u << (15 - sh_j)) < bins) --sh_j;
                o_cb = c_bot; o_ct = c_top; o_cs = sh_j;
            }
        }
        if (lane == 0) { s_cb[j] = o_cb; s_ct[j] = o_ct; s_cs[j] = o_cs; }
    }
    __syncthreads();
    // merge overlapping / adjacent bands (they descend in key with j) into groups; groups end up in s_c*[0..ng)
    if (threadIdx.x == 0 && !s_flag) {
        // The sweep reads a key's region from a table over the cells between the lowest and the highest band.  If
        // that window has more cells than the table has entries, an entry stands for 2^cg cells and the bands
        // are widened to whole entries (more fine bins; the common case is cg = 0).
        uint32_t lo_all = 0xffffffffu, hi_all = 0, cg = 0;
        for (uint32_t j = 0; j < K; ++j)
            if (s_cb[j] <= s_ct[j]) { lo_all = min(lo_all, s_cb[j]); hi_all = max(hi_all, s_ct[j]); }
        if (lo_all <= hi_all)
            while ((hi_all >> cg) - (lo_all >> cg) + 3 > (uint32_t)kCellTab) ++cg;
        s_cg = cg;
        const uint32_t cmask = (1u << cg) - 1u;
        uint32_t ng = 0;
        uint32_t gb = 1, gt = 0, gs = 15;
        bool open = false;
        for (uint32_t j = 0; j < K; ++j) {
            uint32_t cb = s_cb[j], ct = s_ct[j];
            const uint32_t cs = s_cs[j];
            if (cb > ct) continue;
            cb &= ~cmask; ct |= cmask; // stays below the non-finite cells: 65279 ends a block of 32
            if (open && ct + 1 >= gb) {
                gb = min(gb, cb); gt = max(gt, ct); gs = min(gs, cs);
            } else {
                if (open) { s_cb[ng] = gb; s_ct[ng] = gt; s_cs[ng] = gs; ++ng; } // ng <= j: slots already consumed
                gb = cb; gt = ct; gs = cs; open = true;
            }
        }
        if (open) { s_cb[ng] = gb; s_ct[ng] = gt; s_cs[ng] = gs; ++ng; }
        // if the fine bins do not fit, scale every group's bins per cell down by the same factor (rounded
        // down to a power of two, at least one bin per cell)
        uint64_t fine = 0, cells = 0;
        for (uint32_t g = 0; g < ng; ++g) {
            fine += (uint64_t)(s_ct[g] - s_cb[g] + 1) << (15 - s_cs[g]);
            cells += s_ct[g] - s_cb[g] + 1;
        }
        if (cells > (uint64_t)kFineBins) {
            s_flag = 3;
        } else if (fine > (uint64_t)kFineBins) {
            uint32_t extra = 1;
            while ((fine >> extra) > (uint64_t)kFineBins - cells) ++extra; // groups clamped at shift 15 keep 1 bin per cell
            for (uint32_t g = 0; g < ng; ++g) s_cs[g] = min(15u, s_cs[g] + extra);
        }
        s_ng = ng;
    }
    __syncthreads();
    const uint32_t ng = s_ng, cg = s_cg;
    // ---- bin ids in ascending key order: gap_0, fine bins of the lowest group, gap_1, ..., gap_ng, non-finite keys.
    // A gap region is cut at every 11-bit prefix (one bin per piece: keeps the shared-memory atomics of the sweep
    // spread over many words); keys with exponent 255 take the eight pieces that follow gap_ng's, so that one
    // formula serves everything above the highest band.  Groups are stored with descending keys; a = ng - 1 - g
    // is the ascending index.  s_base[a] = first id of gap_a, s_glo[a] = lowest cell of gap_a.
    // Every region -- a gap or a group of fine bins -- maps a key to its bin as base + (key >> shift) with one
    // (base, shift) pair: shift 20 for the gap pieces, the group's bin width for the fine bins.
    uint32_t* s_glo = s_pre; // [kMaxGaps] reuse: the rank prefix is no longer needed
    if (threadIdx.x == 0 && !s_flag) {
        uint32_t id = 0;
        for (uint32_t a = 0; a <= ng; ++a) {
            const uint32_t lo = a == 0 ? 0u : s_ct[ng - a] + 1;              // lowest cell of the gap
            const uint32_t hi = a == ng ? 65279u : s_cb[ng - 1 - a] - 1;      // highest cell (may be lo - 1: empty)
            s_base[a] = id;
            s_glo[a] = lo;
            if (hi + 1 > lo) id += (hi >> 5) - (lo >> 5) + 1;
            if (a < ng) {
                const uint32_t g = ng - 1 - a;
                s_base[kMaxGaps + a] = id; // first fine bin of group a
                id += (s_ct[g] - s_cb[g] + 1) << (15 - s_cs[g]);
            }
        }
        s_base[ng + 1] = id;     // keys with exponent 255: the pieces 2040..2047
        s_base[ng + 2] = id + 8; // number of bins
    }
    __syncthreads();
    const uint32_t tot_bins = s_flag ? 0u : s_base[ng + 2];
    // window of the cell table: the cells from the lowest to the highest band cell and one entry on either side
    // (everything below lies in gap_0, everything above in gap_ng or among the non-finite keys)
    // (in table entries of 2^cg cells each)
    const uint32_t wlo = (ng ? s_cb[ng - 1] : 1u) >> cg, whi = (ng ? s_ct[0] : 1u) >> cg;
    const uint32_t used = whi - wlo + 3;
    const bool bad = s_flag || tot_bins > (uint32_t)kMaxBins || used > (uint32_t)kCellTab;
    if (bad) {
        if (threadIdx.x == 0) *mt = BandMeta{tot_bins, used, 2, s_flag};
        return;
    }
    // (base, shift) of the region that holds a cell, as base << 5 | shift (base may be negative)
    auto entry_of = [&](uint32_t cell) -> uint32_t {
        uint32_t a = 0;
        for (; a < ng; ++a) {
            const uint32_t g = ng - 1 - a;
            if (cell > s_ct[g]) continue;
            if (cell >= s_cb[g]) {
                const uint32_t cs = s_cs[g];
                return (uint32_t)(((int)s_base[kMaxGaps + a] - (int)(s_cb[g] << (15 - cs))) * 32) | cs;
            }
            break;
        }
        return (uint32_t)(((int)s_base[a] - (int)(s_glo[a] >> 5)) * 32) | 20u;
    };
    uint32_t* tab = cell_tab + wr * kCellTab;
    uint32_t* blo = bin_lo + wr * (kMaxBins + 1);
    // entry i serves the cells (wlo - 1 + i) << cg ...; the first one everything below the window, the last one
    // everything above it
    for (uint32_t i = threadIdx.x; i < used; i += kBigThreads) tab[i] = entry_of(i + 1 == used ? 65535u : (wlo + i - 1u) << cg);
    // lower key of every bin: the pieces of the gaps ...
    for (uint32_t b1 = threadIdx.x; b1 < (uint32_t)kL1Bins; b1 += kBigThreads) {
        const uint32_t c0 = b1 << 5, c1 = c0 + 31;
        if (b1 >= 2040u) { blo[s_base[ng + 1] + (b1 - 2040u)] = (b1 << 20) | kGapBit; continue; }
        for (uint32_t a = 0; a <= ng; ++a) {
            const uint32_t lo = s_glo[a];
            const uint32_t hi = a == ng ? 65279u : s_cb[ng - 1 - a] - 1;
            if (hi + 1 <= lo || hi < c0 || lo > c1) continue;
            blo[s_base[a] + b1 - (lo >> 5)] = (max(lo, c0) << 15) | kGapBit;
        }
    }
    // ... and the fine bins of the groups
    for (uint32_t a = 0; a < ng; ++a) {
        const uint32_t g = ng - 1 - a, cs = s_cs[g], first = s_base[kMaxGaps + a];
        const uint32_t nf = (s_ct[g] - s_cb[g] + 1) << (15 - cs);
        for (uint32_t x = threadIdx.x; x < nf; x += kBigThreads) blo[first + x] = (s_cb[g] << 15) + (x << cs);
    }
    if (threadIdx.x == 0) {
        blo[tot_bins] = 0x80000000u;
        uint32_t ls = 0; // bins per code of the byte plane: the codes stay below 128
        while (((tot_bins - 1) >> ls) > 127u) ++ls;
        cell_win[wr] = make_int4((int)wlo - 1, (int)whi + 1, (int)(15 + cg), (int)(ls | (z ? 256u : 0u))); // bit 8: zeros are left out
        *mt = BandMeta{tot_bins, used, 0, ng + 2};
    }
}

// ------------------------------------------------------------------------------------------------
// k_pass_a: every CTA owns one static run of consecutive chunks of one worker (runs balanced by elements, a few
// per SM); histogram words and the cell table of the current layer live in shared memory
// ------------------------------------------------------------------------------------------------
struct SweepRun { uint32_t w, c0, c1; }; // chunks [c0, c1) of worker w
constexpr int kRunDesc = 64;             // chunk descriptors staged in shared memory at a time

template <bool VEC>
__global__ void __launch_bounds__(kBigThreads, 1)
k_pass_a(const float* __restrict__ grads, const float* __restrict__ state, uint8_t* __restrict__ d_code,
         const Chunk* __restrict__ chunks, const SweepRun* __restrict__ runs, uint64_t stride, uint64_t dstride,
         const uint32_t* __restrict__ reg_index /* [L], 0xffffffff: tiny layer */, uint32_t R,
         const uint32_t* __restrict__ cell_tab, const int4* __restrict__ cell_win, const BandMeta* __restrict__ meta,
         uint32_t* __restrict__ bh_cnt, unsigned long long* __restrict__ bh_sum) {
    extern __shared__ __align__(16) uint32_t sh[];
    __shared__ Chunk s_desc[kRunDesc];
    uint32_t* h_cnt = sh;
    uint32_t* h_lo = sh + kMaxBins;
    uint32_t* tab = sh + 2 * kMaxBins; // [kCellTab]
    // the run, its first chunk descriptors and the clean histogram do not depend on the kernels before this one
    const SweepRun run = runs[blockIdx.x];
    for (int i = threadIdx.x; i < 2 * kMaxBins; i += kBigThreads) sh[i] = 0;
    for (uint32_t i = threadIdx.x; i < min(run.c1 - run.c0, (uint32_t)kRunDesc); i += kBigThreads) s_desc[i] = chunks[run.c0 + i];
    pdl_wait();
    __syncthreads();
    const float* gr0 = grads + (size_t)run.w * stride;
    const float* st0 = state + (size_t)run.w * stride;
    uint8_t* dc0 = d_code + (size_t)run.w * dstride;
    int cur_layer = -1;
    // slot of the current layer's histogram; 0xffffffff: none (tiny or handed-over layer); bit 30 (kSkipZeros): the
    // layer's exact zeros are left out of the histogram
    constexpr uint32_t kSkipZeros = 0x40000000u;
    uint32_t wr = 0xffffffffu;
    bool dirty = false;
    int wlo_m1 = 0, whi_p1 = 0;  // cells of the table's first and last entry, in units of 2^(cshift - 15) cells
    uint32_t cshift = 15, lshift = 0; // keys per table entry, bins per code (log2)

    auto flush = [&]() {
        __syncthreads();
        const uint32_t slot = wr & ~kSkipZeros;
        const uint32_t n_bins = meta[slot].n_bins;
        uint32_t* gc = bh_cnt + (size_t)slot * kMaxBins;
        unsigned long long* gs = bh_sum + (size_t)slot * kMaxBins;
        for (uint32_t i = threadIdx.x; i < n_bins; i += kBigThreads) {
            const uint32_t c = h_cnt[i];
            if (c) {
                atomicAdd(&gc[i], c);
                atomicAdd(&gs[i], (unsigned long long)h_lo[i]);
                h_cnt[i] = 0; h_lo[i] = 0;
            }
        }
        __syncthreads();
        dirty = false;
    };
    // (base, shift) of the region a key lies in: one table read; the clamp sends everything outside the window to
    // the table's first or last entry
    auto look = [&](uint32_t key) -> uint32_t { return tab[min(max((int)(key >> cshift), wlo_m1), whi_p1) - wlo_m1]; };
    auto bin_of = [&](uint32_t key, uint32_t e) -> uint32_t { return (uint32_t)(((int)e >> 5) + (int)(key >> (e & 31u))); };
    auto add = [&](uint32_t id, uint32_t key) {
        // 24 significant bits of the square (truncation < 2^-22 relative) summed exactly: the word wraps, the
        // returned old value tells when, and a wrap adds 2^32 to the layer's 64-bit sum in global memory
        const uint32_t sq = (uint32_t)(sq_fixed(key) >> 8);
#ifdef KIMAD_CHECKED
        if (!KIMAD_CHECK(id < meta[wr & ~kSkipZeros].n_bins, 0)) return;
#endif
        atomicAdd(&h_cnt[id], 1u);
        const uint32_t old = atomicAdd(&h_lo[id], sq);
        if (old + sq < old) atomicAdd(bh_sum + (size_t)(wr & ~kSkipZeros) * kMaxBins + id, 1ull << 32); // rare
    };
    // one element: its bin's count and sum; returns its code
    auto acc = [&](uint32_t key) -> uint32_t {
        const uint32_t id = bin_of(key, look(key));
        if (key || !(wr & kSkipZeros)) add(id, key);
        return id >> lshift;
    };
    // The four elements of a quad go through the stages together (all table reads, then the bin ids, then the
    // atomics): four independent chains of dependent shared-memory accesses instead of one after the other.
    // Returns the quad's four codes.
    // Where the sample found a mass of exact zeros (the untouched rows of a sparse gradient), zeros are left out:
    // they add nothing to any sum, they would all hit one word, and the curve stage takes their number from the
    // layer's size.
    auto acc4 = [&](const uint32_t (&k)[4], auto skip) -> uint32_t {
        uint32_t e[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = look(k[i]);
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = bin_of(k[i], e[i]);
        if (decltype(skip)::value) {
#pragma unroll
            for (int i = 0; i < 4; ++i) if (k[i]) add(e[i], k[i]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) add(e[i], k[i]);
        }
        return pack_low_bytes(e[0] >> lshift, e[1] >> lshift, e[2] >> lshift, e[3] >> lshift);
    };

    for (uint32_t c = run.c0; c < run.c1; ++c) {
        const uint32_t di = (c - run.c0) % (uint32_t)kRunDesc;
        if (di == 0 && c != run.c0) { // next window of descriptors
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < min(run.c1 - c, (uint32_t)kRunDesc); i += kBigThreads) s_desc[i] = chunks[c + i];
            __syncthreads();
        }
        Chunk ch = s_desc[di];
        // the chunks of one layer follow each other without a gap: those among the staged descriptors are swept as
        // one span, so that the load pipeline below is filled once per span and not once per chunk
        while (c + 1 < run.c1 && (c + 1 - run.c0) % (uint32_t)kRunDesc != 0) {
            const Chunk& nx = s_desc[(c + 1 - run.c0) % (uint32_t)kRunDesc];
            if (nx.layer != ch.layer || nx.begin != ch.end) break;
            ch.end = nx.end;
            ++c;
        }
        if ((int)ch.layer != cur_layer) {
            if (dirty) flush();
            cur_layer = (int)ch.layer;
            const uint32_t r = reg_index[ch.layer];
            wr = 0xffffffffu;
            __syncthreads(); // the table is no longer read
            if (r != 0xffffffffu && !meta[run.w * R + r].flagged) {
                wr = run.w * R + r;
                const int4 win = cell_win[wr];
                wlo_m1 = win.x; whi_p1 = win.y; cshift = (uint32_t)win.z; lshift = (uint32_t)win.w & 31u;
                const uint32_t* g2 = cell_tab + (size_t)wr * kCellTab;
                const uint32_t used = meta[wr].n_cells;
                for (uint32_t i = threadIdx.x; i < used; i += kBigThreads) tab[i] = g2[i];
                if ((uint32_t)win.w & 256u) wr |= kSkipZeros;
            }
            __syncthreads();
        }
        const bool active = wr != 0xffffffffu;
        const ChunkView cv(ch);
        uint8_t* dc = dc0 + cv.a0;
        {
            const uint32_t q_lo = (cv.first + 3) >> 2, q_hi = cv.len >> 2; // whole quads [q_lo, q_hi)
            // One quad per thread and round; the loads of the round three rounds ahead are issued before the current
            // round is processed (four register sets, taken in turn), so that a round's memory latency lies behind
            // the work of the rounds before it.  VEC: both inputs are 16-byte aligned at every worker's start and a
            // quad is one 128-bit load per input; otherwise four 32-bit loads, served from L1 after the first.
            const float4* gr4 = reinterpret_cast<const float4*>(gr0 + cv.a0); // (only dereferenced as float4 when VEC)
            const float4* st4 = reinterpret_cast<const float4*>(st0 + cv.a0);
            auto fetch = [&](float4& a, float4& b, uint32_t q) {
                if (q < q_hi) {
                    if (VEC) {
                        a = __ldcg(gr4 + q);
                        b = __ldcg(st4 + q);
                    } else {
                        const float* g = reinterpret_cast<const float*>(gr4 + q);
                        const float* t = reinterpret_cast<const float*>(st4 + q);
                        a = make_float4(__ldg(g), __ldg(g + 1), __ldg(g + 2), __ldg(g + 3));
                        b = make_float4(__ldg(t), __ldg(t + 1), __ldg(t + 2), __ldg(t + 3));
                    }
                }
            };
            auto work = [&](const float4& a, const float4& b, uint32_t q, auto skip) {
                const uint32_t k[4] = {key_of(__fsub_rn(a.x, b.x)), key_of(__fsub_rn(a.y, b.y)),
                                       key_of(__fsub_rn(a.z, b.z)), key_of(__fsub_rn(a.w, b.w))};
                reinterpret_cast<uint32_t*>(dc)[q] = active ? acc4(k, skip) : pack_key_codes(k[0], k[1], k[2], k[3]);
            };
            float4 a0, b0, a1, b1, a2, b2, a3, b3;
            uint32_t qb = q_lo + threadIdx.x;
            constexpr uint32_t S = kBigThreads;
            fetch(a0, b0, qb); fetch(a1, b1, qb + S); fetch(a2, b2, qb + 2 * S);
            // four rounds; false when the span ends inside them.  Two forms (with and without the exact zeros), chosen
            // once per four rounds
            auto rounds = [&](auto skip) -> bool {
                fetch(a3, b3, qb + 3 * S); work(a0, b0, qb, skip); qb += S; if (qb >= q_hi) return false;
                fetch(a0, b0, qb + 3 * S); work(a1, b1, qb, skip); qb += S; if (qb >= q_hi) return false;
                fetch(a1, b1, qb + 3 * S); work(a2, b2, qb, skip); qb += S; if (qb >= q_hi) return false;
                fetch(a2, b2, qb + 3 * S); work(a3, b3, qb, skip); qb += S;
                return true;
            };
            const bool zs = active && (wr & kSkipZeros);
            while (qb < q_hi)
                if (!(zs ? rounds(std::true_type{}) : rounds(std::false_type{}))) break;
            if (threadIdx.x < 8) { // ragged edges: [first, min(4 q_lo, len)) and [max(4 q_hi, 4 q_lo), len)
                uint32_t e;
                if (threadIdx.x < 4) { e = cv.first + threadIdx.x; if (e >= min(4 * q_lo, cv.len)) e = 0xffffffffu; }
                else { e = max(4 * q_hi, 4 * q_lo) + (threadIdx.x - 4); if (e >= cv.len) e = 0xffffffffu; }
                if (e != 0xffffffffu) {
                    const uint32_t key = key_of(__fsub_rn(gr0[cv.a0 + e], st0[cv.a0 + e]));
                    dc[e] = (uint8_t)(active ? acc(key) : code_of_key(key));
                }
            }
        }
        if (active) dirty = true;
    }
    if (dirty) flush();
}

// ------------------------------------------------------------------------------------------------
// k_resolve_a: one CTA per (regular layer, worker)
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBigThreads)
k_resolve_a(const LayerDesc* __restrict__ layers, const uint32_t* __restrict__ reg_layers, uint32_t R, uint32_t L,
            const KTab ktab, uint32_t K, const BandMeta* __restrict__ meta,
            const uint32_t* __restrict__ bin_lo, uint32_t* __restrict__ bh_cnt, unsigned long long* __restrict__ bh_sum,
            float* __restrict__ err_out, uint32_t* __restrict__ tau_out, uint32_t* __restrict__ rank_out,
            uint32_t* __restrict__ shift_out, uint32_t* __restrict__ flags, FbList* __restrict__ fb,
            uint2* __restrict__ fb_chunks, uint2* __restrict__ fb_layers, RefineCand* __restrict__ rf,
            uint2* __restrict__ rf_chunks, uint2* __restrict__ rf_layers, uint32_t list_cap, uint32_t w_base) {
    pdl_wait();
    __shared__ uint32_t s_drop[KIMAD_MAX_RATIOS]; // entries not kept by candidate j: n - k_j
    __shared__ int s_loose;
    constexpr int kGroups32 = (kMaxBins + 31) / 32;
    __shared__ uint32_t s_gc[kGroups32]; // per group of 32 bins: entries, then the entries of the groups below it
    __shared__ double s_gs[kGroups32];   // ... and their squares
    __shared__ uint32_t s_w32[32];
    __shared__ double s_w64[32];
    __shared__ int s_bad;
    const uint32_t r = blockIdx.x, w = w_base + blockIdx.y;
    const uint32_t l = reg_layers[r];
    const size_t wr = (size_t)w * R + r, wl = (size_t)w * L + l;
    const BandMeta mt = meta[wr];
    const LayerDesc ld = layers[l];
    if (threadIdx.x == 0) { s_bad = mt.flagged; s_loose = 0; }
    if (threadIdx.x < K) {
        const uint64_t k = ktab.at(w, (size_t)l * K + threadIdx.x);
        s_drop[threadIdx.x] = (uint32_t)(ld.n - k);
    }
    __syncthreads();
    if (!mt.flagged) {
        const uint32_t nb = mt.n_bins, ngrp = (nb + 31u) >> 5; // groups of 32 consecutive bins (ascending keys)
        const uint32_t* blo = bin_lo + wr * (kMaxBins + 1);
        uint32_t* gc = bh_cnt + wr * kMaxBins;
        unsigned long long* gs = bh_sum + wr * kMaxBins;
        const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
        auto bin_sq = [&](uint32_t b) { // the sweep summed squares in units of 2^8 sq_fixed
            return (double)gs[b] * (256.0 * sq_scale(blo[b] >> 23));
        };
        // (1) entries and squares of every group; (2) exclusive prefixes over the groups; (3) a warp per candidate:
        // the group where the running count passes n - k_j by bisection over the prefixes, then the bin inside it
        bool nonfinite = false;
        for (uint32_t g = wid; g < ngrp; g += kBigThreads / 32) {
            const uint32_t bb = 32u * g + lane;
            uint32_t c = 0;
            double sv = 0.0;
            if (bb < nb) {
                c = gc[bb];
                if (c) { sv = bin_sq(bb); nonfinite |= blo[bb] >= 0x7f800000u; }
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                c += __shfl_xor_sync(0xffffffffu, c, o);
                sv += __shfl_xor_sync(0xffffffffu, sv, o);
            }
            if (lane == 0) { s_gc[g] = c; s_gs[g] = sv; }
        }
        if (nonfinite) atomicOr(&flags[w], 1u);
        __syncthreads();
        uint32_t counted;
        {
            const uint32_t c = threadIdx.x < ngrp ? s_gc[threadIdx.x] : 0u;
            const double sv = threadIdx.x < ngrp ? s_gs[threadIdx.x] : 0.0;
            const uint32_t ec = block_excl_scan<uint32_t, kBigThreads>(c, s_w32, &counted);
            const double es = block_excl_scan<double, kBigThreads>(sv, s_w64, nullptr);
            __syncthreads();
            if (threadIdx.x < ngrp) { s_gc[threadIdx.x] = ec; s_gs[threadIdx.x] = es; }
        }
        __syncthreads();
        const uint32_t zeros = (uint32_t)ld.n - counted; // the sweep leaves exact zeros out of its histogram
        for (uint32_t j = wid; j < K; j += kBigThreads / 32) {
            const size_t o = wl * K + j;
            const uint32_t dj = s_drop[j];
            if (lane == 0) rf[o].shift = kNoRefine;
            if (dj == 0 || dj < zeros) { // everything kept; or the threshold is 0 and nothing but zeros is dropped
                if (lane == 0) { err_out[o] = 0.f; tau_out[o] = 0; rank_out[o] = dj ? zeros - dj : 0u; shift_out[o] = 0; }
                continue;
            }
            const uint32_t target = dj - zeros; // entries of the histogram that are dropped, counted from the bottom
            uint32_t lo = 0, hi = ngrp - 1;     // the last group whose prefix does not exceed the target
            while (lo < hi) { const uint32_t mid = (lo + hi + 1) >> 1; if (s_gc[mid] <= target) lo = mid; else hi = mid - 1; }
            const uint32_t bin = 32u * lo + lane;
            uint32_t c = 0;
            double sv = 0.0;
            if (bin < nb) { c = gc[bin]; if (c) sv = bin_sq(bin); }
            uint32_t ic = c;
            double is = sv;
#pragma unroll
            for (int q = 1; q < 32; q <<= 1) {
                const uint32_t yc = __shfl_up_sync(0xffffffffu, ic, q);
                const double ys = __shfl_up_sync(0xffffffffu, is, q);
                if (lane >= (uint32_t)q) { ic += yc; is += ys; }
            }
            const uint32_t before = s_gc[lo] + ic - c;
            double ex_s = __shfl_up_sync(0xffffffffu, is, 1); // exclusive value from the left neighbour: no cancellation
            if (lane == 0) ex_s = 0.0;
            const double below = s_gs[lo] + ex_s;
            const bool mine = c && target >= before && target - before < c; // this bin holds the threshold
            if (!__ballot_sync(0xffffffffu, mine)) { if (lane == 0) atomicMax(&s_bad, 3); continue; }
            if (!mine) continue;
            if (blo[bin] & kGapBit) { atomicMax(&s_bad, 3); continue; } // outside its band
            const uint32_t klo = blo[bin], width = (blo[bin + 1] & ~kGapBit) - klo;
            const uint32_t cb = c, drop = target - before; // entries of the bin that are not kept, < cb
            const double vlo = (double)__uint_as_float(klo);
            // the dropped entries are the `drop` smallest of the bin: their squares sum to something in
            // [drop * vlo^2, drop * mean]; take the midpoint and certify the half-width
            const double upper = sv * ((double)drop / (double)cb);
            const double lower = (double)drop * vlo * vlo;
            double part = 0.5 * (upper + lower), slack = 0.5 * (upper - lower);
            if (drop == 0 || width == 1) { part = lower; slack = 0.0; }
            const double e = below + part;
            if (slack > e * 5e-6) { // acceptance bound on the curve is 1e-5: this candidate's bin is looked at once more
                if (klo == 0u && zeros) { atomicMax(&s_bad, 4); continue; } // (not a bin whose zeros were left out)
                s_loose = 1;
                atomicAdd(&fb->loose_j[j], 1u);
                rf[o] = RefineCand{klo, (uint32_t)(31 - __clz(width)), cb, drop, below};
                continue;
            }
            err_out[o] = (float)e;
            tau_out[o] = klo;
            rank_out[o] = cb - drop;
            shift_out[o] = 31 - __clz(width);
        }
        __syncthreads();
        for (uint32_t bb = threadIdx.x; bb < nb; bb += kBigThreads) // clean for the next step
            if (gc[bb]) { gc[bb] = 0; gs[bb] = 0ull; }
    }
    __syncthreads();
    const int bad = s_bad;
    __shared__ uint32_t s_at;
    if (bad) { // hand the layer and its chunks to the exact path
        if (threadIdx.x == 0) {
            s_at = atomicAdd(&fb->n_chunks, ld.n_chunks);
            fb_layers[atomicAdd(&fb->n_layers, 1u)] = make_uint2(w, l);
            atomicAdd(&fb->total_layers, 1u);
            atomicAdd(&fb->why[bad - 1], 1u);
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < ld.n_chunks; i += kBigThreads)
            if (KIMAD_CHECK(s_at + i < list_cap, 2)) fb_chunks[s_at + i] = make_uint2(w, ld.first_chunk + i);
    } else if (s_loose) { // only loose bounds: refine those candidates
        if (threadIdx.x == 0) {
            s_at = atomicAdd(&fb->rf_chunks, ld.n_chunks);
            rf_layers[atomicAdd(&fb->rf_layers, 1u)] = make_uint2(w, l);
            atomicAdd(&fb->refined, 1u);
        }
        __syncthreads();
        for (uint32_t i = threadIdx.x; i < ld.n_chunks; i += kBigThreads)
            if (KIMAD_CHECK(s_at + i < list_cap, 2)) rf_chunks[s_at + i] = make_uint2(w, ld.first_chunk + i);
    }
}

// ------------------------------------------------------------------------------------------------
// Refinement of loose candidates: the bin that holds such a candidate's threshold is cut into up to 1024 pieces, and
// the entries of the bin -- found by their code byte, completed from the inputs -- are counted and their squares
// summed per piece (the level-2/3 arrays of the exact path serve as storage: a layer is never on both paths at once).
// Costs one pass over the layer's code bytes instead of the exact path's three passes over its inputs.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 6)
k_refine_hist(DSource dbuf, const Chunk* __restrict__ chunks, uint64_t dstride, uint32_t L, uint32_t K,
              const FbList* __restrict__ fb, const uint2* __restrict__ rf_chunks, const RefineCand* __restrict__ rf,
              const CodeSpace codes, uint32_t* __restrict__ g_cnt, unsigned long long* __restrict__ g_ss) {
    pdl_wait();
    __shared__ uint32_t s_klo[KIMAD_MAX_RATIOS], s_shift[KIMAD_MAX_RATIOS], s_j[KIMAD_MAX_RATIOS];
    __shared__ uint32_t s_mask[4]; // the 7-bit codes of the loose candidates' bins
    __shared__ uint32_t s_n;
    const uint32_t n = fb->rf_chunks;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint2 e = rf_chunks[it];
        const Chunk ch = chunks[e.y];
        const size_t wl = (size_t)e.x * L + ch.layer;
        __syncthreads();
        if (threadIdx.x < 4) s_mask[threadIdx.x] = 0;
        if (threadIdx.x == 0) s_n = 0;
        __syncthreads();
        if (threadIdx.x == 0) { // the layer's loose candidates in order of j, every bin once (under its lowest j)
            uint32_t p = 0;
            for (uint32_t j = 0; j < K; ++j) {
                const RefineCand rc = rf[wl * K + j];
                if (rc.shift == kNoRefine || (p && s_klo[p - 1] == rc.klo)) continue; // thresholds descend with j
                s_klo[p] = rc.klo; s_shift[p] = rc.shift; s_j[p] = j;
                ++p;
                const uint32_t code = codes.code(e.x, ch.layer, rc.klo) & 127u;
                s_mask[code >> 5] |= 1u << (code & 31u);
            }
            s_n = p;
        }
        __syncthreads();
        const uint32_t nc = s_n;
        const uint32_t m0 = s_mask[0], m1 = s_mask[1], m2 = s_mask[2], m3 = s_mask[3];
        const ChunkView cv(ch);
        const DView dd(dbuf, e.x, dstride, cv.a0);
        auto wanted = [&](uint32_t code) -> bool {
            const uint32_t word = code < 64u ? (code < 32u ? m0 : m1) : (code < 96u ? m2 : m3);
            return (word >> (code & 31u)) & 1u;
        };
        auto place = [&](uint32_t key) { // the entry's piece, if it lies in one of the loose bins
            for (uint32_t p = 0; p < nc; ++p) {
                const uint32_t d1 = key - s_klo[p], sh = s_shift[p];
                if (d1 < (1u << sh)) {
                    const size_t at = (wl * K + s_j[p]) * kL23Bins + (d1 >> (sh > 10u ? sh - 10u : 0u));
                    atomicAdd(&g_cnt[at], 1u);
                    atomicAdd(&g_ss[at], (unsigned long long)sq_fixed(key));
                    break; // bins are disjoint; candidates that share a bin share a piece histogram (see k_refine_resolve)
                }
            }
        };
        const uint32_t units = (cv.len + 15u) >> 4;
        for (uint32_t u = threadIdx.x; u < units; u += kThreads) {
            const uint32_t e0 = 16u * u;
            uint32_t hit = 0; // the unit's elements whose code is one of the loose bins' codes
            if (e0 >= cv.first && e0 + 16u <= cv.len) {
                const uint4 a = __ldcs(reinterpret_cast<const uint4*>(dd.code) + u);
                const uint32_t x[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        if (wanted((x[i] >> (8 * b)) & 127u)) hit |= 1u << (4 * i + b);
            } else {
                for (uint32_t x = max(e0, cv.first); x < min(e0 + 16u, cv.len); ++x)
                    if (wanted(dd.code[x] & 127u)) hit |= 1u << (x - e0);
            }
            while (hit) { // completed from the inputs four at a time: their loads are independent
                uint32_t pos[4];
                float v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    pos[i] = hit ? (uint32_t)__ffs(hit) - 1u : 0xffffffffu;
                    if (hit) hit &= hit - 1u;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = pos[i] != 0xffffffffu ? dd.at(e0 + pos[i]) : 0.f;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (pos[i] != 0xffffffffu) place(key_of(v[i]));
            }
        }
    }
}

// One CTA per refined layer and pass of the loop; its loose candidates one after the other.  Candidates that share a
// bin were counted into the histogram of the first of them (the lowest j): the later ones read it there.
__global__ void __launch_bounds__(kThreads)
k_refine_resolve(const LayerDesc* __restrict__ layers, uint32_t L, uint32_t K, FbList* __restrict__ fb,
                 const uint2* __restrict__ rf_layers, RefineCand* __restrict__ rf, uint32_t* __restrict__ g_cnt,
                 unsigned long long* __restrict__ g_ss, float* __restrict__ err_out, uint32_t* __restrict__ tau_out,
                 uint32_t* __restrict__ rank_out, uint32_t* __restrict__ shift_out, uint2* __restrict__ fb_chunks,
                 uint2* __restrict__ fb_layers, uint32_t list_cap) {
    pdl_wait();
    __shared__ uint32_t s_w32[8];
    __shared__ double s_w64[8];
    __shared__ int s_bad;
    __shared__ uint32_t s_at;
    const uint32_t n = fb->rf_layers;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint32_t w = rf_layers[it].x, l = rf_layers[it].y;
        const size_t wl = (size_t)w * L + l;
        __syncthreads();
        if (threadIdx.x == 0) s_bad = 0;
        __syncthreads();
        for (uint32_t j = 0; j < K; ++j) {
            const RefineCand rc = rf[wl * K + j];
            if (rc.shift == kNoRefine) continue;
            uint32_t owner = j; // the first loose candidate with this bin holds the pieces
            for (uint32_t i = 0; i < j; ++i) {
                const RefineCand o = rf[wl * K + i];
                if (o.shift != kNoRefine && o.klo == rc.klo) { owner = i; break; }
            }
            const uint32_t sub = rc.shift > 10u ? rc.shift - 10u : 0u, nsub = 1u << (rc.shift - sub);
            const uint32_t* gc = g_cnt + (wl * K + owner) * kL23Bins;
            const unsigned long long* gs = g_ss + (wl * K + owner) * kL23Bins;
            const double scale = sq_scale(rc.klo >> 23);
            // four consecutive pieces per thread, ascending keys
            uint32_t c[4], csum = 0;
            double q[4], qsum = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t b = 4 * threadIdx.x + i;
                c[i] = b < nsub ? gc[b] : 0u;
                q[i] = b < nsub ? (double)gs[b] * scale : 0.0;
                csum += c[i];
                qsum += q[i];
            }
            uint32_t tot;
            uint32_t before = block_excl_scan<uint32_t>(csum, s_w32, &tot);
            double below = block_excl_scan<double>(qsum, s_w64, nullptr);
            if (!KIMAD_CHECK(tot == rc.cb, 7)) s_bad = 1;
            const size_t o = wl * K + j;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (c[i] && rc.drop >= before && rc.drop - before < c[i]) { // the piece that holds the threshold
                    const uint32_t b = 4 * threadIdx.x + i, klo = rc.klo + (b << sub), d2 = rc.drop - before;
                    const double vlo = (double)__uint_as_float(klo);
                    const double upper = q[i] * ((double)d2 / (double)c[i]), lower = (double)d2 * vlo * vlo;
                    double part = 0.5 * (upper + lower), slack = 0.5 * (upper - lower);
                    if (d2 == 0 || sub == 0) { part = lower; slack = 0.0; }
                    const double e = rc.below + below + part;
                    if (slack > e * 5e-6) {
                        s_bad = 1;
                    } else {
                        err_out[o] = (float)e; tau_out[o] = klo; rank_out[o] = c[i] - d2; shift_out[o] = sub;
                    }
                }
                before += c[i];
                below += q[i];
            }
            __syncthreads();
        }
        // clean the pieces, close the candidates
        for (uint32_t j = 0; j < K; ++j) {
            if (rf[wl * K + j].shift == kNoRefine) continue;
            for (uint32_t b = threadIdx.x; b < (uint32_t)kL23Bins; b += kThreads) {
                g_cnt[(wl * K + j) * kL23Bins + b] = 0;
                g_ss[(wl * K + j) * kL23Bins + b] = 0ull;
            }
        }
        __syncthreads();
        for (uint32_t j = threadIdx.x; j < K; j += kThreads) rf[wl * K + j].shift = kNoRefine;
        if (s_bad) { // still too loose (a bin with very many entries): the exact path after all
            const LayerDesc ld = layers[l];
            if (threadIdx.x == 0) {
                s_at = atomicAdd(&fb->n_chunks, ld.n_chunks);
                fb_layers[atomicAdd(&fb->n_layers, 1u)] = make_uint2(w, l);
                atomicAdd(&fb->total_layers, 1u);
                atomicAdd(&fb->why[3], 1u);
            }
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < ld.n_chunks; i += kThreads)
                if (KIMAD_CHECK(s_at + i < list_cap, 2)) fb_chunks[s_at + i] = make_uint2(w, ld.first_chunk + i);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Bitonic sort (descending) of np = 512 .. kTinyMax keys in shared memory with sixteen consecutive keys per thread
// held in registers: compare-exchanges at distances below 16 stay inside a thread, distances 16 .. 256 are a
// shuffle with the thread 1 .. 16 lanes away, and only distances of 512 and more (six of the 78 stages at 4096
// keys) go through shared memory.  The first np / 16 threads hold keys (whole warps: np >= 512); all threads of
// the CTA take part in the barriers.
// ------------------------------------------------------------------------------------------------
template <int STRIDE>
__device__ __forceinline__ void tiny_ce_inside(uint32_t (&v)[16], bool desc) {
#pragma unroll
    for (int e = 0; e < 16; ++e)
        if (!(e & STRIDE)) {
            const uint32_t hi = max(v[e], v[e | STRIDE]), lo = min(v[e], v[e | STRIDE]);
            v[e] = desc ? hi : lo;
            v[e | STRIDE] = desc ? lo : hi;
        }
}
// the stages of the sizes 2 .. 8: direction by the key's position inside the thread
template <int SIZE>
__device__ __forceinline__ void tiny_sort_inside(uint32_t (&v)[16]) {
#pragma unroll
    for (int str = SIZE / 2; str > 0; str >>= 1)
#pragma unroll
        for (int e = 0; e < 16; ++e)
            if (!(e & str)) {
                const uint32_t hi = max(v[e], v[e | str]), lo = min(v[e], v[e | str]);
                const bool desc = (e & SIZE) == 0;
                v[e] = desc ? hi : lo;
                v[e | str] = desc ? lo : hi;
            }
}
__device__ __forceinline__ void tiny_sort_blocked(uint32_t* s_key, uint32_t np) {
    const uint32_t t = threadIdx.x, nthr = np >> 4;
    const bool holds = t < nthr;
    uint32_t v[16];
    if (holds) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 x = reinterpret_cast<const uint4*>(s_key)[4 * t + q];
            v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
        }
        tiny_sort_inside<2>(v); tiny_sort_inside<4>(v); tiny_sort_inside<8>(v);
    }
    for (uint32_t size = 16; size <= np; size <<= 1) { // from here on the direction depends on the thread
        const bool desc = ((16u * t) & size) == 0;
        for (uint32_t str = size >> 1; str >= 16u; str >>= 1) {
            const uint32_t dt = str >> 4;                  // the partner thread is t ^ dt
            const bool keep_max = ((t & dt) == 0) == desc; // the lower position keeps the larger key when descending
            if (dt >= 32u) { // another warp: through shared memory
                __syncthreads(); // s_key is no longer read
                if (holds) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        reinterpret_cast<uint4*>(s_key)[4 * t + q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                }
                __syncthreads();
                if (holds) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint4 x = reinterpret_cast<const uint4*>(s_key)[4 * (t ^ dt) + q];
                        const uint32_t pv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) v[4 * q + i] = keep_max ? max(v[4 * q + i], pv[i]) : min(v[4 * q + i], pv[i]);
                    }
                }
            } else if (holds) { // a lane of the same warp (the warps that hold keys are whole)
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const uint32_t pv = __shfl_xor_sync(0xffffffffu, v[e], dt);
                    v[e] = keep_max ? max(v[e], pv) : min(v[e], pv);
                }
            }
        }
        if (holds) { tiny_ce_inside<8>(v, desc); tiny_ce_inside<4>(v, desc); tiny_ce_inside<2>(v, desc); tiny_ce_inside<1>(v, desc); }
    }
    __syncthreads();
    if (holds) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            reinterpret_cast<uint4*>(s_key)[4 * t + q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// k_tiny_exact: layers of at most kTinyMax elements, sorted in shared memory (one CTA each)
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_tiny_exact(const float* __restrict__ grads, const float* __restrict__ state, uint64_t stride,
             const LayerDesc* __restrict__ layers,
             const uint32_t* __restrict__ tiny_layers, uint32_t L, const KTab ktab, uint32_t K,
             float* __restrict__ err_out, uint32_t* __restrict__ tau_out, uint32_t* __restrict__ rank_out,
             uint32_t* __restrict__ shift_out, uint32_t* __restrict__ flags) {
    pdl_wait();
    extern __shared__ __align__(16) unsigned char tiny_smem[];
    double* s_suf = reinterpret_cast<double*>(tiny_smem);                // [kTinyMax] squares of the entries ranked >= i
    uint32_t* s_key = reinterpret_cast<uint32_t*>(s_suf + kTinyMax);     // [kTinyMax]
    __shared__ double s_w64[8];
    const uint32_t l = tiny_layers[blockIdx.x], w = blockIdx.y;
    const LayerDesc ld = layers[l];
    const uint32_t n = (uint32_t)ld.n;
    // d is recomputed here (the same single subtraction as in the sweep), so that this kernel depends on the
    // step's inputs only and can run beside the sample and sweep kernels
    const float* gr = grads + (size_t)w * stride + ld.begin;
    const float* st = state + (size_t)w * stride + ld.begin;
    uint32_t np = 1;
    while (np < n) np <<= 1;
    bool nonfinite = false;
    for (uint32_t i = threadIdx.x; i < np; i += kThreads) {
        const uint32_t key = i < n ? key_of(__fsub_rn(gr[i], st[i])) : 0u;
        nonfinite |= key >= 0x7f800000u;
        s_key[i] = key;
    }
    if (nonfinite) atomicOr(&flags[w], 1u);
    __syncthreads();
    if (np >= 512u) tiny_sort_blocked(s_key, np);
    else
    for (uint32_t size = 2; size <= np; size <<= 1)       // bitonic sort, descending
        for (uint32_t str = size >> 1; str > 0; str >>= 1) {
            for (uint32_t i = threadIdx.x; i < np / 2; i += kThreads) {
                const uint32_t a = 2 * i - (i & (str - 1)), b = a + str;
                const bool desc = (a & size) == 0;
                const uint32_t ka = s_key[a], kb = s_key[b];
                if ((ka < kb) == desc) { s_key[a] = kb; s_key[b] = ka; }
            }
            __syncthreads();
        }
    // suffix sums of squares, smallest magnitudes first: position q = n-1-i runs over ascending magnitude
    constexpr int PER = kTinyMax / kThreads;
    double loc[PER];
    double sum = 0.0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t q = threadIdx.x * PER + i; // q-th smallest
        double v = 0.0;
        if (q < n) v = (double)__uint_as_float(s_key[n - 1 - q]);
        loc[i] = v * v;
        sum += loc[i];
    }
    double run = block_excl_scan<double>(sum, s_w64, nullptr);
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const uint32_t q = threadIdx.x * PER + i;
        run += loc[i];
        if (q < n) s_suf[n - 1 - q] = run; // squares of the ranks >= n-1-q
    }
    __syncthreads();
    const size_t wl = (size_t)w * L + l;
    for (uint32_t j = threadIdx.x; j < K; j += kThreads) {
        const uint32_t k = (uint32_t)ktab.at(w, (size_t)l * K + j);
        const size_t o = wl * K + j;
        const uint32_t t = s_key[k - 1];
        int lo = 0, hi = (int)k - 1; // first rank whose key equals t
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (s_key[mid] == t) hi = mid; else lo = mid + 1; }
        err_out[o] = k < n ? (float)s_suf[k] : 0.f;
        tau_out[o] = t;
        rank_out[o] = k - (uint32_t)lo;
        shift_out[o] = 0;
    }
}

// ------------------------------------------------------------------------------------------------
// exact radix path over the handed-over chunks.  The list is usually empty, but a handed-over layer may be large and
// may hold one key millions of times (the exact zeros of a sparse gradient): every thread therefore adds up the run
// of consecutive elements of its own that fall into one bin and issues its atomics when the bin changes, and keeps
// four elements' loads in flight.
// ------------------------------------------------------------------------------------------------
constexpr int kFbAhead = 4; // elements per thread whose loads are issued together

__global__ void __launch_bounds__(kThreads)
k_fb_hist1(DSource dbuf, const Chunk* __restrict__ chunks, uint64_t dstride, uint32_t L,
           const FbList* __restrict__ fb, const uint2* __restrict__ fb_chunks, uint32_t* __restrict__ g_cnt,
           unsigned long long* __restrict__ g_ss, uint32_t* __restrict__ flags) {
    pdl_wait();
    __shared__ uint32_t s_cnt[kL1Bins], s_hi[kL1Bins], s_lo[kL1Bins];
    const uint32_t n = fb->n_chunks;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint2 e = fb_chunks[it];
        const Chunk ch = chunks[e.y];
        const ChunkView cv(ch);
        const DView dd(dbuf, e.x, dstride, cv.a0);
        for (int b = threadIdx.x; b < kL1Bins; b += kThreads) { s_cnt[b] = 0; s_hi[b] = 0; s_lo[b] = 0; }
        __syncthreads();
        // a thread sees at most kChunkElems / kThreads elements of a chunk: its two partial sums stay below 2^32
        uint32_t cur = 0, cn = 0, chi = 0, clo = 0;
        bool nonfinite = false;
        auto flush = [&]() {
            if (cn) { atomicAdd(&s_cnt[cur], cn); atomicAdd(&s_hi[cur], chi); atomicAdd(&s_lo[cur], clo); }
        };
        for (uint32_t x0 = cv.first + threadIdx.x; x0 < cv.len; x0 += kFbAhead * kThreads) {
            float v[kFbAhead];
#pragma unroll
            for (int u = 0; u < kFbAhead; ++u) v[u] = x0 + u * kThreads < cv.len ? dd.at(x0 + u * kThreads) : 0.f;
#pragma unroll
            for (int u = 0; u < kFbAhead; ++u) {
                if (x0 + u * kThreads >= cv.len) break;
                const uint32_t key = key_of(v[u]);
                const uint32_t sq = (uint32_t)sq_fixed(key);
                if ((key >> 20) != cur) { flush(); cur = key >> 20; cn = 0; chi = 0; clo = 0; }
                ++cn; chi += sq >> 16; clo += sq & 0xffffu;
                nonfinite |= key >= 0x7f800000u;
            }
        }
        flush();
        if (nonfinite) atomicOr(&flags[e.x], 1u);
        __syncthreads();
        uint32_t* gc = g_cnt + ((size_t)e.x * L + ch.layer) * kL1Bins;
        unsigned long long* gs = g_ss + ((size_t)e.x * L + ch.layer) * kL1Bins;
        for (int b = threadIdx.x; b < kL1Bins; b += kThreads)
            if (s_cnt[b]) {
                atomicAdd(&gc[b], s_cnt[b]);
                atomicAdd(&gs[b], ((unsigned long long)s_hi[b] << 16) + s_lo[b]);
            }
        __syncthreads();
    }
}

template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_fb_hist23(DSource dbuf, const Chunk* __restrict__ chunks, uint64_t dstride, uint32_t L, uint32_t K,
            const FbList* __restrict__ fb, const uint2* __restrict__ fb_chunks, const SlotTab* __restrict__ slots,
            uint32_t* __restrict__ g_cnt, unsigned long long* __restrict__ g_ss) {
    pdl_wait();
    __shared__ uint8_t s_first[kL1Bins]; // level-1 bin -> first slot whose prefix starts with it (0xff: none)
    __shared__ uint8_t s_num[kL1Bins];   // ... and how many consecutive slots share that bin (level 3)
    __shared__ uint32_t s_prefix[KIMAD_MAX_RATIOS];
    const uint32_t n = fb->n_chunks;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint2 e = fb_chunks[it];
        const Chunk ch = chunks[e.y];
        const size_t wl = (size_t)e.x * L + ch.layer;
        const SlotTab& stab = slots[wl];
        const uint32_t ns = stab.n;
        for (int b = threadIdx.x; b < kL1Bins; b += kThreads) { s_first[b] = 0xff; s_num[b] = 0; }
        for (uint32_t s = threadIdx.x; s < ns; s += kThreads) s_prefix[s] = stab.prefix[s];
        __syncthreads();
        if (threadIdx.x == 0)
            for (uint32_t s = 0; s < ns; ++s) {
                const uint32_t b1 = LEVEL == 2 ? s_prefix[s] : (s_prefix[s] >> 10);
                if (s_first[b1] == 0xff) s_first[b1] = (uint8_t)s;
                s_num[b1]++;
            }
        __syncthreads();
        const ChunkView cv(ch);
        const DView dd(dbuf, e.x, dstride, cv.a0);
        uint32_t* gc = g_cnt + wl * K * kL23Bins;
        unsigned long long* gs = g_ss + wl * K * kL23Bins;
        uint32_t cur = 0xffffffffu, cn = 0; // (slot, bin) of the thread's current run, its entries and squares
        unsigned long long csq = 0;
        auto flush = [&]() {
            if (cn) {
                atomicAdd(&gc[cur], cn);
                if (LEVEL == 2) atomicAdd(&gs[cur], csq);
            }
        };
        for (uint32_t x0 = cv.first + threadIdx.x; x0 < cv.len; x0 += kFbAhead * kThreads) {
            float v[kFbAhead];
#pragma unroll
            for (int u = 0; u < kFbAhead; ++u) v[u] = x0 + u * kThreads < cv.len ? dd.at(x0 + u * kThreads) : 0.f;
#pragma unroll
            for (int u = 0; u < kFbAhead; ++u) {
                if (x0 + u * kThreads >= cv.len) break;
                const uint32_t key = key_of(v[u]);
                const uint32_t f = s_first[key >> 20];
                if (f == 0xff) continue;
                uint32_t at = 0xffffffffu;
                if (LEVEL == 2) {
                    at = f * (uint32_t)kL23Bins + ((key >> 10) & 1023u);
                } else {
                    const uint32_t nn = s_num[key >> 20], p21 = key >> 10;
                    for (uint32_t s = f; s < f + nn; ++s)
                        if (s_prefix[s] == p21) { at = s * (uint32_t)kL23Bins + (key & 1023u); break; }
                    if (at == 0xffffffffu) continue;
                }
                if (at != cur) { flush(); cur = at; cn = 0; csq = 0; }
                ++cn;
                if (LEVEL == 2) csq += (unsigned long long)sq_fixed(key);
            }
        }
        flush();
        __syncthreads();
    }
}

} // namespace kimad
