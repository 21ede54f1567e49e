// Stages (d)-(f): Top-K selection at the chosen k, ordered sparse pack, EF21 update.
//
// After the DP every (worker, layer) knows a key interval [lo, lo + 2^shift) that contains its
// threshold and the rank of the threshold inside that interval (shift = 0 when the curve stage already
// resolved all 31 bits).  One sweep over the byte codes the curve stage left (k_sel_count) counts, per 2048-element slice,
// the entries above the interval, remembers the few entries inside it and marks the 32-element groups that
// can hold a kept entry; k_sel_resolve turns the remembered entries (or their per-layer histogram) into the
// exact threshold; k_sel_slices and k_sel_scan derive every slice's and chunk's output offset and leave one
// job record per chunk; k_sel_write compacts in index order and updates the estimator, reading only the
// marked groups of sparse slices.  No kernel waits on another: offsets come from stored counts.
#pragma once
#include "kimad_curve.cuh"

namespace kimad {

constexpr int kListCap = 32;                    // in-interval entries remembered per chunk
constexpr uint32_t kListOverflow = 0xffffffffu; // more than that: the chunk is recounted exactly
constexpr int kLowBins = 1024;                  // bins of the in-interval histogram

// A chunk (at most 32768 elements from its 16-byte aligned start) is cut into 16 slices of 2048 elements; in
// the sweeps of this stage a warp works on a slice by itself, so no sweep needs a block-wide barrier.
constexpr int kSliceElems = 2048;
constexpr int kSlices = 16;
constexpr int kSparseGroups = 32; // the write sweep reads a slice group by group when at most this many are marked

struct ChunkSel { // per (worker, chunk)
    uint32_t n_in;             // entries inside the interval, or kListOverflow
    uint16_t above[kSlices];   // per slice: entries whose key lies above the interval; after k_sel_scan: entries kept
                               // before the slice inside the chunk
    uint16_t eq[kSlices];      // after k_sel_recount / k_sel_scan: entries equal to tau per slice, then before the slice
    uint32_t low[kListCap];    // the entries inside the interval: slice << 16 | (key - lo), any order
    uint32_t _pad;
    uint64_t mask[kSlices];    // per slice: bit g set when the 32-element group g may hold a kept entry (key >= the
                               // interval's lower end); a superset of the groups the write sweep has to read
};

// Everything the write sweep needs to know about a (worker, chunk) besides the data, gathered by k_sel_scan so
// that the write sweep starts from loads whose addresses depend on the block index only.
struct ChunkJob {
    uint32_t mode;      // 0: nothing of this chunk is kept; 1: threshold tau; 2: the whole layer is kept
    uint32_t tau;
    uint32_t keep_eq;   // entries equal to tau that are kept, over the layer (lowest indices first)
    uint32_t gt_before; // entries above tau in the layer's earlier chunks
    uint32_t eq_before; // entries equal to tau in the layer's earlier chunks
    uint32_t cnt_gt;    // entries above tau / equal to tau in this chunk
    uint32_t cnt_eq;
    uint32_t idx0;      // layer-local index of the chunk's aligned start (may wrap; added back by the sweep)
    uint64_t base;      // first output position of the layer in the worker's packed buffers
};

// Second round of the select stage: layers whose interval was wider than 2^10 keys and whose entries
// inside it could not be collected (a chunk list overflowed, or more than kSortCap entries) get their
// interval narrowed by the coarse histogram and are counted once more over their own chunks.
struct Round2 {
    uint32_t n_chunks;
    uint32_t n_layers;
    uint32_t _pad[2];
};
constexpr int kSortCap = 4096;

// ------------------------------------------------------------------------------------------------
// Counting sweep of one chunk: warp w takes the slices w and w + 8.
__device__ __forceinline__ void sel_count_chunk(const DSource& dbuf, const Chunk& ch, uint32_t w,
                                                uint32_t chunk_id, uint32_t n_chunks, uint64_t dstride, uint32_t L,
                                                const Sel* __restrict__ sel, const LayerDesc* __restrict__ layers,
                                                ChunkSel* __restrict__ csel, uint32_t* __restrict__ low_hist,
                                                uint32_t* __restrict__ recount_n, uint2* __restrict__ recount_list,
                                                uint32_t list_cap, uint32_t* s_n, uint32_t* s_low) {
    const size_t wl = (size_t)w * L + ch.layer;
    const Sel s = sel[wl];
    ChunkSel* out = csel + (size_t)w * n_chunks + chunk_id;
    const ChunkView cv(ch);
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (s.k == 0 || (uint64_t)s.k == layers[ch.layer].n) { // nothing / everything kept: no need to look at the data
        if (threadIdx.x < kSlices) {
            const uint32_t lo = max(cv.first, threadIdx.x * kSliceElems), hi = min(cv.len, (threadIdx.x + 1) * kSliceElems);
            out->above[threadIdx.x] = (uint16_t)((s.k && hi > lo) ? hi - lo : 0u);
            out->eq[threadIdx.x] = 0;
        }
        if (threadIdx.x == 0) out->n_in = 0;
        return;
    }
    const uint32_t lo = s.tau, width = 1u << s.shift;
    const uint32_t hshift = s.shift > 10 ? s.shift - 10 : 0; // the histogram has at most kLowBins bins
    const bool exact = s.shift == 0;
    if (threadIdx.x == 0) *s_n = 0;
    uint32_t* gh = low_hist + wl * kLowBins; // the layer's in-interval histogram: few entries, counted in place
    __syncthreads();
    const DView dd(dbuf, w, dstride, cv.a0);
    // Codes first: an entry whose code (the byte the sweep left for it) is larger than the code of the interval's
    // keys lies above the interval, one with a smaller code below; only entries with the interval's own code are
    // completed from the inputs.  Codes are 7-bit numbers, so "x >= t" for the four bytes of a word is bit 7 of
    // every byte of x + (0x80 - t) * 0x01010101.
    const uint32_t add_gt = (0x80u - (s.code + 1u)) * 0x01010101u, add_ge = (0x80u - s.code) * 0x01010101u;
    for (uint32_t sl = wid; sl < (uint32_t)kSlices; sl += kThreads / 32) {
        uint32_t above = 0; // low half: entries above the interval; high half: entries equal to an exact threshold
        uint64_t mask = 0;
        auto visit = [&](uint32_t key) -> bool { // true: the key is not below the interval
            const uint32_t d1 = key - lo; // wraps to >= 2^31 for keys below the interval
            if (d1 < width) {
                // an exact threshold needs no list and no histogram, only the slice's number of equal entries (there
                // may be millions of them: the exact zeros of a sparse gradient)
                if (exact) {
                    above += 0x10000u;
                } else {
                    if (KIMAD_CHECK((d1 >> hshift) < (uint32_t)kLowBins, 1)) atomicAdd(&gh[d1 >> hshift], 1u);
                    const uint32_t p = atomicAdd(s_n, 1u);
                    if (p < (uint32_t)kListCap) s_low[p] = (sl << 16) | d1;
                }
            } else {
                above += d1 < 0x80000000u;
            }
            return d1 < 0x80000000u;
        };
        // a lane takes sixteen consecutive codes (one 128-bit load) of each of the slice's four rows of 512 elements;
        // a 32-element group is a pair of lanes
        constexpr int ROWS = kSliceElems / 512;
        const uint32_t u0 = sl * (kSliceElems / 16) + lane; // this lane's 16-element unit in row 0
        uint4 a[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const uint32_t e0 = 16 * (u0 + r * 32);
            if (e0 >= cv.first && e0 + 16 <= cv.len) a[r] = __ldcs(reinterpret_cast<const uint4*>(dd.code) + u0 + r * 32);
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const uint32_t e0 = 16 * (u0 + r * 32);
            bool f = false; // this lane holds an entry that is not below the interval
            if (e0 >= cv.first && e0 + 16 <= cv.len) {
                const uint32_t x[4] = {a[r].x, a[r].y, a[r].z, a[r].w};
                uint32_t ge[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) ge[j] = (x[j] + add_ge) & 0x80808080u;
                if (ge[0] | ge[1] | ge[2] | ge[3]) { // with a sparse budget few lanes hold a code that is not below the interval's
                    uint32_t hit = 0; // rare: the unit's entries with the interval's own code, bit k -> element k
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t gt = (x[j] + add_gt) & 0x80808080u;
                        above += __popc(gt);
                        f |= gt != 0; // entries with the interval's code mark the group only if they are not below it
                        const uint32_t border = ge[j] ^ gt; // bit 8 k + 7 -> element k of this word
                        hit |= (((border >> 7) & 1u) | ((border >> 14) & 2u) | ((border >> 21) & 4u) | ((border >> 28) & 8u)) << (4 * j);
                    }
                    while (hit) { // completed from the inputs two at a time: their loads are independent
                        const uint32_t p0 = __ffs(hit) - 1;
                        hit &= hit - 1;
                        const uint32_t p1 = hit ? __ffs(hit) - 1 : p0;
                        hit &= hit - 1; // (0 stays 0)
                        const float v0 = dd.at(e0 + p0), v1 = dd.at(e0 + p1);
                        f |= visit(key_of(v0));
                        if (p1 != p0) f |= visit(key_of(v1));
                    }
                }
            } else if (e0 < cv.len) { // ragged first or last unit of the chunk
                for (uint32_t e = e0; e < e0 + 16; ++e)
                    if (e >= cv.first && e < cv.len) f |= visit(key_of(dd.at(e)));
            }
            uint32_t m = __ballot_sync(0xffffffffu, f);
            if (m) { // pairs of lanes -> 16 group bits of this row
                m = (m | (m >> 1)) & 0x55555555u;
                m = (m | (m >> 1)) & 0x33333333u;
                m = (m | (m >> 2)) & 0x0f0f0f0fu;
                m = (m | (m >> 4)) & 0x00ff00ffu;
                m = (m | (m >> 8)) & 0x0000ffffu;
                mask |= (uint64_t)m << (16 * r);
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) above += __shfl_xor_sync(0xffffffffu, above, o);
        if (lane == 0) { out->above[sl] = (uint16_t)above; out->eq[sl] = (uint16_t)(above >> 16); out->mask[sl] = mask; }
    }
    __syncthreads();
    const uint32_t n_in = *s_n;
    if (threadIdx.x < min(n_in, (uint32_t)kListCap)) out->low[threadIdx.x] = s_low[threadIdx.x];
    if (threadIdx.x == 0) {
        if (n_in <= (uint32_t)kListCap) {
            out->n_in = n_in;
        } else {
            out->n_in = kListOverflow;
            const uint32_t at = atomicAdd(recount_n, 1u);
            // capacity: a chunk can be listed once per select round
            if (KIMAD_CHECK(at < list_cap, 2)) recount_list[at] = make_uint2(w, chunk_id);
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads, 6)
k_sel_count(DSource dbuf, const Chunk* __restrict__ chunks, uint32_t n_chunks, uint64_t dstride,
            uint32_t L, const Sel* __restrict__ sel, const LayerDesc* __restrict__ layers, ChunkSel* __restrict__ csel,
            uint32_t* __restrict__ low_hist, uint32_t* __restrict__ recount_n, uint2* __restrict__ recount_list,
            uint32_t list_cap, uint32_t w_base) {
    pdl_wait();
    __shared__ uint32_t s_n;
    __shared__ uint32_t s_low[kListCap];
    sel_count_chunk(dbuf, chunks[blockIdx.x], w_base + blockIdx.y, blockIdx.x, n_chunks, dstride, L, sel, layers, csel, low_hist,
                    recount_n, recount_list, list_cap, &s_n, s_low);
}

// second round: only the chunks of the layers listed in r2
__global__ void __launch_bounds__(kThreads)
k_sel_count_r2(DSource dbuf, const Chunk* __restrict__ chunks, uint32_t n_chunks, uint64_t dstride,
               uint32_t L, const Sel* __restrict__ sel, const LayerDesc* __restrict__ layers,
               ChunkSel* __restrict__ csel, uint32_t* __restrict__ low_hist, uint32_t* __restrict__ recount_n,
               uint2* __restrict__ recount_list, uint32_t list_cap, const Round2* __restrict__ r2,
               const uint2* __restrict__ r2_chunks) {
    pdl_wait();
    __shared__ uint32_t s_n;
    __shared__ uint32_t s_low[kListCap];
    const uint32_t n = r2->n_chunks;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint2 e = r2_chunks[it];
        sel_count_chunk(dbuf, chunks[e.y], e.x, e.y, n_chunks, dstride, L, sel, layers, csel, low_hist, recount_n,
                        recount_list, list_cap, &s_n, s_low);
    }
}

// Exact threshold of one (worker, layer) from what the counting sweep left behind.  The whole CTA works on it.
// first round: may narrow the interval and list the layer for the second round; second round: the interval is at
// most 32 keys wide and the histogram is exact.
__device__ __forceinline__ void sel_resolve_layer(uint32_t l, uint32_t w, uint32_t L, const LayerDesc* __restrict__ layers,
                                                  uint32_t n_chunks, const ChunkSel* __restrict__ csel,
                                                  uint32_t* __restrict__ low_hist, Sel* __restrict__ sel, bool round1,
                                                  Round2* __restrict__ r2, uint2* __restrict__ r2_layers,
                                                  uint2* __restrict__ r2_chunks, uint32_t* s_key /* [kSortCap] */,
                                                  uint32_t* s_w32, uint32_t* s_n, uint32_t* s_over) {
    const size_t wl = (size_t)w * L + l;
    const LayerDesc ld = layers[l];
    Sel s = sel[wl];
    if (s.k == 0 || (uint64_t)s.k == ld.n) return;
    uint32_t* gh = low_hist + wl * kLowBins;
    const uint32_t hshift = s.shift > 10 ? s.shift - 10 : 0;
    if (s.shift == 0) { // already exact: bin 0 holds the number of entries equal to tau
        if (threadIdx.x == 0) gh[0] = 0;
        return;
    }
    bool sorted = false;
    if (round1) { // collect the entries inside the interval from the chunk lists and sort them
        if (threadIdx.x == 0) { *s_n = 0; *s_over = 0; }
        __syncthreads();
        const ChunkSel* cs = csel + (size_t)w * n_chunks + ld.first_chunk;
        for (uint32_t i = threadIdx.x; i < ld.n_chunks; i += kThreads) {
            const uint32_t n_in = cs[i].n_in;
            if (n_in == kListOverflow) { *s_over = 1; continue; }
            if (!n_in) continue;
            const uint32_t at = atomicAdd(s_n, n_in);
            if (at + n_in > (uint32_t)kSortCap) { *s_over = 1; continue; }
            for (uint32_t e = 0; e < n_in; ++e) s_key[at + e] = cs[i].low[e] & 0xffffu;
        }
        __syncthreads();
        sorted = !*s_over;
        if (sorted) {
            // the rank-th largest of the collected entries (16-bit numbers) by two 8-bit digits: a histogram of the
            // upper digit, then one of the lower digit among the entries that share the upper digit found
            const uint32_t cnt = *s_n;
            static_assert(kThreads == 256, "one thread per digit");
            __shared__ uint32_t s_h[256];
            __shared__ uint32_t s_digit, s_gt;
            uint32_t rank = s.keep_eq, hi_digit = 0, greater = 0; // rank <= cnt by construction
            for (int pass = 0; pass < 2; ++pass) {
                s_h[threadIdx.x] = 0; // kThreads == 256
                __syncthreads();
                for (uint32_t i = threadIdx.x; i < cnt; i += kThreads) {
                    const uint32_t k = s_key[i];
                    if (pass == 0) atomicAdd(&s_h[k >> 8], 1u);
                    else if ((k >> 8) == hi_digit) atomicAdd(&s_h[k & 255u], 1u);
                }
                __syncthreads();
                if (threadIdx.x < 32) { // warp 0: lane L takes the digits 255 - 8 L down to 248 - 8 L
                    const uint32_t lane = threadIdx.x, top = 255u - 8u * lane;
                    uint32_t mine = 0;
#pragma unroll
                    for (uint32_t j = 0; j < 8; ++j) mine += s_h[top - j];
                    uint32_t incl = mine;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= (uint32_t)o) incl += y;
                    }
                    const uint32_t hit = __ballot_sync(0xffffffffu, incl >= rank);
                    if (hit && lane == (uint32_t)(__ffs(hit) - 1)) {
                        uint32_t acc = incl - mine, d = top;
                        while (acc + s_h[d] < rank) { acc += s_h[d]; --d; }
                        s_digit = d;
                        s_gt = acc; // entries of this pass's candidates with a larger digit
                    }
                }
                __syncthreads();
                if (pass == 0) { hi_digit = s_digit; greater = s_gt; rank -= s_gt; }
                else { greater += s_gt; }
            }
            if (threadIdx.x == 0) {
                const uint32_t t = (hi_digit << 8) | s_digit;
                s.tau_low = t;
                s.tau += t;
                s.keep_eq = s.keep_eq - greater; // rank among the entries equal to t: those above t come first
                s.shift = 0;
                sel[wl] = s;
            }
        }
    }
    __syncthreads();
    if (!sorted) { // histogram of the interval: exact when it has at most kLowBins keys, else it narrows the interval
        uint32_t* s_incl = s_key; // [kLowBins], reuse
        for (int b = threadIdx.x; b < kLowBins; b += kThreads) s_incl[kLowBins - 1 - b] = gh[b];
        __syncthreads();
        scan_bins<kLowBins>(s_incl, nullptr, s_w32, nullptr);
        if (threadIdx.x == 0) {
            const int p = find_pos<kLowBins>(s_incl, s.keep_eq); // keep_eq holds the rank inside the interval
            const uint32_t above = p ? s_incl[p - 1] : 0u;
            const uint32_t bin = (uint32_t)(kLowBins - 1 - p);
            s.keep_eq -= above;
            s.tau += bin << hshift;
            s.tau_low = hshift ? 0u : bin;
            s.shift = hshift;
            sel[wl] = s;
        }
        if (hshift) { // not exact yet: the layer and its chunks go to the second round
            __shared__ uint32_t s_at;
            if (threadIdx.x == 0) {
                s_at = atomicAdd(&r2->n_chunks, ld.n_chunks);
                r2_layers[atomicAdd(&r2->n_layers, 1u)] = make_uint2(w, l);
            }
            __syncthreads();
            for (uint32_t i = threadIdx.x; i < ld.n_chunks; i += kThreads) r2_chunks[s_at + i] = make_uint2(w, ld.first_chunk + i);
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kLowBins; b += kThreads) gh[b] = 0; // clean for the next use
    __syncthreads();
}

__global__ void __launch_bounds__(kThreads)
k_sel_resolve(uint32_t L, const LayerDesc* __restrict__ layers, uint32_t n_chunks, const ChunkSel* __restrict__ csel,
              uint32_t* __restrict__ low_hist, Sel* __restrict__ sel, Round2* __restrict__ r2,
              uint2* __restrict__ r2_layers, uint2* __restrict__ r2_chunks, uint32_t w_base) {
    pdl_wait();
    __shared__ __align__(16) uint32_t s_key[kSortCap];
    __shared__ uint32_t s_w32[8];
    __shared__ uint32_t s_n, s_over;
    sel_resolve_layer(blockIdx.x, w_base + blockIdx.y, L, layers, n_chunks, csel, low_hist, sel, true, r2, r2_layers, r2_chunks, s_key,
                      s_w32, &s_n, &s_over);
}

__global__ void __launch_bounds__(kThreads)
k_sel_resolve_r2(uint32_t L, const LayerDesc* __restrict__ layers, uint32_t n_chunks, const ChunkSel* __restrict__ csel,
                 uint32_t* __restrict__ low_hist, Sel* __restrict__ sel, Round2* __restrict__ r2,
                 uint2* __restrict__ r2_layers, uint2* __restrict__ r2_chunks) {
    pdl_wait();
    __shared__ __align__(16) uint32_t s_key[kSortCap];
    __shared__ uint32_t s_w32[8];
    __shared__ uint32_t s_n, s_over;
    const uint32_t n = r2->n_layers;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x)
        sel_resolve_layer(r2_layers[it].y, r2_layers[it].x, L, layers, n_chunks, csel, low_hist, sel, false, r2, r2_layers,
                          r2_chunks, s_key, s_w32, &s_n, &s_over);
}

// Exact per-slice (gt, eq) of the chunks whose list overflowed: warp w recounts the slices w and w + 8.
__global__ void __launch_bounds__(kThreads)
k_sel_recount(DSource dbuf, const Chunk* __restrict__ chunks, uint32_t n_chunks, uint64_t dstride,
              uint32_t L, const Sel* __restrict__ sel, const uint32_t* __restrict__ recount_n,
              const uint2* __restrict__ recount_list, ChunkSel* __restrict__ csel) {
    pdl_wait();
    const uint32_t n = *recount_n;
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (uint32_t it = blockIdx.x; it < n; it += gridDim.x) {
        const uint2 e = recount_list[it];
        const Chunk ch = chunks[e.y];
        const Sel s = sel[(size_t)e.x * L + ch.layer];
        const ChunkView cv(ch);
        const DView dd(dbuf, e.x, dstride, cv.a0);
        ChunkSel* out = csel + (size_t)e.x * n_chunks + e.y;
        for (uint32_t sl = wid; sl < (uint32_t)kSlices; sl += kThreads / 32) {
            uint32_t gt = 0, eq = 0;
            const uint32_t x0 = max(cv.first, sl * kSliceElems), x1 = min(cv.len, (sl + 1) * kSliceElems);
            for (uint32_t x = x0 + lane; x < x1; x += 32) {
                const uint32_t key = key_of(dd.at(x));
                gt += key > s.tau;
                eq += key == s.tau;
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                gt += __shfl_xor_sync(0xffffffffu, gt, o);
                eq += __shfl_xor_sync(0xffffffffu, eq, o);
            }
            if (lane == 0) { out->above[sl] = (uint16_t)gt; out->eq[sl] = (uint16_t)eq; }
        }
        // The recount is authoritative.  A chunk listed in the first round may have been counted again in the
        // second (narrowed interval) and then own a fresh in-interval list; k_sel_slices must not add that list
        // on top of the exact counts written here.
        if (threadIdx.x == 0) out->n_in = kListOverflow;
    }
}

// Per chunk (one warp each, lane = slice): entries above tau and equal to tau in every slice (from the lists, or
// already recounted), turned into prefixes inside the chunk; chunk_cnt = the chunk's totals.
__global__ void __launch_bounds__(kThreads)
k_sel_slices(const Chunk* __restrict__ chunks, uint32_t n_chunks, uint32_t w_base, uint32_t n_workers, uint32_t L,
             const Sel* __restrict__ sel, ChunkSel* __restrict__ csel, uint2* __restrict__ chunk_cnt) {
    pdl_wait();
    const uint32_t lane = threadIdx.x & 31;
    uint64_t it = (uint64_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (it >= (uint64_t)n_workers * n_chunks) return;
    it += (uint64_t)w_base * n_chunks; // workers w_base .. w_base + n_workers - 1
    const uint32_t w = (uint32_t)(it / n_chunks), ci = (uint32_t)(it % n_chunks);
    const Sel s = sel[(size_t)w * L + chunks[ci].layer];
    ChunkSel& c = csel[it];
    uint32_t g = 0, q = 0;
    if (lane < (uint32_t)kSlices) { g = c.above[lane]; q = c.eq[lane]; }
    const uint32_t n_in = c.n_in;
    if (n_in != kListOverflow)
        for (uint32_t e = 0; e < n_in; ++e) { // entries inside the interval join their slice's counts
            const uint32_t en = c.low[e];
            if ((en >> 16) == lane) {
                g += (en & 0xffffu) > s.tau_low;
                q += (en & 0xffffu) == s.tau_low;
            }
        }
    uint32_t ig = g, iq = q;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t yg = __shfl_up_sync(0xffffffffu, ig, o), yq = __shfl_up_sync(0xffffffffu, iq, o);
        if (lane >= (uint32_t)o) { ig += yg; iq += yq; }
    }
    if (lane < (uint32_t)kSlices) { c.above[lane] = (uint16_t)(ig - g); c.eq[lane] = (uint16_t)(iq - q); }
    if (lane == 31) chunk_cnt[it] = make_uint2(ig, iq);
}

// Exclusive prefix of the chunk totals over the layer's earlier chunks, stored with the layer's threshold as the
// write sweep's job record of every chunk.
__global__ void __launch_bounds__(kThreads)
k_sel_scan(const LayerDesc* __restrict__ layers, const Chunk* __restrict__ chunks, uint32_t n_chunks, uint32_t L,
           const Sel* __restrict__ sel, const uint2* __restrict__ chunk_cnt, ChunkJob* __restrict__ jobs,
           uint32_t* __restrict__ recount_n, FbList* __restrict__ fb, Round2* __restrict__ r2, uint32_t w_base) {
    pdl_wait();
    __shared__ uint32_t s_w[8];
    const LayerDesc ld = layers[blockIdx.x];
    const uint32_t w = w_base + blockIdx.y;
    const Sel s = sel[(size_t)w * L + blockIdx.x];
    const uint2* cc = chunk_cnt + (size_t)w * n_chunks + ld.first_chunk;
    ChunkJob* jb = jobs + (size_t)w * n_chunks + ld.first_chunk;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) { // all work lists (of these workers) have been consumed by now
        *recount_n = 0;
        fb->n_chunks = 0;
        fb->n_layers = 0;
        fb->rf_chunks = 0;
        fb->rf_layers = 0;
        r2->n_chunks = 0;
        r2->n_layers = 0;
    }
    const bool all = (uint64_t)s.k == ld.n;
    uint32_t run_g = 0, run_e = 0;
    for (uint32_t base = 0; base < ld.n_chunks; base += kThreads) {
        const uint32_t i = base + threadIdx.x;
        const uint2 v = i < ld.n_chunks ? cc[i] : make_uint2(0, 0);
        uint32_t tg, te;
        const uint32_t eg = block_excl_scan<uint32_t>(v.x, s_w, &tg);
        const uint32_t ee = block_excl_scan<uint32_t>(v.y, s_w, &te);
        if (i < ld.n_chunks) {
            const ChunkView cv(chunks[ld.first_chunk + i]);
            ChunkJob j;
            j.tau = s.tau;
            j.keep_eq = s.keep_eq;
            j.gt_before = run_g + eg;
            j.eq_before = run_e + ee;
            j.cnt_gt = v.x;
            j.cnt_eq = v.y;
            j.idx0 = (uint32_t)(cv.a0 - ld.begin);
            j.base = s.base;
            const bool none = s.k == 0 || (!all && v.x == 0 && (v.y == 0 || j.eq_before >= s.keep_eq));
            j.mode = none ? 0u : (all ? 2u : 1u);
            jb[i] = j;
        }
        run_g += tg;
        run_e += te;
    }
}

// ------------------------------------------------------------------------------------------------
// (e) + (f).  A warp compacts a slice by itself: every lane owns 16 consecutive elements of a 512-element
// round, so that ranks inside a round follow the index order; positions come from warp scans.
// ------------------------------------------------------------------------------------------------
// DENSE: tuned for steps whose budget keeps more than a few per cent of the entries (the host picks the
// instantiation from the budgets; both are correct for any input).
template <bool BF16, bool DENSE>
__global__ void __launch_bounds__(kThreads, DENSE ? 3 : 8)
k_sel_write(const float* __restrict__ grads, float* __restrict__ state, const Chunk* __restrict__ chunks,
            uint32_t n_chunks, uint64_t dstride, uint64_t stride, const ChunkSel* __restrict__ csel,
            const ChunkJob* __restrict__ jobs, uint64_t cap, uint32_t* __restrict__ out_idx, void* __restrict__ out_val,
            uint32_t w_base) {
    pdl_wait();
    const uint32_t w = w_base + blockIdx.y;
    const ChunkJob jb = jobs[(size_t)w * n_chunks + blockIdx.x];
    if (jb.mode == 0) return; // nothing kept in this chunk
    const Chunk ch = chunks[blockIdx.x];
    const ChunkSel& cs = csel[(size_t)w * n_chunks + blockIdx.x];
    const bool all = jb.mode == 2;
    const uint2 cnt = make_uint2(jb.cnt_gt, jb.cnt_eq), pre = make_uint2(jb.gt_before, jb.eq_before);
    const uint32_t keep_eq = jb.keep_eq;
    const uint32_t tau = jb.tau;
    const ChunkView cv(ch);
    // d is recomputed from the inputs; every element of the estimator is read before this kernel updates it
    const float* gr = grads + (size_t)w * stride + cv.a0;
    float* st = state + (size_t)w * stride + cv.a0;
    uint32_t* oi = out_idx + (size_t)w * cap + jb.base;
    float* ov32 = reinterpret_cast<float*>(out_val) + (size_t)w * cap + jb.base;
    __nv_bfloat16* ov16 = reinterpret_cast<__nv_bfloat16*>(out_val) + (size_t)w * cap + jb.base;
    const uint32_t idx0 = jb.idx0;
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const bool st_vec = ((reinterpret_cast<uintptr_t>(st) | reinterpret_cast<uintptr_t>(gr)) & 15u) == 0; // 128-bit access to both
    __shared__ uint8_t s_pos[kThreads / 32][kSparseGroups]; // per warp: the marked groups of a slice, ascending
    __shared__ uint32_t s_stage[DENSE ? kThreads / 32 : 1][DENSE ? 2 * 16 * 32 : 1]; // per warp: a round's indices, values

    for (uint32_t sl = wid; sl < (uint32_t)kSlices; sl += kThreads / 32) {
        const uint32_t x0 = sl * kSliceElems;
        if (x0 >= cv.len) break;
        // entries equal to tau are kept while their rank among equals (ascending index) is below keep_eq
        const uint32_t gt_before = pre.x + cs.above[sl], eq_before = pre.y + cs.eq[sl];
        const uint32_t gt_here = (sl + 1 < (uint32_t)kSlices ? cs.above[sl + 1] : cnt.x) - cs.above[sl];
        const uint32_t eq_here = (sl + 1 < (uint32_t)kSlices ? cs.eq[sl + 1] : cnt.y) - cs.eq[sl];
        // eq_mode 0: none of this slice's equals is kept; 1: all are; 2: ranks must be counted
        const int eq_mode = (all || eq_here == 0 || eq_before >= keep_eq) ? 0 : (eq_before + eq_here <= keep_eq ? 1 : 2);
        if (!all && gt_here == 0 && eq_mode == 0) continue; // nothing kept in this slice
        uint32_t eq_seen = eq_before;
        uint32_t pos = gt_before + min(eq_before, keep_eq); // position of the slice's first kept entry in the layer
        const uint64_t gm = cs.mask[sl];
        const uint32_t n_groups = __popcll(gm);
        if (!all && n_groups <= (uint32_t)kSparseGroups) {
            // sparse slice: read only the 32-element groups the counting sweep marked; a quarter warp per group,
            // four groups per pass, in ascending order, so that lane order is index order
            uint8_t* sp = s_pos[wid];
            const uint32_t lo32 = (uint32_t)gm, hi32 = (uint32_t)(gm >> 32), lt = (1u << lane) - 1u;
            __syncwarp();
            if ((lo32 >> lane) & 1u) sp[__popc(lo32 & lt)] = (uint8_t)lane;
            if ((hi32 >> lane) & 1u) sp[__popc(lo32) + __popc(hi32 & lt)] = (uint8_t)(32u + lane);
            __syncwarp();
            for (uint32_t it = 0; it < n_groups; it += 4) {
                const uint32_t r = it + (lane >> 3);
                uint32_t keepm = 0, eqm = 0, e0 = 0;
                auto classify = [&](float v, int i) {
                    const uint32_t key = key_of(v);
                    if (key > tau || (eq_mode == 1 && key == tau)) keepm |= 1u << i;
                    if (eq_mode == 2 && key == tau) eqm |= 1u << i;
                };
                float vq[4] = {0.f, 0.f, 0.f, 0.f}, sq[4] = {0.f, 0.f, 0.f, 0.f}; // d and the state of this lane's quad
                if (r < n_groups) {
                    e0 = x0 + (uint32_t)sp[r] * 32u + (lane & 7u) * 4u;
                    if (e0 >= cv.first && e0 + 4 <= cv.len) {
                        // the state is requested together with d: a kept entry's update then waits for one
                        // memory round trip, not two
                        float gq[4];
                        if (st_vec) {
                            const float4 a = __ldg(reinterpret_cast<const float4*>(gr + e0));
                            const float4 b = *reinterpret_cast<const float4*>(st + e0);
                            gq[0] = a.x; gq[1] = a.y; gq[2] = a.z; gq[3] = a.w;
                            sq[0] = b.x; sq[1] = b.y; sq[2] = b.z; sq[3] = b.w;
                        } else {
#pragma unroll
                            for (int i = 0; i < 4; ++i) { gq[i] = __ldg(gr + e0 + i); sq[i] = st[e0 + i]; }
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i) { vq[i] = __fsub_rn(gq[i], sq[i]); classify(vq[i], i); }
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (e0 + i >= cv.first && e0 + i < cv.len) {
                                sq[i] = st[e0 + i];
                                vq[i] = __fsub_rn(__ldg(gr + e0 + i), sq[i]);
                                classify(vq[i], i);
                            }
                    }
                }
                if (eq_mode == 2) { // uniform over the warp
                    uint32_t incl = __popc(eqm);
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= (uint32_t)o) incl += y;
                    }
                    uint32_t eq_rank = eq_seen + incl - __popc(eqm);
                    for (uint32_t m = eqm; m; m &= m - 1) {
                        if (eq_rank < keep_eq) keepm |= m & (0u - m);
                        ++eq_rank;
                    }
                    eq_seen += __shfl_sync(0xffffffffu, incl, 31);
                }
                uint32_t incl = __popc(keepm);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= (uint32_t)o) incl += y;
                }
                uint32_t o = pos + incl - __popc(keepm);
                pos += __shfl_sync(0xffffffffu, incl, 31);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (((keepm >> i) & 1u) && KIMAD_CHECK(jb.base + o < cap, 3)) {
                        oi[o] = idx0 + e0 + i;
                        float sent;
                        if (BF16) {
                            const __nv_bfloat16 h = __float2bfloat16_rn(vq[i]);
                            ov16[o] = h;
                            sent = __bfloat162float(h);
                        } else {
                            ov32[o] = vq[i];
                            sent = vq[i];
                        }
                        st[e0 + i] = __fadd_rn(sq[i], sent);
                        ++o;
                    }
            }
            continue;
        }
        constexpr int E = 16;
        for (uint32_t rb = x0; rb < min(cv.len, x0 + kSliceElems); rb += E * 32) {
            const uint32_t t0 = rb + E * lane;
            uint32_t keepm = 0, eqm = 0;
            const bool full = rb >= cv.first && rb + E * 32 <= cv.len; // round fully inside the chunk
            float v[E];
            float sv[DENSE ? E : 1]; // the dense instantiation keeps the estimator's values for its update
            if (full) {
                if (st_vec) {
#pragma unroll
                    for (int u = 0; u < E / 4; ++u) {
                        const float4 a = __ldg(reinterpret_cast<const float4*>(gr + t0) + u);
                        const float4 b = *(reinterpret_cast<const float4*>(st + t0) + u);
                        v[4 * u] = __fsub_rn(a.x, b.x); v[4 * u + 1] = __fsub_rn(a.y, b.y);
                        v[4 * u + 2] = __fsub_rn(a.z, b.z); v[4 * u + 3] = __fsub_rn(a.w, b.w);
                        if (DENSE) { sv[4 * u] = b.x; sv[4 * u + 1] = b.y; sv[4 * u + 2] = b.z; sv[4 * u + 3] = b.w; }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < E; ++i) {
                        const float b = st[t0 + i];
                        v[i] = __fsub_rn(__ldg(gr + t0 + i), b);
                        if (DENSE) sv[i] = b;
                    }
                }
#pragma unroll
                for (int i = 0; i < E; ++i) {
                    const uint32_t key = key_of(v[i]);
                    if (all || key > tau || (eq_mode == 1 && key == tau)) keepm |= 1u << i;
                    if (eq_mode == 2 && key == tau) eqm |= 1u << i;
                }
            } else {
#pragma unroll
                for (int i = 0; i < E; ++i) {
                    const uint32_t e = t0 + i;
                    const bool in = e >= cv.first && e < cv.len;
                    const uint32_t key = key_of(in ? __fsub_rn(__ldg(gr + e), st[e]) : 0.f);
                    if (in && (all || key > tau || (eq_mode == 1 && key == tau))) keepm |= 1u << i;
                    if (in && eq_mode == 2 && key == tau) eqm |= 1u << i;
                }
            }
            if (eq_mode == 2) { // uniform over the warp
                uint32_t incl = __popc(eqm);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= (uint32_t)o) incl += y;
                }
                uint32_t eq_rank = eq_seen + incl - __popc(eqm);
                for (uint32_t m = eqm; m; m &= m - 1) {
                    if (eq_rank < keep_eq) keepm |= m & (0u - m);
                    ++eq_rank;
                }
                eq_seen += __shfl_sync(0xffffffffu, incl, 31);
            }
            uint32_t incl = __popc(keepm);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= (uint32_t)o) incl += y;
            }
            uint32_t o = pos + incl - __popc(keepm);
            const uint32_t round_total = __shfl_sync(0xffffffffu, incl, 31);
            pos += round_total;
            if (DENSE && full && round_total >= 48u) {
                // many kept entries: values come from the registers and the state is read before it is needed,
                // so that no store waits for a load of its own
                // the round's entries are laid out in shared memory first, so that the packed buffers are written
                // with consecutive lanes on consecutive entries
                uint32_t* sg_idx = s_stage[wid];
                uint32_t* sg_val = sg_idx + E * 32;
                uint32_t ol = incl - __popc(keepm); // position inside the round
#pragma unroll
                for (int i = 0; i < E; ++i)
                    if ((keepm >> i) & 1u) {
                        sg_idx[ol] = idx0 + t0 + i;
                        float sent;
                        if (BF16) {
                            const __nv_bfloat16 h = __float2bfloat16_rn(v[i]);
                            sg_val[ol] = (uint32_t)__bfloat16_as_ushort(h);
                            sent = __bfloat162float(h);
                        } else {
                            sg_val[ol] = __float_as_uint(v[i]);
                            sent = v[i];
                        }
                        sv[i] = __fadd_rn(sv[i], sent);
                        ++ol;
                    }
                __syncwarp();
                const uint32_t round_pos = pos - round_total;
                for (uint32_t q = lane; q < round_total; q += 32) {
                    if (!KIMAD_CHECK(jb.base + round_pos + q < cap, 3)) continue;
                    oi[round_pos + q] = sg_idx[q];
                    if (BF16) ov16[round_pos + q] = __ushort_as_bfloat16((unsigned short)sg_val[q]);
                    else ov32[round_pos + q] = __uint_as_float(sg_val[q]);
                }
                __syncwarp();
                if (st_vec) {
                    if (keepm) {
#pragma unroll
                        for (int u = 0; u < E / 4; ++u)
                            if ((keepm >> (4 * u)) & 15u)
                                *(reinterpret_cast<float4*>(st + t0) + u) = make_float4(sv[4 * u], sv[4 * u + 1], sv[4 * u + 2], sv[4 * u + 3]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < E; ++i)
                        if ((keepm >> i) & 1u) st[t0 + i] = sv[i];
                }
                continue;
            }
            while (keepm) {
                const int i = __ffs(keepm) - 1;
                keepm &= keepm - 1;
                const uint32_t e = t0 + i;
                if (!KIMAD_CHECK(jb.base + o < cap && e >= cv.first && e < cv.len, 3)) { ++o; continue; }
                const float was = st[e];
                const float val = __fsub_rn(__ldg(gr + e), was); // both loaded a moment ago: L1 hits
                oi[o] = idx0 + e;
                float sent;
                if (BF16) {
                    const __nv_bfloat16 h = __float2bfloat16_rn(val);
                    ov16[o] = h;
                    sent = __bfloat162float(h);
                } else {
                    ov32[o] = val;
                    sent = val;
                }
                st[e] = __fadd_rn(was, sent);
                ++o;
            }
        }
    }
}

} // namespace kimad
