// Plain structs and integer helpers shared by the host planner and the kernels of the CUDA library.
#pragma once
#include <stdint.h>

#include "kimad.h"

#if defined(__CUDACC__)
#define KIMAD_HD __host__ __device__ __forceinline__
#else
#define KIMAD_HD inline
#endif

// Checked build (-DKIMAD_CHECKED): indices into the workspace and the output buffers are tested before use; a failed
// test sets its bit in a status word that the host reads (kimad_debug_check) and the access is skipped -- nothing
// traps.  Bits: 0 sweep: bin outside the layer's histogram; 1 counting sweep: bin outside the in-interval histogram;
// 2 a work list (exact path, second select round, recount) appended beyond its capacity; 3 write sweep: packed
// position beyond the capacity; 4 write sweep: element index outside its layer; 5 DP: cell or back-pointer outside
// its row; 6 curve: bin outside the layer's histogram; 7 curve: the pieces of a refined bin do not add up to the bin.
// In the ordinary build KIMAD_CHECK(cond, bit) is `true`.
#if defined(KIMAD_CHECKED) && defined(__CUDACC__)
__device__ unsigned int g_kimad_check_word;
#define KIMAD_CHECK(cond, bit) ((cond) ? true : (atomicOr(&g_kimad_check_word, 1u << (bit)), false))
#else
#define KIMAD_CHECK(cond, bit) (true)
#endif

namespace kimad {

// A chunk is the part of one layer that falls inside one aligned window of kChunkElems elements of
// the flat per-worker vector.  One CTA streams one chunk.
constexpr uint64_t kChunkElems = 32768;
constexpr int kDpWorkersPerLaunch = 32;

struct Chunk {
    uint32_t layer;
    uint32_t _pad;
    uint64_t begin; // flat element index inside the worker's vector
    uint64_t end;
};

struct LayerDesc {
    uint64_t begin;
    uint64_t n;
    uint32_t first_chunk;
    uint32_t n_chunks;
};

// Radix-select state of one (worker, layer, candidate) between digit passes.
struct Cand {
    double err_low;  // sum of squares of everything known to lie below the current bin
    uint32_t rank;   // 1-based rank of the wanted key inside the current bin, counted from the top
    uint32_t gt;     // keys known to be larger than everything in the current bin
    uint32_t slot;   // which histogram slot of this (worker, layer) refines the current bin
    uint32_t prefix; // the bin: top 11 / 21 / 31 bits of the key after digit 1 / 2 / 3
};

struct SlotTab {
    uint32_t n;
    uint32_t prefix[KIMAD_MAX_RATIOS];
};

// What the select kernels need to know about one (worker, layer) after the DP.  The threshold lies in
// the key interval [tau, tau + 2^shift) and is the keep_eq-th largest key inside it; k_sel_resolve
// narrows that to the exact threshold (shift = 0) and to the number of ties kept.
struct Sel {
    uint32_t tau;     // lower key of the interval, then the exact threshold key
    uint32_t keep_eq; // rank inside the interval, then: entries equal to tau that are kept (lowest indices first)
    uint32_t k;       // 0: nothing to pack for this layer (the worker failed)
    uint32_t shift;   // log2 of the interval width (<= 10)
    uint32_t tau_low; // exact threshold minus the interval's lower key
    uint32_t code;    // the code (byte plane of the sweep) of the keys of the interval: entries with a larger code lie
                      // above the interval, entries with a smaller one below
    uint64_t base;    // first output position of the layer in the worker's packed buffers
};

// The candidate table k_{l,j}: one table for all workers (wstride = 0: the ratio grid applied to the layer sizes), or
// one per worker (the ratio fitted to each worker's budget).
struct KTab {
    const uint64_t* p;
    uint64_t wstride;
    KIMAD_HD uint64_t at(uint32_t w, size_t i) const { return p[(size_t)w * wstride + i]; }
};

// Size in bytes of candidate k of a layer of n elements and the entries it keeps (Eq. 3's b_ij; the paper fixes no
// encoding).  cost model 0: k (4 + vb).  cost model 1: once the sparse size reaches the dense size vb n the layer is
// sent densely: every value, no indices; it then keeps all n entries and loses nothing.
KIMAD_HD uint64_t candidate_bytes(uint64_t n, uint64_t k, uint32_t bpe, uint32_t cost_model, bool* dense) {
    const uint64_t vb = bpe - 4;
    const bool d = cost_model == 1 && k * bpe >= vb * n;
    if (dense) *dense = d;
    return d ? vb * n : k * bpe;
}

// Budget cells a candidate of `bytes` occupies when c bytes are split into D cells (rounded up, so
// the byte constraint of Eq. 3 can never be exceeded).  c > 0.
KIMAD_HD uint64_t budget_cells(uint64_t bytes, uint32_t D, uint64_t c) { return (bytes * (uint64_t)D + c - 1) / c; }

} // namespace kimad
