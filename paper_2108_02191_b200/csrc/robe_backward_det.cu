// Deterministic backward (Section 3.1 backward equation, evaluated in a fixed order).
//
// Blocks are numbered q = p*C + c in input order (p = position in indices, c = chunk).
//   1. key kernel      key[q] = h(e, x_p, c); val[q] = where the block's gradient elements
//                      start in grad_out (sign off) or q itself (sign on); or both left by the
//                      forward of the same step
//   2. radix sort      stable LSD sort of (key, val) by key - our own passes: digit count per
//                      CTA range, per-digit exclusive scan, ranked scatter through shared
//                      memory (so that every digit's run leaves the CTA as one coalesced piece)
//   3. apply kernel    one thread per touched array slot j sums, left to right in fp32 from +0,
//                      the terms of the sorted blocks whose key lies in [j-Z+1, j], then performs
//                      ONE add (dense gradient) or ONE fma (SGD) on slot j.  The thread that owns
//                      slot j is the one at the first sorted block of that key window, so it only
//                      ever walks forward through the sorted list.  Slots [0, Z-1), which also
//                      receive the wrapped tails of blocks near the end of the array, are handled
//                      by a small second kernel (those terms come last: their keys are the largest).
//                      Walks over hundreds of blocks (an id repeated many times in the batch)
//                      are finished by a third kernel that keeps a whole step of terms in flight.
// No atomics on floating-point data and no waits between CTAs: the result is bit-reproducible.
#include "robe_internal.h"

namespace robe {

namespace {

constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kSortItems = 16;                          // keys per thread per tile
constexpr int kSortTile = kSortThreads * kSortItems;    // 4096
constexpr int kRadix = 256;
constexpr int kSortMaxGrid = 148 * 4;

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

struct SortPlan {
    uint64_t nb;        // number of (key,val) pairs
    uint32_t grid;      // CTAs of the count / scatter kernels
    uint64_t tiles;     // total tiles
};

SortPlan make_plan(uint64_t nb) {
    SortPlan sp;
    sp.nb = nb;
    sp.tiles = (nb + kSortTile - 1) / kSortTile;
    sp.grid = (uint32_t)(sp.tiles < (uint64_t)kSortMaxGrid ? sp.tiles : (uint64_t)kSortMaxGrid);
    if (sp.grid == 0) sp.grid = 1;
    return sp;
}

// tiles [first, first+count) of CTA b: contiguous, near-equal split
__device__ __forceinline__ void cta_tiles(uint64_t tiles, uint32_t grid, uint32_t b,
                                          uint64_t& first, uint64_t& count) {
    uint64_t per = tiles / grid, rem = tiles % grid;
    count = per + (b < rem ? 1 : 0);
    first = per * b + (b < rem ? b : rem);
}

struct KeyArgs {
    MapParams mp;
    IdList indices;
    const int64_t* offsets;
    int64_t nbags;
    int64_t nnz;
    const int32_t* status;
};

// bag_of[p] = bag number of id position p (multi-hot only)
__global__ void __launch_bounds__(256) det_bag_of_kernel(KeyArgs a, uint32_t* bag_of) {
    const int64_t k = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    if (k >= a.nbags) return;
    int64_t lo = __ldg(a.offsets + k), hi = __ldg(a.offsets + k + 1);
    lo = lo < 0 ? 0 : (lo > a.nnz ? a.nnz : lo);
    hi = hi < lo ? lo : (hi > a.nnz ? a.nnz : hi);
    for (int64_t p = lo + lane; p < hi; p += 32) bag_of[p] = (uint32_t)k;
}

// key[q] = h(e, x_p, c) for q = p*C + c.  val[q] = q when the sign hash is on (the apply kernel
// then needs the id again), else the position bag*d + c*Z of the block's first gradient element.
// One thread per id: the part of the hash that all chunks of the id share is evaluated once.
template <bool SIGN>
__global__ void __launch_bounds__(256)
det_keys_kernel(KeyArgs a, const uint32_t* bag_of, uint32_t* keys, uint32_t* vals) {
    const uint64_t p = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (p >= (uint64_t)a.nnz) return;
    const MapParams& mp = a.mp;
    const uint64_t bag = bag_of ? (uint64_t)bag_of[p] : p;
    const uint32_t e = table_of_bag(bag, mp);
    const uint64_t x = (uint64_t)a.indices.load((int64_t)p);
    const uint64_t q0 = p * mp.C;
    if (mp.R > 1) {  // rows clubbed into one block: a single key
        keys[q0] = id_block_start(mp, e, x, 0);
        vals[q0] = SIGN ? (uint32_t)q0 : (uint32_t)(bag * mp.d);
        return;
    }
    const uint64_t base = hash_base(mp.h, e, x);
    for (uint32_t c = 0; c < mp.C; ++c) {
        if (!ROBE_CHK(q0 + c < (uint64_t)a.nnz * mp.C, ROBE_DBG_SORT_POS)) break;
        keys[q0 + c] = block_start(mp, base, c);
        vals[q0 + c] = SIGN ? (uint32_t)(q0 + c) : (uint32_t)(bag * mp.d + c * mp.Z);
    }
}

// The same, one thread per block: for many blocks per id (small Z) the writes of one thread per
// id would be far apart, and re-evaluating the shared part of the hash per block costs less.
template <bool SIGN>
__global__ void __launch_bounds__(256)
det_keys_by_block_kernel(KeyArgs a, const uint32_t* bag_of, uint32_t* keys, uint32_t* vals,
                         uint64_t nb) {
    const uint64_t q = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (q >= nb) return;
    const MapParams& mp = a.mp;
    const uint32_t p = (uint32_t)q / mp.C;
    const uint32_t c = (uint32_t)q - p * mp.C;
    const uint64_t bag = bag_of ? (uint64_t)bag_of[p] : (uint64_t)p;
    const uint32_t e = table_of_bag(bag, mp);
    const uint64_t x = (uint64_t)a.indices.load(p);
    keys[q] = id_block_start(mp, e, x, c);
    vals[q] = SIGN ? (uint32_t)q : (uint32_t)(bag * mp.d + c * mp.Z);
}


// ---- radix sort pass, kernel 1: digit histogram of each CTA's contiguous key range
__global__ void __launch_bounds__(kSortThreads)
sort_count_kernel(const uint32_t* keys, uint32_t* counts, uint64_t nb, uint64_t tiles,
                  uint32_t shift, uint32_t mask) {
    __shared__ uint32_t hist[kSortWarps][kRadix];
    for (int k = 0; k < kSortWarps; ++k) hist[k][threadIdx.x] = 0;
    __syncthreads();
    uint64_t first, count;
    cta_tiles(tiles, gridDim.x, blockIdx.x, first, count);
    const uint64_t begin = first * kSortTile;
    uint64_t end = (first + count) * kSortTile;
    if (end > nb) end = nb;
    uint32_t* mine = hist[threadIdx.x >> 5];
    for (uint64_t i = begin + threadIdx.x; i < end; i += kSortThreads)
        atomicAdd(&mine[(keys[i] >> shift) & mask], 1u);
    __syncthreads();
    uint32_t total = 0;
    for (int k = 0; k < kSortWarps; ++k) total += hist[k][threadIdx.x];
    counts[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x] = total;
}

// Exclusive scan of the 256 values held one per thread (value v of thread t): returns the sum
// of the values of threads below t.  All 256 threads of the CTA call it; contains __syncthreads.
__device__ __forceinline__ uint32_t cta_exclusive_scan_256(uint32_t v, uint32_t* warp_sums) {
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= (uint32_t)o) inc += n;
    }
    if (lane == 31) warp_sums[w] = inc;
    __syncthreads();
    uint32_t before = 0;
    for (uint32_t k = 0; k < w; ++k) before += warp_sums[k];
    __syncthreads();  // warp_sums may be reused by the caller's next scan
    return before + inc - v;
}

// ---- kernel 2: one CTA per digit: exclusive scan of that digit's per-CTA counts, in place, and
// the digit's total into totals[digit]
__global__ void __launch_bounds__(kSortThreads)
sort_scan_kernel(uint32_t* counts, uint32_t* totals, uint32_t grid) {
    __shared__ uint32_t warp_sums[kSortWarps];
    uint32_t* row = counts + (uint64_t)blockIdx.x * grid;
    uint32_t carry = 0;
    for (uint32_t b0 = 0; b0 < grid; b0 += kSortThreads) {
        const uint32_t b = b0 + threadIdx.x;
        const uint32_t v = b < grid ? row[b] : 0u;
        const uint32_t ex = cta_exclusive_scan_256(v, warp_sums);
        if (b < grid) row[b] = carry + ex;
        // total of this chunk = exclusive prefix of the last thread + its value
        __shared__ uint32_t chunk_total;
        if (threadIdx.x == kSortThreads - 1) chunk_total = ex + v;
        __syncthreads();
        carry += chunk_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) totals[blockIdx.x] = carry;
}

// ---- kernel 3: ranked scatter (STABLE: keeps the input order inside a digit - the LSD sort needs
// that; the binned backward does not and takes ranks from shared-memory counters).  Per tile of 4096 pairs: every warp ranks its 512 pairs
// by digit (16 rounds of ballots, earlier rounds and lower lanes first), the ranks are
// extended over the warps, the pairs are laid out in shared memory in (digit, original order),
// and then written out so that each digit's pairs go to consecutive addresses.
template <bool STABLE>
__global__ void __launch_bounds__(kSortThreads, 4)
sort_scatter_kernel(const uint32_t* __restrict__ kin, const uint32_t* __restrict__ vin,
                    uint32_t* __restrict__ kout, uint32_t* __restrict__ vout,
                    const uint32_t* __restrict__ cta_offsets, const uint32_t* __restrict__ totals,
                    uint64_t nb, uint64_t tiles, uint32_t shift, uint32_t mask) {
    __shared__ uint32_t skey[kSortTile];
    __shared__ uint32_t sval[kSortTile];
    __shared__ uint32_t wcnt[kSortWarps][kRadix];
    __shared__ uint32_t base[kRadix];    // where the next pair of this digit goes, minus dstart
    __shared__ uint32_t dstart[kRadix];  // start of the digit's run inside the tile
    __shared__ uint32_t warp_sums[kSortWarps];
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    {
        // start of this digit in the output = pairs of lower digits + this digit's pairs in
        // lower CTAs
        const uint32_t below = cta_exclusive_scan_256(totals[threadIdx.x], warp_sums);
        base[threadIdx.x] = below + cta_offsets[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x];
    }
    uint64_t first, count;
    cta_tiles(tiles, gridDim.x, blockIdx.x, first, count);
    for (uint64_t t = first; t < first + count; ++t) {
        for (int k = 0; k < kSortWarps; ++k) wcnt[k][threadIdx.x] = 0;
        __syncthreads();
        const uint64_t tbegin = t * kSortTile;
        const uint64_t wbegin = tbegin + (uint64_t)w * (32 * kSortItems);
        uint32_t key[kSortItems], rank[kSortItems];
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
            const uint64_t idx = wbegin + r * 32 + lane;
            key[r] = idx < nb ? kin[idx] : 0u;
        }
        if (!STABLE) {
            // any order inside a digit will do: the rank is what a shared-memory counter hands out
#pragma unroll
            for (int r = 0; r < kSortItems; ++r) {
                rank[r] = 0;
                if (wbegin + r * 32 + lane < nb) rank[r] = atomicAdd(&wcnt[w][(key[r] >> shift) & mask], 1u);
            }
        }
#pragma unroll
        for (int r = 0; STABLE && r < kSortItems; ++r) {
            const bool valid = wbegin + r * 32 + lane < nb;
            const uint32_t dg = valid ? ((key[r] >> shift) & mask) : 0u;
            // lanes holding the same digit: one ballot per digit bit (a fixed cost, where
            // __match_any_sync takes time in proportion to the number of distinct digits)
            uint32_t peers = __ballot_sync(0xFFFFFFFFu, valid);
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const bool bit = (dg >> b) & 1u;
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, bit);
                peers &= bit ? bal : ~bal;
            }
            uint32_t before = 0;
            if (valid) before = wcnt[w][dg];
            __syncwarp();
            if (valid && (peers & lt) == 0) wcnt[w][dg] = before + __popc(peers);
            __syncwarp();
            rank[r] = before + __popc(peers & lt);
        }
        __syncthreads();
        // per digit: exclusive prefix over the warps of this tile, and the tile's total
        uint32_t tile_total = 0;
        for (int k = 0; k < kSortWarps; ++k) {
            const uint32_t c = wcnt[k][threadIdx.x];
            wcnt[k][threadIdx.x] = tile_total;
            tile_total += c;
        }
        const uint32_t ds = cta_exclusive_scan_256(tile_total, warp_sums);  // syncs inside
        dstart[threadIdx.x] = ds;
        // from here base[] holds (output position of the digit's next pair) - (its position in
        // the tile), so that a pair at tile position lp goes to base[digit] + lp
        base[threadIdx.x] -= ds;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
            const uint64_t idx = wbegin + r * 32 + lane;
            if (idx < nb) {
                const uint32_t dg = (key[r] >> shift) & mask;
                const uint32_t lp = dstart[dg] + wcnt[w][dg] + rank[r];
                if (!ROBE_CHK(lp < (uint32_t)kSortTile, ROBE_DBG_SHARED)) continue;
                skey[lp] = key[r];
                sval[lp] = vin[idx];  // payloads are only passed through: read them this late
            }
        }
        __syncthreads();
        const uint32_t in_tile = (uint32_t)(nb - tbegin < (uint64_t)kSortTile ? nb - tbegin
                                                                               : (uint64_t)kSortTile);
        for (uint32_t lp = threadIdx.x; lp < in_tile; lp += kSortThreads) {
            const uint32_t k = skey[lp];
            const uint32_t dst = base[(k >> shift) & mask] + lp;
            if (!ROBE_CHK((uint64_t)dst < nb, ROBE_DBG_SORT_POS)) continue;
            kout[dst] = k;
            vout[dst] = sval[lp];
        }
        __syncthreads();
        base[threadIdx.x] += ds + tile_total;  // undo the shift, advance past this tile's pairs
        // (the next tile's first barrier orders this update before its readers)
    }
}

// A round of the apply kernel whose walks got long, handed over to the long-walk kernel: where
// the tile starts, how far the lanes have come, and per lane its slot, its sum so far and its
// position in the tile.
struct LongWalk {
    uint64_t i0;
    uint32_t fbase;         // lane l goes on at sorted position i0 + fbase + e(l)
    uint32_t pad;
    uint32_t j[32];
    float acc[32];
    uint32_t state[32];     // e | going << 8 | touched << 9
};

struct ApplyArgs {
    MapParams mp;
    const float* grad_out;
    IdList indices;  // only read when the sign hash is on
    float* target;
    float lr;
    uint64_t nb;
    const int32_t* status;
    AdamState adam;          // update mode 2 only
    uint32_t* long_count;    // number of handed-over rounds (may run past long_cap)
    LongWalk* long_walks;
    uint32_t long_cap;
    // window apply (densely touched arrays): per array window of 2^win_log2 slots, did the window kernel
    // leave it to the position-tile kernel?  nullptr = there is no window kernel in this call
    const uint8_t* win_left;
    const uint32_t* any_left;  // number of windows left over (0: the tile kernel has nothing to do)
    uint32_t win_log2;         // log2 of the window length
    uint64_t grad_elems;       // elements of grad_out (read by the debug build's index checks only)
    int l2_keep;               // binned adds: the reductions carry the L2 "keep" policy
};

// The term that the sorted block with payload v contributes to the slot at in-block offset o
// (o < Z), or nothing if o is past the end of a short last block.
template <bool SIGN, bool SHORT>
__device__ __forceinline__ bool block_term(const ApplyArgs& a, const uint32_t* bag_of, uint32_t v,
                                           uint32_t o, float& term) {
    const MapParams& mp = a.mp;
    if (!SIGN) {
        // v = bag*d + c*Z: the block's first element in grad_out
        if (SHORT) {
            const uint32_t cz = v - (v / mp.d) * mp.d;
            if (cz + o >= mp.d) return false;
        }
        if (!ROBE_CHK((uint64_t)v + o < a.grad_elems, ROBE_DBG_GRAD_POS)) return false;
        term = __ldg(a.grad_out + (uint64_t)v + o);
        return true;
    }
    const uint32_t p = v / mp.C;  // v = q
    const uint32_t c = v - p * mp.C;
    const uint32_t i = c * mp.Z + o;
    if (i >= mp.d) return false;
    const uint64_t bag = bag_of ? (uint64_t)__ldg(bag_of + p) : (uint64_t)p;
    if (!ROBE_CHK(bag * mp.d + i < a.grad_elems, ROBE_DBG_GRAD_POS)) return false;
    const uint32_t e = table_of_bag(bag, mp);
    const uint64_t x = (uint64_t)a.indices.load(p);
    term = sign_of(mp, hash_base(mp.g, e, x), i) * __ldg(a.grad_out + bag * mp.d + i);
    return true;
}

// What a served slot does with its sum delta (MODE): 0 - add it to a dense gradient; 1 - the
// SGD step M[j] = fma(-lr, delta, M[j]); 3 - the Adagrad step; 2 - the Adam step (Kingma & Ba, Algorithm 1; the paper
// trains five of its six models with Adam, Section 5) on the slot and its two moment slots, every
// operation a separate correctly rounded fp32 one.  `old` is target[j].
template <int MODE>
__device__ __forceinline__ void commit_slot(const ApplyArgs& a, uint32_t j, float delta, float old) {
    if (!ROBE_CHK(j < a.mp.m, ROBE_DBG_ARRAY_SLOT)) return;
    if (MODE == 0) {
        a.target[j] = __fadd_rn(old, delta);
    } else if (MODE == 1) {
        a.target[j] = __fmaf_rn(-a.lr, delta, old);
    } else if (MODE == 3) {
        // Adagrad (Duchi, Hazan, Singer): one accumulator of squared gradients per slot
        const AdamState& ad = a.adam;  // m2 = the accumulators, eps
        const float s = __fadd_rn(ad.m2[j], __fmul_rn(delta, delta));
        ad.m2[j] = s;
        const float den = __fadd_rn(__fsqrt_rn(s), ad.eps);
        a.target[j] = __fsub_rn(old, __fmul_rn(a.lr, __fdiv_rn(delta, den)));
    } else {
        const AdamState& ad = a.adam;
        const float m = __fadd_rn(__fmul_rn(ad.beta1, ad.m1[j]), __fmul_rn(__fsub_rn(1.0f, ad.beta1), delta));
        const float v = __fadd_rn(__fmul_rn(ad.beta2, ad.m2[j]),
                                  __fmul_rn(__fsub_rn(1.0f, ad.beta2), __fmul_rn(delta, delta)));
        ad.m1[j] = m;
        ad.m2[j] = v;
        const float den = __fadd_rn(__fsqrt_rn(__fdiv_rn(v, ad.bias2)), ad.eps);
        a.target[j] = __fsub_rn(old, __fmul_rn(a.lr, __fdiv_rn(__fdiv_rn(m, ad.bias1), den)));
    }
}

// Slots j in [Z-1, m).  The sorted blocks that reach slot j are those with key in [j-Z+1, j];
// the slot is served from the FIRST of them: position i serves slot K[i]+u iff i starts a run of
// equal keys and the previous key is below K[i]+u-Z+1, i.e. u >= Z - min(Z, K[i]-K[i-1]).  The
// server then only walks forward through the sorted list, adding terms while the key stays <= j.
//
// One warp takes 32 consecutive sorted positions (a tile).  Keys and payloads live in a
// warp-private ring of 128 positions in shared memory, filled by coalesced loads.  The
// (position, offset) pairs of the tile that serve a slot are numbered through and dealt out one
// per lane, 32 per round.  In a round all lanes step through the ring together, each from its own
// position, UN positions per step (4 in the first step, then 8): ring reads, then the gradient
// loads, then the adds in sorted order; the next 32 positions are fetched one step ahead of
// their first use.  A walk that is still going after 64 positions (an id that occurs many
// times in the batch) is handed, with its sums so far, to the long-walk kernel below, whose
// division of labour adds such a chain several times faster.  Only if the list of handed-over
// rounds is full does it go on here, 16 positions per step, with the gradient rows of the
// positions after those asked into L2 ahead of time.
constexpr uint32_t kRing = 128;
// window apply: the array is cut into windows of 2^8 .. 2^11 slots, one CTA each
constexpr uint32_t kWinLog2Min = 9, kWinLog2Max = 11;
constexpr uint32_t kWinThreads = 512;     // threads of the window kernel (<= the shortest window)
constexpr uint32_t kWinMaxZ = 128;        // longest block the window kernel takes
constexpr uint32_t kWinEnt = 512;         // sorted blocks per chunk, at most
constexpr uint32_t kWinStage = 6144;      // gradient elements per chunk, at most (>= kWinMaxZ)
constexpr uint32_t kNoKey = 0xFFFFFFFFu;  // above every slot number (m + d <= 2^32)

struct ApplyTile {
    const uint32_t* K;
    const uint32_t* V;
    uint64_t nb;
    uint64_t i0;          // first sorted position of the tile
    uint2* ring;          // warp-private, kRing entries
    uint32_t loaded_end;  // the ring holds tile-relative positions [loaded_end - kRing, loaded_end)
    // (key, payload) of tile-relative position r, or a key above every slot past the end
    __device__ __forceinline__ uint2 fetch(uint32_t r) const {
        const uint64_t idx = i0 + r;
        if (idx >= nb) return make_uint2(kNoKey, 0u);
        return make_uint2(__ldg(K + idx), __ldg(V + idx));
    }
};

struct ApplyWalk {
    float acc;
    bool touched, done, pending;
    uint2 ahead;     // positions [loaded_end, loaded_end + 32), fetched but not yet in the ring
    uint32_t fbase;  // the next step starts at tile-relative position fbase + sub
};

// The positions fetched last enter the ring.  pf != nullptr: their gradient rows are asked
// into L2 (pf = grad_out + the first offset of the lanes' chunk).
__device__ __forceinline__ void walk_commit(ApplyTile& tl, ApplyWalk& wk, uint32_t lane,
                                            const float* pf) {
    __syncwarp();
    tl.ring[(tl.loaded_end + lane) & (kRing - 1)] = wk.ahead;
    if (pf != nullptr && wk.ahead.x != kNoKey)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + wk.ahead.y));
    tl.loaded_end += 32;
    wk.pending = false;
    __syncwarp();
}

// Start of a step of UN positions: the positions fetched one step ago enter the ring, and the
// ones the step after this one will read are fetched.
template <int UN>
__device__ __forceinline__ void walk_advance(ApplyTile& tl, ApplyWalk& wk, uint32_t EPW,
                                             uint32_t lane, const float* pf) {
    if (wk.pending) walk_commit(tl, wk, lane, pf);
    // the next step reads up to position fbase + UN + (EPW-1) + (UN-1)
    if (tl.loaded_end <= wk.fbase + 2 * UN + EPW - 2) {
        wk.ahead = tl.fetch(tl.loaded_end + lane);
        wk.pending = true;
    }
}

// Steps of UN positions until no lane goes on, or (limit != 0) until fbase reaches limit.
// Returns whether every lane is done.
template <bool SIGN, bool SHORT, int UN>
__device__ __forceinline__ bool walk_steps(const ApplyArgs& a, const uint32_t* bag_of, ApplyTile& tl,
                                           ApplyWalk& wk, uint32_t j, uint32_t sub, uint32_t EPW,
                                           uint32_t lane, uint32_t limit) {
    for (;; wk.fbase += UN) {
        if (limit != 0 && wk.fbase >= limit) return false;
        walk_advance<UN>(tl, wk, EPW, lane, nullptr);
        uint2 kv[UN];
#pragma unroll
        for (int t = 0; t < UN; ++t) kv[t] = tl.ring[(wk.fbase + sub + t) & (kRing - 1)];
        float term[UN];
        bool ok[UN];
        bool in_last = false;
#pragma unroll
        for (int t = 0; t < UN; ++t) {
            const bool in = !wk.done && kv[t].x <= j;  // sorted: true on a prefix
            ok[t] = false;
            if (in) ok[t] = block_term<SIGN, SHORT>(a, bag_of, kv[t].y, j - kv[t].x, term[t]);
            if (t == UN - 1) in_last = in;
        }
#pragma unroll
        for (int t = 0; t < UN; ++t)
            if (ok[t]) {
                wk.acc = __fadd_rn(wk.acc, term[t]);
                wk.touched = true;
            }
        wk.done = wk.done || !in_last;
        if (__ballot_sync(0xFFFFFFFFu, !wk.done) == 0) {
            wk.fbase += UN;
            return true;
        }
    }
}

// The same for a long walk of plain blocks (sign off, no short last block): more positions per
// step, each term's place in grad_out computed while its key is compared.
__device__ __forceinline__ bool walk_deep(const ApplyArgs& a, ApplyTile& tl, ApplyWalk& wk, uint32_t j,
                                          uint32_t sub, uint32_t EPW, uint32_t lane,
                                          uint32_t chunk_off, uint32_t limit) {
    constexpr int UN = 16;
    const float* pf = a.grad_out + chunk_off;
    // the ring has to reach the end of the first step before the one-step-ahead fetches take over
    if (wk.pending) walk_commit(tl, wk, lane, pf);
    while (tl.loaded_end < wk.fbase + EPW + UN - 1) {
        wk.ahead = tl.fetch(tl.loaded_end + lane);
        walk_commit(tl, wk, lane, pf);
    }
    for (;; wk.fbase += UN) {
        if (limit != 0 && wk.fbase >= limit) return false;
        walk_advance<UN>(tl, wk, EPW, lane, pf);
        uint32_t at[UN];
        uint32_t n_in = 0;
#pragma unroll
        for (int t = 0; t < UN; ++t) {
            const uint2 e = tl.ring[(wk.fbase + sub + t) & (kRing - 1)];
            n_in += (!wk.done && e.x <= j) ? 1u : 0u;  // sorted: a prefix of the step
            at[t] = e.y + (j - e.x);
        }
        const uint32_t n_max = __reduce_max_sync(0xFFFFFFFFu, n_in);  // warp-uniform
        float term[UN];
#pragma unroll
        for (int t = 0; t < UN; ++t) {
            term[t] = 0.0f;
            if ((uint32_t)t < n_max) {
                if ((uint32_t)t < n_in && ROBE_CHK((uint64_t)at[t] < a.grad_elems, ROBE_DBG_GRAD_POS))
                    term[t] = __ldg(a.grad_out + at[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < UN; ++t) {
            if ((uint32_t)t < n_max) {
                if ((uint32_t)t < n_in) wk.acc = __fadd_rn(wk.acc, term[t]);
            }
        }
        if (n_in != 0) wk.touched = true;
        wk.done = wk.done || n_in < (uint32_t)UN;
        if (n_max < (uint32_t)UN) {  // no lane goes on
            wk.fbase += UN;
            return true;
        }
    }
}

template <bool SIGN, int MODE, bool SHORT>
__global__ void __launch_bounds__(256)
det_apply_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                 const uint32_t* __restrict__ bag_of) {
    constexpr int UN = 8;
    constexpr uint32_t kDeepAfter = 64;       // positions after which a walk takes 16 per step, if it stays here
    constexpr uint32_t kHandOverAfter = 64;   // positions after which it goes to the long-walk kernel (128 and 256
                                              // measured slower on Zipf ids, 32 no faster)
    __shared__ uint2 ring_s[8][kRing];
    if (a.status != nullptr && *a.status != 0) return;
    if (a.any_left != nullptr && *a.any_left == 0) return;  // the window kernel served every slot
    const MapParams& mp = a.mp;
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    ApplyTile tl;
    tl.K = K;
    tl.V = V;
    tl.nb = a.nb;
    tl.i0 = ((uint64_t)blockIdx.x * 8 + w) * 32;
    if (tl.i0 >= a.nb) return;  // whole warp
    tl.ring = ring_s[w];
    const uint2 mine = tl.fetch(lane);
    tl.ring[lane] = mine;
    tl.ring[32 + lane] = tl.fetch(32 + lane);
    tl.loaded_end = 64;

    // first offset served from this lane's position (Z = none)
    uint32_t kprev = __shfl_up_sync(0xFFFFFFFFu, mine.x, 1);
    if (lane == 0 && tl.i0 > 0) kprev = __ldg(K + tl.i0 - 1);
    uint32_t own_lo = mp.Z;
    if (tl.i0 + lane < a.nb) {
        if (tl.i0 + lane == 0) own_lo = 0;
        else if (kprev != mine.x) {
            const uint32_t gap = mine.x - kprev;
            own_lo = gap >= mp.Z ? 0u : mp.Z - gap;
        }
    }
    __syncwarp();

    // Served (position, offset) pairs are numbered tile-wide - position after position, offsets
    // ascending - and dealt out 32 per round, one pair per lane, so that no lane idles on a pair
    // that serves nothing.
    const uint32_t cnt = mp.Z - own_lo;
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= (uint32_t)o) incl += n;
    }
    const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);

    for (uint32_t r0 = 0; r0 < total; r0 += 32) {
        const uint32_t idx = r0 + lane;
        // position e of pair idx: the first lane whose inclusive count exceeds idx
        uint32_t e = 0;
#pragma unroll
        for (int step = 16; step >= 1; step >>= 1) {
            const uint32_t v = __shfl_sync(0xFFFFFFFFu, incl, e + step - 1);
            if (v <= idx) e += step;
        }
        if (e > 31) e = 31;  // idx >= total: no pair
        const uint32_t incl_e = __shfl_sync(0xFFFFFFFFu, incl, e);
        const uint32_t lo_e = __shfl_sync(0xFFFFFFFFu, own_lo, e);
        const uint32_t s = __shfl_sync(0xFFFFFFFFu, mine.x, e);
        const uint32_t u = mp.Z - (incl_e - idx);  // lo_e <= u < Z for a real pair
        const uint64_t j64 = (uint64_t)s + u;
        // j64 >= m: wrapped part, j64 < Z-1: low slots - both belong to the other kernel
        bool active = idx < total && u >= lo_e && u < mp.Z && j64 < mp.m && j64 + 1 >= mp.Z;
        if (active && a.win_left != nullptr) active = a.win_left[j64 >> a.win_log2] != 0;
        if (__ballot_sync(0xFFFFFFFFu, active) == 0) continue;
        const uint32_t j = (uint32_t)j64;
        float old = 0.0f;
        if (active && ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) old = a.target[j];

        if (tl.loaded_end > kRing) {  // an earlier long walk moved the ring past the tile's start
            __syncwarp();
            tl.ring[lane] = mine;
            tl.ring[32 + lane] = tl.fetch(32 + lane);
            tl.loaded_end = 64;
            __syncwarp();
        }

        // the lane walks from its own position e: step n reads positions fbase + e + t
        ApplyWalk wk;
        wk.acc = 0.0f;
        wk.touched = false;
        wk.done = !active;
        wk.pending = false;
        wk.ahead = make_uint2(kNoKey, 0u);
        wk.fbase = 0;
        if (!walk_steps<SIGN, SHORT, 4>(a, bag_of, tl, wk, j, e, 32u, lane, 4)) {
            if (!SIGN && !SHORT) {
                if (!walk_steps<SIGN, SHORT, UN>(a, bag_of, tl, wk, j, e, 32u, lane, kDeepAfter) &&
                    !walk_deep(a, tl, wk, j, e, 32u, lane, u & ~31u, kHandOverAfter)) {
                    // long walks: hand the round over if the list has room, else go on here
                    uint32_t rec = a.long_cap;
                    if (a.long_cap != 0) {
                        if (lane == 0) rec = atomicAdd(a.long_count, 1u);
                        rec = __shfl_sync(0xFFFFFFFFu, rec, 0);
                    }
                    if (rec < a.long_cap) {
                        LongWalk* lw = a.long_walks + rec;
                        if (lane == 0) {
                            lw->i0 = tl.i0;
                            lw->fbase = wk.fbase;
                        }
                        lw->j[lane] = j;
                        lw->acc[lane] = wk.acc;
                        lw->state[lane] = e | (wk.done ? 0u : 1u << 8) | (wk.touched ? 1u << 9 : 0u);
                        if (!wk.done) wk.touched = false;  // finished (and stored) by the other kernel
                    } else {
                        walk_deep(a, tl, wk, j, e, 32u, lane, u & ~31u, 0);
                    }
                }
            } else {
                walk_steps<SIGN, SHORT, UN>(a, bag_of, tl, wk, j, e, 32u, lane, 0);
            }
        }
        if (wk.touched) commit_slot<MODE>(a, j, wk.acc, old);
    }
}

// ---- window apply: the slot-major way, for arrays that a call touches densely (plain blocks
// of full length).  The array is cut into windows of W = 2^win_log2 slots.
//
// lo_of[b] = first sorted position whose block reaches slot b*W or a later one (key + Z-1 >= b*W),
// hi_of[b] = first sorted position whose key is >= b*W; both for b = 0 .. number of windows.
constexpr int kBoundsPer = 8;  // sorted positions per thread

__global__ void __launch_bounds__(256)
det_bounds_kernel(const uint32_t* __restrict__ K, uint64_t nb, uint32_t* lo_of, uint32_t* hi_of,
                  uint32_t nwin, uint32_t win_log2, uint32_t Z, const int32_t* status) {
    // after a failed input check K was not written: the loops below rely on sorted keys
    if (status != nullptr && *status != 0) return;
    const uint64_t i0 = ((uint64_t)blockIdx.x * 256 + threadIdx.x) * kBoundsPer;
    if (i0 > nb) return;
    uint64_t k[kBoundsPer + 1];  // k[t] = key before position i0 + t
    k[0] = i0 > 0 ? (uint64_t)__ldg(K + i0 - 1) : 0;
#pragma unroll
    for (int t = 0; t < kBoundsPer; ++t) k[t + 1] = i0 + t < nb ? (uint64_t)__ldg(K + i0 + t) : ~0ull;
#pragma unroll
    for (int t = 0; t < kBoundsPer; ++t) {
        const uint64_t i = i0 + t;
        if (i > nb) break;
        // windows b with b*W in (k[t], k[t+1]] get hi_of[b] = i (and b = 0 at i = 0)
        uint64_t from = i > 0 ? (k[t] >> win_log2) + 1 : 0;
        uint64_t to = i < nb ? (k[t + 1] >> win_log2) : nwin;
        for (uint64_t b = from; b <= to && b <= nwin; ++b)
            if (ROBE_CHK(b <= (uint64_t)nwin, ROBE_DBG_WINDOW)) hi_of[b] = (uint32_t)i;
        from = i > 0 ? ((k[t] + (Z - 1)) >> win_log2) + 1 : 0;
        to = i < nb ? ((k[t + 1] + (Z - 1)) >> win_log2) : nwin;
        for (uint64_t b = from; b <= to && b <= nwin; ++b) lo_of[b] = (uint32_t)i;
    }
}

// win_left[b] = 1 for a window reached by more than n_max sorted blocks (an id that occurs very
// often in the batch falls there): the position-tile kernel and the long-walk kernel serve the
// slots of such windows, the window kernel all others.  *any_left counts them.
__global__ void __launch_bounds__(256)
det_window_classify_kernel(const uint32_t* __restrict__ lo_of, const uint32_t* __restrict__ hi_of,
                           uint32_t nwin, uint32_t n_max, uint8_t* win_left, uint32_t* any_left,
                           const int32_t* status) {
    if (status != nullptr && *status != 0) return;
    const uint32_t b = blockIdx.x * 256 + threadIdx.x;
    const bool left = b < nwin && hi_of[b + 1] - lo_of[b] > n_max;
    if (b < nwin) win_left[b] = left ? 1 : 0;
    const uint32_t votes = __ballot_sync(0xFFFFFFFFu, left);
    if ((threadIdx.x & 31) == 0 && votes != 0) atomicAdd(any_left, (uint32_t)__popc(votes));
}

// One CTA per window of W = 2^LOG2W slots.  The sorted blocks that reach the window are positions
// [lo_of[b], hi_of[b+1]); with their keys taken relative to w0 - (Z-1) ("offsets", 0 .. W+Z-2)
// pre[t] = number of those blocks with offset < t, so that slot w0 + s is reached by the blocks
// lo + [pre[s], pre[s+Z]) - those with key in [j-Z+1, j] - already in sorted order.  pre[] is
// written straight from the sorted keys: the block at relative position e stores e into
// pre[offset of block e-1 + 1 .. its own offset].  The blocks then stream through shared memory in
// chunks, each chunk with its gradient elements (fetched by coalesced loads); every thread owns
// the slots tid, tid+T, ... (T threads) of the window and adds, per chunk, the terms of its slots' ranges
// from first to last, keeping the running sums in registers.  All slots are committed at the end.
template <int MODE, int LOG2W>
__global__ void __launch_bounds__(kWinThreads, 4)
det_apply_window_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                        const uint32_t* __restrict__ lo_of, const uint32_t* __restrict__ hi_of,
                        uint32_t chunk, int vec4) {
    constexpr uint32_t W = 1u << LOG2W;
    constexpr int kSlots = W / kWinThreads;
    __shared__ uint2 ent[kWinEnt];  // .x = (row of the block in stage[]) - key, .y = payload
    __shared__ __align__(16) float stage[kWinStage];
    __shared__ uint32_t pre[W + kWinMaxZ + 8];
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    const uint32_t tid = threadIdx.x;
    const uint32_t b = blockIdx.x;
    const uint32_t lo = lo_of[b], hi = hi_of[b + 1];
    if (a.win_left[b] != 0) return;
    const uint32_t Z = mp.Z;
    const uint64_t w0 = (uint64_t)b << LOG2W;
    const uint32_t n = hi - lo;
    if (n == 0) return;
    if (tid < W / 32) {  // ask the window's target lines into L2 for the commit at the end
        const uint64_t j = w0 + ((uint64_t)tid << 5);
        if (j < mp.m) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.target + j));
    }
    const bool one_chunk = n <= chunk;
    const uint32_t span = W + Z - 1;           // offsets 0 .. span-1; pre[0 .. span]
    const uint32_t bias = (uint32_t)w0 - (Z - 1);  // offset = key - bias (mod 2^32; keys reach >= bias)
    for (uint32_t e = tid; e <= n; e += kWinThreads) {
        const uint32_t from = e > 0 ? __ldg(K + lo + e - 1) - bias + 1 : 0;
        uint32_t to = span;
        if (e < n) {
            const uint32_t k = __ldg(K + lo + e);
            to = k - bias;
            if (one_chunk && ROBE_CHK(e < kWinEnt, ROBE_DBG_SHARED)) ent[e] = make_uint2(e * Z - k, __ldg(V + lo + e));
        }
        for (uint32_t t = from; t <= to; ++t)
            if (ROBE_CHK(t < W + kWinMaxZ + 8, ROBE_DBG_SHARED)) pre[t] = e;
    }
    __syncthreads();
    // a window in the middle of the array: every slot exists and none is a low slot
    const bool inner = b != 0 && w0 + W <= (uint64_t)mp.m;
    const uint32_t j0 = (uint32_t)w0 + tid;  // the thread's first slot
    float acc[kSlots];
#pragma unroll
    for (int q = 0; q < kSlots; ++q) acc[q] = 0.0f;
    for (uint32_t c0 = 0; c0 < n; c0 += chunk) {
        const uint32_t c1 = c0 + chunk < n ? c0 + chunk : n;
        const uint32_t ne = c1 - c0;
        if (!one_chunk) {
            if (c0 != 0) __syncthreads();  // the chunk before has been used
            for (uint32_t e = tid; e < ne; e += kWinThreads)
                if (ROBE_CHK(e < kWinEnt && (uint64_t)lo + c0 + e < a.nb, ROBE_DBG_SHARED))
                    ent[e] = make_uint2(e * Z - __ldg(K + lo + c0 + e), __ldg(V + lo + c0 + e));
            __syncthreads();
        }
        if (vec4) {
            const uint32_t zq = Z >> 2, tot = ne * zq;
            const bool pow2 = mp.log2Z != 0xFFFFFFFFu;
            for (uint32_t t = tid; t < tot; t += kWinThreads) {
                const uint32_t e = pow2 ? t >> (mp.log2Z - 2) : t / zq, o = t - e * zq;
                if (ROBE_CHK(4u * t + 3u < kWinStage && (uint64_t)ent[e].y + 4u * o + 3u < a.grad_elems,
                             ROBE_DBG_GRAD_POS))
                    reinterpret_cast<float4*>(stage)[t] =
                        __ldg(reinterpret_cast<const float4*>(a.grad_out + ent[e].y) + o);
            }
        } else {
            const uint32_t tot = ne * Z;
            for (uint32_t t = tid; t < tot; t += kWinThreads) {
                const uint32_t e = t / Z, o = t - e * Z;
                if (ROBE_CHK(t < kWinStage && (uint64_t)ent[e].y + o < a.grad_elems, ROBE_DBG_GRAD_POS))
                    stage[t] = __ldg(a.grad_out + ((uint64_t)ent[e].y + o));
            }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kSlots; ++q) {
            const uint32_t sl = tid + q * kWinThreads;
            const uint32_t first = pre[sl], last = pre[sl + Z];
            const uint32_t f = (first > c0 ? first : c0) - c0;
            const uint32_t l = (last < c1 ? last : c1) - c0;  // (wraps when last < c0: then f >= l)
            if (first < c1 && last > c0) {
                const uint32_t j = j0 + q * kWinThreads;  // (a slot past the array is dropped at the commit)
                float s = acc[q];
                for (uint32_t e = f; e < l; ++e)
                    if (ROBE_CHK(e < kWinEnt && ent[e].x + j < kWinStage, ROBE_DBG_SHARED))
                        s = __fadd_rn(s, stage[ent[e].x + j]);
                acc[q] = s;
            }
        }
    }
    // commit: the old values of all the thread's slots are asked for together
    float old[kSlots];
    bool has[kSlots];
#pragma unroll
    for (int q = 0; q < kSlots; ++q) {
        const uint32_t sl = tid + q * kWinThreads;
        has[q] = pre[sl + Z] != pre[sl];
        if (!inner) {
            // low slots belong to the low-slot kernel; past the array lie the wrapped tails (the same)
            const uint64_t j64 = w0 + sl;
            has[q] = has[q] && j64 < mp.m && j64 + 1 >= Z;
        }
        old[q] = has[q] ? a.target[j0 + q * kWinThreads] : 0.0f;
    }
#pragma unroll
    for (int q = 0; q < kSlots; ++q)
        if (has[q]) commit_slot<MODE>(a, j0 + q * kWinThreads, acc[q], old[q]);
}

// Long walks (plain blocks only).  One CTA of eight warps per handed-over round, in steps of
// kLongStep = 64 positions.  Lane l of EVERY warp stands for slot l of the round.  The keys come
// from a ring of 512 positions in shared memory.  The chain of dependent adds of one slot is the
// definition's, so everything else is kept off the warp that adds:
//   warp 0      adds the terms of each slot in sorted order, one step per iteration;
//   warps 1..6  copy: each takes every sixth position of the step kLongDepth ahead, and a lane
//               copies the term of its slot with cp.async into its own column of that step's
//               buffer (a whole step in flight without a register per term);
//   warp 7      brings the keys of later steps into the ring (asked for an iteration before they
//               are stored) and finds, by bisection, how many positions of the NEXT step reach
//               each slot - sorted keys make "this position still reaches slot j" a prefix property.
// kLongDepth + 1 buffers; ONE barrier per step.
constexpr int kLongStep = 64;
constexpr int kLongWarps = 8;
constexpr int kLongCopiers = kLongWarps - 2;
constexpr int kLongDepth = 4;                 // steps ahead of the adder whose copies are issued
constexpr int kLongBufs = kLongDepth + 1;
constexpr uint32_t kLongRing = 512;           // >= (kLongDepth + 2) steps + 32 positions of lane spread, power of two
static_assert((kLongDepth + 2) * kLongStep + 32 <= (int)kLongRing, "ring too short");
static_assert(kLongStep == 64, "the scout warp brings in two keys per lane and step");

template <int MODE>
__global__ void __launch_bounds__(32 * kLongWarps)
det_apply_long_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V) {
    __shared__ float terms_s[kLongBufs][kLongStep][32];
    __shared__ uint2 ring[kLongRing];
    __shared__ uint32_t reach_s[2][32];  // by step parity: positions of the step that reach each slot
    __shared__ uint32_t go_on[2];        // by step parity: is there a step to add?
    __shared__ uint32_t rec_s;
    if (a.status != nullptr && *a.status != 0) return;
    const uint32_t tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const uint32_t n_rec = *a.long_count < a.long_cap ? *a.long_count : a.long_cap;
    const uint32_t dst0 = (uint32_t)__cvta_generic_to_shared(&terms_s[0][0][lane]);
    constexpr uint32_t kBufBytes = kLongStep * 32 * sizeof(float);
    constexpr int kPerCopier = (kLongStep + kLongCopiers - 1) / kLongCopiers;
    const bool adder = w == 0, scout = w == kLongWarps - 1;
    // Rounds differ in length by orders of magnitude: a CTA takes the next one when it is free
    // (a.long_count[1] counts the rounds taken) instead of a fixed share.
    for (;;) {
        if (tid == 0) rec_s = atomicAdd(a.long_count + 1, 1u);
        __syncthreads();  // (the barriers inside a round order this store after all reads of the last one)
        const uint32_t rec = rec_s;
        if (rec >= n_rec) break;
        if (!ROBE_CHK(rec < a.long_cap, ROBE_DBG_LONG_WALK)) break;
        const LongWalk* lw = a.long_walks + rec;
        const uint64_t i0 = lw->i0;
        const uint32_t j = lw->j[lane];
        const uint32_t st = lw->state[lane];
        const uint32_t e = st & 0xFFu;
        const bool mine = (st >> 8) & 1u;  // this lane's walk was handed over
        float acc = lw->acc[lane];         // used by warp 0 only
        bool touched = (st >> 9) & 1u;
        auto fetch = [&](uint32_t r) -> uint2 {
            const uint64_t idx = i0 + r;
            if (idx >= a.nb) return make_uint2(kNoKey, 0u);
            return make_uint2(__ldg(K + idx), __ldg(V + idx));
        };
        // This copier warp's share of the copies of the step that starts at tile-relative position `base`.
        auto issue = [&](uint32_t base, uint32_t buf) {
            const uint32_t dst = dst0 + buf * kBufBytes;
            uint2 kv[kPerCopier];
#pragma unroll
            for (int q = 0; q < kPerCopier; ++q) {
                const uint32_t t = (w - 1) + q * kLongCopiers;
                kv[q] = ring[(base + e + (t < (uint32_t)kLongStep ? t : 0u)) & (kLongRing - 1)];
            }
#pragma unroll
            for (int q = 0; q < kPerCopier; ++q) {
                const uint32_t t = (w - 1) + q * kLongCopiers;
                if (t < (uint32_t)kLongStep && mine && kv[q].x <= j &&
                    ROBE_CHK((uint64_t)kv[q].y + (j - kv[q].x) < a.grad_elems, ROBE_DBG_GRAD_POS)) {
                    const float* src = a.grad_out + (kv[q].y + (j - kv[q].x));
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + t * 128u), "l"(src));
                }
            }
            asm volatile("cp.async.commit_group;");
        };
        // How many positions of that step reach slot j: first t with key > j, by bisection.
        auto reach = [&](uint32_t base) -> uint32_t {
            if (!mine) return 0u;
            uint32_t lo = 0, hi = kLongStep;
            while (lo < hi) {
                const uint32_t mid = (lo + hi) >> 1;
                if (ring[(base + e + mid) & (kLongRing - 1)].x <= j) lo = mid + 1; else hi = mid;
            }
            return lo;
        };
        // a step reads positions base + e + t, e < 32, t < kLongStep: [base, base + kLongStep + 32);
        // the ring is kept filled up to the end of the step kLongDepth steps ahead
        constexpr uint32_t kAhead = (kLongDepth + 1) * kLongStep + 32;
        uint32_t base = lw->fbase;
        uint32_t ring_end = base + kAhead;
        for (uint32_t r = tid; r < kAhead; r += 32 * kLongWarps)
            ring[(base + r) & (kLongRing - 1)] = fetch(base + r);
        if (tid == 0) go_on[0] = 1u;
        __syncthreads();
        uint2 pend0 = make_uint2(kNoKey, 0u), pend1 = pend0;  // scout: keys of ring_end + lane, + 32 + lane
        if (scout) {
            pend0 = fetch(ring_end + lane);
            pend1 = fetch(ring_end + 32 + lane);
            reach_s[0][lane] = reach(base);
        } else if (!adder) {
#pragma unroll
            for (int s = 0; s < kLongDepth; ++s) issue(base + s * kLongStep, s);
            asm volatile("cp.async.wait_group %0;" ::"n"(kLongDepth - 1) : "memory");  // step 0 is in
        }
        for (uint32_t step = 0;; ++step) {
            // the copies of `step` are in (every copier waited for its own) and the adds of
            // step - 1 are done, so its buffer may be refilled; the ring holds the next keys
            __syncthreads();
            if (go_on[step & 1u] == 0) break;
            if (adder) {
                const float(*buf)[32] = terms_s[step % kLongBufs];
                const uint32_t n_cur = reach_s[step & 1u][lane];
                const uint32_t n_max = __reduce_max_sync(0xFFFFFFFFu, n_cur);
                for (uint32_t t0 = 0; t0 < n_max; t0 += 16) {
                    float x[16];
#pragma unroll
                    for (int q = 0; q < 16; ++q) x[q] = buf[t0 + q][lane];
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        if (t0 + q < n_cur) acc = __fadd_rn(acc, x[q]);
                }
                if (n_cur != 0) touched = true;
            } else if (scout) {
                // keys: asked for a whole iteration before they are stored into the ring
                const uint2 f0 = fetch(ring_end + kLongStep + lane);
                const uint2 f1 = fetch(ring_end + kLongStep + 32 + lane);
                const uint32_t n_nxt = reach(base + kLongStep);
                reach_s[(step + 1) & 1u][lane] = n_nxt;
                const bool any_next = __ballot_sync(0xFFFFFFFFu, n_nxt != 0) != 0;
                if (lane == 0) go_on[(step + 1) & 1u] = any_next ? 1u : 0u;
                ring[(ring_end + lane) & (kLongRing - 1)] = pend0;
                ring[(ring_end + 32 + lane) & (kLongRing - 1)] = pend1;
                pend0 = f0;
                pend1 = f1;
            } else {
                issue(base + kLongDepth * kLongStep, (step + kLongDepth) % kLongBufs);
                asm volatile("cp.async.wait_group %0;" ::"n"(kLongDepth - 1) : "memory");  // step + 1 is in
            }
            ring_end += kLongStep;
            base += kLongStep;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (adder && mine && touched) commit_slot<MODE>(a, j, acc, a.target[j]);
    }
}

// Slots j in [0, Z-1): plain blocks with key <= j first, then the wrapped tails of blocks
// whose key lies in [m + j - (Z-1), m-1] (o = j + m - key).  One warp per slot: the lanes fetch
// the terms of 32 consecutive sorted positions, then all lanes add them in order.
constexpr unsigned kLowWarps = 4;

template <bool SIGN, bool SHORT>
__device__ __forceinline__ void low_walk(const ApplyArgs& a, const uint32_t* __restrict__ K,
                                         const uint32_t* __restrict__ V, const uint32_t* bag_of,
                                         uint64_t from, uint64_t to, uint64_t j_plus, float& acc,
                                         bool& touched) {
    const uint32_t lane = threadIdx.x & 31;
    for (uint64_t i0 = from; i0 < to; i0 += 32) {
        const uint64_t i = i0 + lane;
        float term = 0.0f;
        bool ok = false;
        if (i < to) ok = block_term<SIGN, SHORT>(a, bag_of, __ldg(V + i), (uint32_t)(j_plus - __ldg(K + i)), term);
        const uint32_t oks = __ballot_sync(0xFFFFFFFFu, ok);
        if (oks != 0) touched = true;
        for (uint32_t rest = oks; rest != 0; rest &= rest - 1) {
            const int src = __ffs((int)rest) - 1;
            acc = __fadd_rn(acc, __shfl_sync(0xFFFFFFFFu, term, src));
        }
    }
}

// first sorted position with key >= bound (warp-uniform)
__device__ __forceinline__ uint64_t first_at_least(const uint32_t* __restrict__ K, uint64_t nb, uint64_t bound) {
    uint64_t lo = 0, hi = nb;
    while (lo < hi) {
        const uint64_t mid = lo + ((hi - lo) >> 1);
        if ((uint64_t)__ldg(K + mid) >= bound) hi = mid; else lo = mid + 1;
    }
    return lo;
}

template <bool SIGN, int MODE, bool SHORT>
__global__ void __launch_bounds__(32 * kLowWarps)
det_apply_low_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                     const uint32_t* __restrict__ bag_of) {
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    const uint32_t j = blockIdx.x * kLowWarps + (threadIdx.x >> 5);
    if (j + 1 >= mp.Z) return;
    float acc = 0.0f;
    bool touched = false;
    low_walk<SIGN, SHORT>(a, K, V, bag_of, 0, first_at_least(K, a.nb, (uint64_t)j + 1), j, acc, touched);
    const uint64_t lowkey = (uint64_t)mp.m - (mp.Z - 1) + j;  // > j because m >= Z
    low_walk<SIGN, SHORT>(a, K, V, bag_of, first_at_least(K, a.nb, lowkey), a.nb, (uint64_t)j + mp.m, acc,
                          touched);
    if (touched && (threadIdx.x & 31) == 0) commit_slot<MODE>(a, j, acc, a.target[j]);
}

// Binned (not deterministic) backward: after ONE scatter pass on the top key bits the blocks are
// grouped by array region (a bin covers 2^shift consecutive slots, 16 MB or so), and this kernel
// adds them in that order with red.global: thread (i, u) adds term u of sorted block i.  The
// blocks in flight at any moment fall into one or two bins, so the read-modify-write of the array
// happens in L2 and every array sector crosses the DRAM bus about once per call instead of once
// per block that touches it.  a.lr carries the scale (1 for a dense gradient, -lr for SGD).
constexpr int kBinnedPer = 8;  // sorted blocks per thread group, all their loads in flight together

template <bool SIGN, bool SHORT>
__global__ void __launch_bounds__(256)
binned_apply_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                    const uint32_t* __restrict__ bag_of, uint32_t log2Zp) {
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    const uint64_t tid = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    const uint64_t i0 = (tid >> log2Zp) * kBinnedPer;
    const uint32_t u = (uint32_t)(tid & ((1u << log2Zp) - 1u));
    if (i0 >= a.nb || u >= mp.Z) return;
    uint32_t k[kBinnedPer], v[kBinnedPer];
#pragma unroll
    for (int t = 0; t < kBinnedPer; ++t) {
        const uint64_t i = i0 + t < a.nb ? i0 + t : a.nb - 1;
        k[t] = __ldg(K + i);
        v[t] = __ldg(V + i);
    }
    const uint64_t pol = l2_keep_policy(a.l2_keep != 0);
    float term[kBinnedPer];
    bool ok[kBinnedPer];
#pragma unroll
    for (int t = 0; t < kBinnedPer; ++t)
        ok[t] = i0 + t < a.nb && block_term<SIGN, SHORT>(a, bag_of, v[t], u, term[t]);
#pragma unroll
    for (int t = 0; t < kBinnedPer; ++t) {
        if (ok[t]) {
            uint64_t j = (uint64_t)k[t] + u;
            if (j >= mp.m) j -= mp.m;
            if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) red_add(a.target + j, a.lr * term[t], pol);
        }
    }
}

uint32_t bits_for(uint32_t m) {  // bits needed for keys in [0, m)
    uint32_t b = 1;
    while (b < 32 && (1ull << b) < (uint64_t)m) ++b;
    return b;
}

struct Layout {
    size_t keysA, keysB, valsA, valsB, bag_of, counts, totals, long_count, long_walks, bounds, win_left,
        total;
    uint32_t long_cap, nwin, win_log2;
};

// Window length of the window apply: 2048 slots, fewer for a small array so that there are
// still several CTAs per SM.
uint32_t window_log2(uint32_t m) {
    uint32_t l = kWinLog2Max;
    while (l > kWinLog2Min && (m >> l) < 1024u) --l;
    return l;
}

Layout make_layout(uint64_t nb, int64_t nnz, bool bags, uint32_t m) {
    Layout L;
    size_t off = 0;
    const size_t kb = align256((nb ? nb : 1) * sizeof(uint32_t));
    L.keysA = off; off += kb;
    L.keysB = off; off += kb;
    L.valsA = off; off += kb;
    L.valsB = off; off += kb;
    L.bag_of = off; off += bags ? align256((size_t)(nnz ? nnz : 1) * sizeof(uint32_t)) : 0;
    L.counts = off; off += align256((size_t)kRadix * kSortMaxGrid * sizeof(uint32_t));
    L.totals = off; off += align256((size_t)kRadix * sizeof(uint32_t));
    // list of long walks: room for one round per 128 blocks, within 64 .. 2^20 rounds
    uint64_t cap = nb / 128;
    cap = cap < 64 ? 64 : (cap > (1u << 20) ? (1u << 20) : cap);
    L.long_cap = (uint32_t)cap;
    L.long_count = off; off += 256;
    L.long_walks = off; off += align256((size_t)cap * sizeof(LongWalk));
    // window apply: first sorted position of every array window, a left-over flag per window and,
    // in the flag array's first aligned word past the flags, the count of left-over windows
    L.win_log2 = window_log2(m);
    L.nwin = (uint32_t)((((uint64_t)m - 1) >> L.win_log2) + 1);
    L.bounds = off; off += 2 * align256(((size_t)L.nwin + 1) * sizeof(uint32_t));
    L.win_left = off; off += align256((size_t)L.nwin + 256);
    L.total = off;
    return L;
}

// The window kernel pays when most slots are reached, so that walking every slot is no waste.
bool use_window_apply(const MapParams& mp, uint64_t nb, bool sign) {
    if (sign || mp.d % mp.Z != 0 || mp.Z > kWinMaxZ || nb == 0) return false;
    return nb * mp.Z * 2 >= mp.m;
}

struct WindowBuffers {
    uint32_t* lo_of;
    uint32_t* hi_of;
    uint8_t* left;
    uint32_t nwin, win_log2;
    // second stream for the kernels that serve the left-over windows, or nullptr
    cudaStream_t side;
    cudaEvent_t fork_event, join_event;
};

template <bool SIGN, int MODE>
void launch_apply(ApplyArgs aa, const uint32_t* K, const uint32_t* V, const uint32_t* bag_of,
                  const WindowBuffers& wb, cudaStream_t st) {
    const MapParams& mp = aa.mp;
    const bool windows = !SIGN && use_window_apply(mp, aa.nb, SIGN);
    uint32_t chunk = kWinStage / mp.Z;
    if (chunk > kWinEnt) chunk = kWinEnt;
    if (windows) {
        const size_t flags = ((size_t)wb.nwin + 255) & ~(size_t)255;
        uint32_t* any_left = (uint32_t*)(wb.left + flags);
        cudaMemsetAsync(any_left, 0, sizeof(uint32_t), st);
        const uint64_t per_cta = 256ull * kBoundsPer;
        det_bounds_kernel<<<(unsigned)(aa.nb / per_cta + 1), 256, 0, st>>>(K, aa.nb, wb.lo_of, wb.hi_of,
                                                                          wb.nwin, wb.win_log2, mp.Z, aa.status);
        // a window reached by many times the average number of blocks holds an often repeated id
        const uint64_t mean = (((uint64_t)1 << wb.win_log2) + mp.Z) * aa.nb / mp.m + 1;
        const uint64_t n_max = mean * 4 > 512 ? mean * 4 : 512;
        det_window_classify_kernel<<<(wb.nwin + 255) / 256, 256, 0, st>>>(
            wb.lo_of, wb.hi_of, wb.nwin, (uint32_t)(n_max < 0xFFFFFFFFull ? n_max : 0xFFFFFFFFull), wb.left,
            any_left, aa.status);
        aa.win_left = wb.left;
        aa.any_left = any_left;
        aa.win_log2 = wb.win_log2;
    }
    // With windows, the kernels below serve the left-over windows only: a few long-running CTAs.
    // They go to the second stream (of higher priority) and the window kernel runs beside them.
    const bool forked = windows && wb.side != nullptr;
    cudaStream_t ts = st;
    if (forked) {
        cudaEventRecord(wb.fork_event, st);
        cudaStreamWaitEvent(wb.side, wb.fork_event, 0);
        ts = wb.side;
    }
    const unsigned blocks = (unsigned)((aa.nb + 255) / 256);  // one warp per 32 sorted positions
    const unsigned low_blocks = (mp.Z - 1 + kLowWarps - 1) / kLowWarps;  // one warp per low slot
    if (mp.d % mp.Z != 0) {
        det_apply_kernel<SIGN, MODE, true><<<blocks, 256, 0, ts>>>(aa, K, V, bag_of);
        if (mp.Z > 1)
            det_apply_low_kernel<SIGN, MODE, true><<<low_blocks, 32 * kLowWarps, 0, ts>>>(aa, K, V, bag_of);
    } else {
        det_apply_kernel<SIGN, MODE, false><<<blocks, 256, 0, ts>>>(aa, K, V, bag_of);
        if (!SIGN) {
            // the rounds the apply kernel handed over; a grid-stride loop over the list
            const unsigned lblocks = aa.long_cap < 148u * 8u ? aa.long_cap : 148u * 8u;
            det_apply_long_kernel<MODE><<<lblocks, 32 * kLongWarps, 0, ts>>>(aa, K, V);
        }
        if (mp.Z > 1)
            det_apply_low_kernel<SIGN, MODE, false><<<low_blocks, 32 * kLowWarps, 0, ts>>>(aa, K, V, bag_of);
    }
    if (forked) cudaEventRecord(wb.join_event, wb.side);
    if (windows) {
        const int vec4 = mp.Z % 4 == 0 && mp.d % 4 == 0 && ((uintptr_t)aa.grad_out & 15) == 0;
        switch (wb.win_log2) {
            case 9: det_apply_window_kernel<MODE, 9><<<wb.nwin, kWinThreads, 0, st>>>(aa, K, V, wb.lo_of, wb.hi_of, chunk, vec4); break;
            case 10: det_apply_window_kernel<MODE, 10><<<wb.nwin, kWinThreads, 0, st>>>(aa, K, V, wb.lo_of, wb.hi_of, chunk, vec4); break;
            default: det_apply_window_kernel<MODE, 11><<<wb.nwin, kWinThreads, 0, st>>>(aa, K, V, wb.lo_of, wb.hi_of, chunk, vec4); break;
        }
    }
    if (forked) cudaStreamWaitEvent(st, wb.join_event, 0);
}

}  // namespace

size_t det_workspace_bytes(const MapParams& mp, int64_t nbags, int64_t nnz, bool bags) {
    (void)nbags;
    const uint64_t nb = (uint64_t)nnz * mp.C;
    return make_layout(nb, nnz, bags, mp.m).total;
}

void block_key_buffers(const Problem& pb, void* workspace, uint32_t** keys, uint32_t** vals) {
    const uint64_t nb = (uint64_t)pb.nnz * pb.mp.C;
    const Layout L = make_layout(nb, pb.nnz, pb.offsets != nullptr, pb.mp.m);
    *keys = (uint32_t*)((char*)workspace + L.keysA);
    *vals = (uint32_t*)((char*)workspace + L.valsA);
}

// bag_of (pooled input) into the workspace
static void launch_bag_of(const Problem& pb, const Layout& L, char* ws, cudaStream_t st) {
    uint32_t* bag_of = (uint32_t*)(ws + L.bag_of);
    KeyArgs ka{pb.mp, pb.indices, pb.offsets, pb.nbags, pb.nnz, pb.status};
    // positions that malformed offsets leave uncovered fall back to bag 0 (memory-safe)
    cudaMemsetAsync(bag_of, 0, (size_t)pb.nnz * sizeof(uint32_t), st);
    det_bag_of_kernel<<<(unsigned)((pb.nbags + 7) / 8), 256, 0, st>>>(ka, bag_of);
}

cudaError_t launch_block_keys(const Problem& pb, void* workspace, size_t workspace_bytes,
                              cudaStream_t st) {
    if (pb.nnz == 0 || pb.nbags == 0) return cudaSuccess;
    const MapParams& mp = pb.mp;
    const bool bags = pb.offsets != nullptr;
    const uint64_t nb = (uint64_t)pb.nnz * mp.C;
    const Layout L = make_layout(nb, pb.nnz, bags, mp.m);
    if (workspace == nullptr || workspace_bytes < L.total) return cudaErrorInvalidValue;
    char* ws = (char*)workspace;
    uint32_t* kA = (uint32_t*)(ws + L.keysA);
    uint32_t* vA = (uint32_t*)(ws + L.valsA);
    uint32_t* bag_of = bags ? (uint32_t*)(ws + L.bag_of) : nullptr;
    KeyArgs ka{mp, pb.indices, pb.offsets, pb.nbags, pb.nnz, pb.status};
    if (bags) launch_bag_of(pb, L, ws, st);
    if (mp.C <= 8) {
        const unsigned kb = (unsigned)((pb.nnz + 255) / 256);
        if (pb.sign) det_keys_kernel<true><<<kb, 256, 0, st>>>(ka, bag_of, kA, vA);
        else det_keys_kernel<false><<<kb, 256, 0, st>>>(ka, bag_of, kA, vA);
    } else {
        const unsigned kb = (unsigned)((nb + 255) / 256);
        if (pb.sign) det_keys_by_block_kernel<true><<<kb, 256, 0, st>>>(ka, bag_of, kA, vA, nb);
        else det_keys_by_block_kernel<false><<<kb, 256, 0, st>>>(ka, bag_of, kA, vA, nb);
    }
    return cudaGetLastError();
}

cudaError_t launch_backward_det(const Problem& pb, const float* grad_out, float* target, int mode,
                                float lr, const AdamState* adam, void* workspace,
                                size_t workspace_bytes, cudaStream_t st, bool keys_kept) {
    if (pb.nnz == 0 || pb.nbags == 0) return cudaSuccess;
    const MapParams& mp = pb.mp;
    const bool bags = pb.offsets != nullptr;
    const uint64_t nb = (uint64_t)pb.nnz * mp.C;
    const Layout L = make_layout(nb, pb.nnz, bags, mp.m);
    if (workspace == nullptr || workspace_bytes < L.total) return cudaErrorInvalidValue;
    // the payload of a block is a 32-bit position in grad_out
    if ((uint64_t)pb.nbags * mp.d > (1ull << 32)) return cudaErrorInvalidValue;
    char* ws = (char*)workspace;
    uint32_t* kA = (uint32_t*)(ws + L.keysA);
    uint32_t* kB = (uint32_t*)(ws + L.keysB);
    uint32_t* vA = (uint32_t*)(ws + L.valsA);
    uint32_t* vB = (uint32_t*)(ws + L.valsB);
    uint32_t* bag_of = bags ? (uint32_t*)(ws + L.bag_of) : nullptr;
    uint32_t* counts = (uint32_t*)(ws + L.counts);
    uint32_t* totals = (uint32_t*)(ws + L.totals);

    if (!keys_kept) {
        const cudaError_t err = launch_block_keys(pb, workspace, workspace_bytes, st);
        if (err != cudaSuccess) return err;
    } else if (bags && pb.sign) {
        launch_bag_of(pb, L, ws, st);  // the signed terms look the id's bag up again
    }

    const SortPlan sp = make_plan(nb);
    const uint32_t bits = bits_for(mp.m);
    if (mode == 3) {
        // binned: one pass on the top key bits, then atomic adds in bin order.  A bin spans 2^22
        // slots (16 MB of fp32: the span that measured fastest on a 1 GB array - small enough to
        // be updated in L2, large enough that the scatter writes long runs) unless that would
        // need more than 256 bins or the array is smaller than one such span.
        const uint32_t shift = bits > 30 ? bits - 8 : (bits > 22 ? 22 : (bits > 8 ? bits - 8 : 0));
        const uint32_t mask = (1u << (bits - shift)) - 1u;
        sort_count_kernel<<<sp.grid, kSortThreads, 0, st>>>(kA, counts, nb, sp.tiles, shift, mask);
        sort_scan_kernel<<<kRadix, kSortThreads, 0, st>>>(counts, totals, sp.grid);
        sort_scatter_kernel<false><<<sp.grid, kSortThreads, 0, st>>>(kA, vA, kB, vB, counts, totals, nb,
                                                                    sp.tiles, shift, mask);
        ApplyArgs ab{mp, grad_out, pb.indices, target, lr, nb, pb.status, AdamState{}, nullptr, nullptr, 0,
                     nullptr, nullptr, 0, (uint64_t)pb.nbags * mp.d, pb.l2_keep};
        uint32_t log2Zp = 0;
        while ((1u << log2Zp) < mp.Z) ++log2Zp;
        const uint64_t groups = (nb + kBinnedPer - 1) / kBinnedPer;
        const unsigned blocks = (unsigned)(((groups << log2Zp) + 255) / 256);
        const bool shortb = mp.d % mp.Z != 0;
        if (pb.sign) {
            if (shortb) binned_apply_kernel<true, true><<<blocks, 256, 0, st>>>(ab, kB, vB, bag_of, log2Zp);
            else binned_apply_kernel<true, false><<<blocks, 256, 0, st>>>(ab, kB, vB, bag_of, log2Zp);
        } else {
            if (shortb) binned_apply_kernel<false, true><<<blocks, 256, 0, st>>>(ab, kB, vB, bag_of, log2Zp);
            else binned_apply_kernel<false, false><<<blocks, 256, 0, st>>>(ab, kB, vB, bag_of, log2Zp);
        }
        return cudaGetLastError();
    }
    const uint32_t npass = (bits + 7) / 8;
    const uint32_t bpp = (bits + npass - 1) / npass;
    for (uint32_t pass = 0; pass < npass; ++pass) {
        const uint32_t shift = pass * bpp;
        const uint32_t width = bits - shift < bpp ? bits - shift : bpp;
        const uint32_t mask = (1u << width) - 1u;
        sort_count_kernel<<<sp.grid, kSortThreads, 0, st>>>(kA, counts, nb, sp.tiles, shift, mask);
        sort_scan_kernel<<<kRadix, kSortThreads, 0, st>>>(counts, totals, sp.grid);
        sort_scatter_kernel<true><<<sp.grid, kSortThreads, 0, st>>>(kA, vA, kB, vB, counts, totals, nb,
                                                                   sp.tiles, shift, mask);
        uint32_t* t = kA; kA = kB; kB = t;
        t = vA; vA = vB; vB = t;
    }

    uint32_t* long_count = (uint32_t*)(ws + L.long_count);
    cudaMemsetAsync(long_count, 0, 2 * sizeof(uint32_t), st);  // [0] rounds handed over, [1] rounds taken
    ApplyArgs aa{mp, grad_out, pb.indices, target, lr, nb, pb.status, adam ? *adam : AdamState{},
                 long_count, (LongWalk*)(ws + L.long_walks), L.long_cap, nullptr, nullptr, 0,
                 (uint64_t)pb.nbags * mp.d, 0};
    const WindowBuffers wb{(uint32_t*)(ws + L.bounds),
                           (uint32_t*)(ws + L.bounds + align256(((size_t)L.nwin + 1) * sizeof(uint32_t))),
                           (uint8_t*)(ws + L.win_left), L.nwin, L.win_log2,
                           pb.side, pb.fork_event, pb.join_event};
    if (pb.sign) {
        if (mode == 4) launch_apply<true, 3>(aa, kA, vA, bag_of, wb, st);
        else if (mode == 2) launch_apply<true, 2>(aa, kA, vA, bag_of, wb, st);
        else if (mode == 1) launch_apply<true, 1>(aa, kA, vA, bag_of, wb, st);
        else launch_apply<true, 0>(aa, kA, vA, bag_of, wb, st);
    } else {
        if (mode == 4) launch_apply<false, 3>(aa, kA, vA, bag_of, wb, st);
        else if (mode == 2) launch_apply<false, 2>(aa, kA, vA, bag_of, wb, st);
        else if (mode == 1) launch_apply<false, 1>(aa, kA, vA, bag_of, wb, st);
        else launch_apply<false, 0>(aa, kA, vA, bag_of, wb, st);
    }
    return cudaGetLastError();
}

}  // namespace robe
