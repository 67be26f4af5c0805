// Deterministic backward (Section 3.1 backward equation, evaluated in a fixed order).
//
// Blocks are numbered q = p*C + c in input order (p = position in indices, c = chunk).
//   1. key kernel      key[q] = h(e, x_p, c), val[q] = q
//   2. radix sort      stable LSD sort of (key, val) by key - our own three-kernel passes
//                      (digit count per CTA range, exclusive scan, ranked scatter)
//   3. apply kernel    one thread per touched array slot j walks the sorted blocks whose
//                      key lies in [j-Z+1, j] in sorted order and sums their terms left to
//                      right in fp32 from +0, then performs ONE add (dense gradient) or ONE
//                      fma (SGD) on slot j.  Slots [0, Z-1), which also receive the wrapped
//                      tails of blocks near the end of the array, are handled by a small
//                      second kernel (those terms come last: their keys are the largest).
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
    const int64_t* indices;
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

// key[q] = h(e, x_p, c), val[q] = q for q = p*C + c
__global__ void __launch_bounds__(256)
det_keys_kernel(KeyArgs a, const uint32_t* bag_of, uint32_t* keys, uint32_t* vals, uint64_t nb) {
    const uint64_t q = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (q >= nb) return;
    const MapParams& mp = a.mp;
    const uint64_t p = q / mp.C;
    const uint32_t c = (uint32_t)(q - p * mp.C);
    const uint64_t bag = bag_of ? (uint64_t)bag_of[p] : p;
    const uint32_t e = table_of_bag(bag, mp);
    const uint64_t x = (uint64_t)__ldg(a.indices + p);
    keys[q] = block_start(mp, hash_base(mp.h, e, x), c);
    vals[q] = (uint32_t)q;
}

// ---- radix sort pass, kernel 1: digit histogram of each CTA's contiguous key range
__global__ void __launch_bounds__(kSortThreads)
sort_count_kernel(const uint32_t* keys, uint32_t* counts, uint64_t nb, uint64_t tiles,
                  uint32_t shift, uint32_t mask) {
    __shared__ uint32_t hist[kRadix];
    hist[threadIdx.x] = 0;
    __syncthreads();
    uint64_t first, count;
    cta_tiles(tiles, gridDim.x, blockIdx.x, first, count);
    const uint64_t begin = first * kSortTile;
    uint64_t end = (first + count) * kSortTile;
    if (end > nb) end = nb;
    for (uint64_t i = begin + threadIdx.x; i < end; i += kSortThreads)
        atomicAdd(&hist[(keys[i] >> shift) & mask], 1u);
    __syncthreads();
    counts[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x] = hist[threadIdx.x];
}

// ---- kernel 2: exclusive scan of counts[digit][cta] in digit-major order (one CTA)
__global__ void __launch_bounds__(1024) sort_scan_kernel(uint32_t* counts, uint32_t n) {
    __shared__ uint32_t partial[1024];
    const uint32_t per = (n + 1023) / 1024;
    const uint32_t lo = threadIdx.x * per;
    const uint32_t hi = lo + per < n ? lo + per : n;
    uint32_t sum = 0;
    for (uint32_t i = lo; i < hi; ++i) sum += counts[i];
    partial[threadIdx.x] = sum;
    __syncthreads();
    // Hillis-Steele inclusive scan over the 1024 partial sums
    for (uint32_t offs = 1; offs < 1024; offs <<= 1) {
        uint32_t v = threadIdx.x >= offs ? partial[threadIdx.x - offs] : 0;
        __syncthreads();
        partial[threadIdx.x] += v;
        __syncthreads();
    }
    uint32_t run = partial[threadIdx.x] - sum;  // exclusive prefix of this thread's range
    for (uint32_t i = lo; i < hi; ++i) {
        uint32_t c = counts[i];
        counts[i] = run;
        run += c;
    }
}

// ---- kernel 3: stable ranked scatter
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* kin, const uint32_t* vin, uint32_t* kout, uint32_t* vout,
                    const uint32_t* offsets, uint64_t nb, uint64_t tiles, uint32_t shift,
                    uint32_t mask) {
    __shared__ uint32_t base[kRadix];
    __shared__ uint32_t wcnt[kSortWarps][kRadix];
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    base[threadIdx.x] = offsets[(uint64_t)threadIdx.x * gridDim.x + blockIdx.x];
    uint64_t first, count;
    cta_tiles(tiles, gridDim.x, blockIdx.x, first, count);
    for (uint64_t t = first; t < first + count; ++t) {
        for (int k = 0; k < kSortWarps; ++k) wcnt[k][threadIdx.x] = 0;
        __syncthreads();
        const uint64_t wbegin = t * kSortTile + (uint64_t)w * (32 * kSortItems);
        uint32_t key[kSortItems], rank[kSortItems];
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
            const uint64_t idx = wbegin + r * 32 + lane;
            const bool valid = idx < nb;
            key[r] = valid ? kin[idx] : 0u;
            const uint32_t dg = valid ? ((key[r] >> shift) & mask) : (uint32_t)kRadix;
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, dg);
            uint32_t before = 0;
            if (valid) before = wcnt[w][dg];
            __syncwarp();
            if (valid && (peers & lt) == 0) wcnt[w][dg] = before + __popc(peers);
            __syncwarp();
            rank[r] = before + __popc(peers & lt);
        }
        __syncthreads();
        // exclusive prefix over the warps of this tile, per digit
        uint32_t tile_total = 0;
        {
            uint32_t run = 0;
            for (int k = 0; k < kSortWarps; ++k) {
                uint32_t c = wcnt[k][threadIdx.x];
                wcnt[k][threadIdx.x] = run;
                run += c;
            }
            tile_total = run;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
            const uint64_t idx = wbegin + r * 32 + lane;
            if (idx < nb) {
                const uint32_t dg = (key[r] >> shift) & mask;
                const uint32_t dst = base[dg] + wcnt[w][dg] + rank[r];
                kout[dst] = key[r];
                vout[dst] = vin[idx];
            }
        }
        __syncthreads();
        base[threadIdx.x] += tile_total;
        __syncthreads();
    }
}

struct ApplyArgs {
    MapParams mp;
    const float* grad_out;
    const int64_t* indices;  // only read when the sign hash is on
    float* target;
    float lr;
    uint64_t nb;
    const int32_t* status;
};

// The term block (key, q) contributes to slot at in-block offset o, or nothing if o is past
// the (possibly short) block.
template <bool SIGN>
__device__ __forceinline__ bool block_term(const ApplyArgs& a, const uint32_t* bag_of, uint32_t q,
                                           uint32_t o, float& term) {
    const MapParams& mp = a.mp;
    const uint32_t p = q / mp.C;
    const uint32_t c = q - p * mp.C;
    const uint32_t i = c * mp.Z + o;
    if (o >= mp.Z || i >= mp.d) return false;
    const uint64_t bag = bag_of ? (uint64_t)__ldg(bag_of + p) : (uint64_t)p;
    term = __ldg(a.grad_out + bag * mp.d + i);
    if (SIGN) {
        const uint32_t e = table_of_bag(bag, mp);
        const uint64_t x = (uint64_t)__ldg(a.indices + p);
        term = sign_of(mp, hash_base(mp.g, e, x), i) * term;
    }
    return true;
}

template <bool SGD>
__device__ __forceinline__ void commit_slot(float* target, uint32_t j, float acc, float lr) {
    if (SGD) target[j] = __fmaf_rn(-lr, acc, target[j]);
    else target[j] = __fadd_rn(target[j], acc);
}

// Slots j in [Z-1, m): thread (i, u) serves slot K[i]+u if sorted position i starts a run of
// equal keys and no later run starts at or before that slot.
template <bool SIGN, bool SGD>
__global__ void __launch_bounds__(256)
det_apply_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                 const uint32_t* __restrict__ bag_of, uint32_t log2Zp) {
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    const uint64_t tid = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    const uint64_t i = tid >> log2Zp;
    const uint32_t u = (uint32_t)(tid & ((1u << log2Zp) - 1u));
    if (i >= a.nb || u >= mp.Z) return;
    const uint32_t kh = K[i];
    if (i > 0 && K[i - 1] == kh) return;  // not the first of its run
    const uint64_t j64 = (uint64_t)kh + u;
    if (j64 >= mp.m || j64 + 1 < mp.Z) return;  // wrapped part / low slots: other kernel
    const uint32_t j = (uint32_t)j64;

    // end of the run of kh (galloping, then bisection)
    uint64_t lo = i, hi = i + 1, step = 1;
    while (hi < a.nb && K[hi] == kh) {
        lo = hi;
        step <<= 1;
        hi = lo + step;
    }
    if (hi > a.nb) hi = a.nb;
    while (hi - lo > 1) {
        const uint64_t mid = lo + ((hi - lo) >> 1);
        if (K[mid] == kh) lo = mid; else hi = mid;
    }
    const uint64_t run_end = hi;
    if (run_end < a.nb && K[run_end] <= j) return;  // a later run owns slot j

    // first sorted position whose key reaches slot j: key >= j - (Z-1)
    const uint32_t lowkey = j - (mp.Z - 1);
    uint64_t first = i;
    if (lowkey < kh && i > 0) {
        uint64_t h2 = i, l2 = i;
        bool found_low = false;
        step = 1;
        while (h2 > 0) {
            const uint64_t probe = h2 >= step ? h2 - step : 0;
            if (K[probe] >= lowkey) {
                h2 = probe;
                step <<= 1;
            } else {
                l2 = probe;
                found_low = true;
                break;
            }
        }
        if (found_low) {
            while (h2 - l2 > 1) {
                const uint64_t mid = l2 + ((h2 - l2) >> 1);
                if (K[mid] >= lowkey) h2 = mid; else l2 = mid;
            }
        }
        first = h2;
    }

    float acc = 0.0f;
    bool touched = false;
    constexpr int PF = 4;
    for (uint64_t ii = first; ii < run_end; ii += PF) {
        float term[PF];
        bool ok[PF];
#pragma unroll
        for (int t = 0; t < PF; ++t) {
            ok[t] = false;
            if (ii + t < run_end) ok[t] = block_term<SIGN>(a, bag_of, V[ii + t], j - K[ii + t], term[t]);
        }
#pragma unroll
        for (int t = 0; t < PF; ++t)
            if (ok[t]) {
                acc = __fadd_rn(acc, term[t]);
                touched = true;
            }
    }
    if (touched) commit_slot<SGD>(a.target, j, acc, a.lr);
}

// Slots j in [0, Z-1): plain blocks with key <= j first, then the wrapped tails of blocks
// whose key lies in [m + j - (Z-1), m-1] (o = j + m - key).
template <bool SIGN, bool SGD>
__global__ void __launch_bounds__(128)
det_apply_low_kernel(ApplyArgs a, const uint32_t* __restrict__ K, const uint32_t* __restrict__ V,
                     const uint32_t* __restrict__ bag_of) {
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    for (uint32_t j = threadIdx.x; j + 1 < mp.Z; j += blockDim.x) {
        float acc = 0.0f, term;
        bool touched = false;
        for (uint64_t ii = 0; ii < a.nb && K[ii] <= j; ++ii)
            if (block_term<SIGN>(a, bag_of, V[ii], j - K[ii], term)) {
                acc = __fadd_rn(acc, term);
                touched = true;
            }
        const uint32_t lowkey = mp.m - (mp.Z - 1) + j;  // > j because m >= Z
        uint64_t lo = 0, hi = a.nb;                     // first position with key >= lowkey
        while (lo < hi) {
            const uint64_t mid = lo + ((hi - lo) >> 1);
            if (K[mid] >= lowkey) hi = mid; else lo = mid + 1;
        }
        for (uint64_t ii = lo; ii < a.nb; ++ii)
            if (block_term<SIGN>(a, bag_of, V[ii], j + (mp.m - K[ii]), term)) {
                acc = __fadd_rn(acc, term);
                touched = true;
            }
        if (touched) commit_slot<SGD>(a.target, j, acc, a.lr);
    }
}

uint32_t bits_for(uint32_t m) {  // bits needed for keys in [0, m)
    uint32_t b = 1;
    while (b < 32 && (1ull << b) < (uint64_t)m) ++b;
    return b;
}

struct Layout {
    size_t keysA, keysB, valsA, valsB, bag_of, counts, total;
};

Layout make_layout(uint64_t nb, int64_t nnz, bool bags) {
    Layout L;
    size_t off = 0;
    const size_t kb = align256((nb ? nb : 1) * sizeof(uint32_t));
    L.keysA = off; off += kb;
    L.keysB = off; off += kb;
    L.valsA = off; off += kb;
    L.valsB = off; off += kb;
    L.bag_of = off; off += bags ? align256((size_t)(nnz ? nnz : 1) * sizeof(uint32_t)) : 0;
    L.counts = off; off += align256((size_t)kRadix * kSortMaxGrid * sizeof(uint32_t));
    L.total = off;
    return L;
}

}  // namespace

size_t det_workspace_bytes(const MapParams& mp, int64_t nbags, int64_t nnz, bool bags) {
    (void)nbags;
    const uint64_t nb = (uint64_t)nnz * mp.C;
    return make_layout(nb, nnz, bags).total;
}

cudaError_t launch_backward_det(const Problem& pb, const float* grad_out, float* target, int sgd,
                                float lr, void* workspace, size_t workspace_bytes,
                                cudaStream_t st) {
    if (pb.nnz == 0 || pb.nbags == 0) return cudaSuccess;
    const MapParams& mp = pb.mp;
    const bool bags = pb.offsets != nullptr;
    const uint64_t nb = (uint64_t)pb.nnz * mp.C;
    const Layout L = make_layout(nb, pb.nnz, bags);
    if (workspace == nullptr || workspace_bytes < L.total) return cudaErrorInvalidValue;
    char* ws = (char*)workspace;
    uint32_t* kA = (uint32_t*)(ws + L.keysA);
    uint32_t* kB = (uint32_t*)(ws + L.keysB);
    uint32_t* vA = (uint32_t*)(ws + L.valsA);
    uint32_t* vB = (uint32_t*)(ws + L.valsB);
    uint32_t* bag_of = bags ? (uint32_t*)(ws + L.bag_of) : nullptr;
    uint32_t* counts = (uint32_t*)(ws + L.counts);

    KeyArgs ka{mp, pb.indices, pb.offsets, pb.nbags, pb.nnz, pb.status};
    if (bags) {
        // positions that malformed offsets leave uncovered fall back to bag 0 (memory-safe)
        cudaMemsetAsync(bag_of, 0, (size_t)pb.nnz * sizeof(uint32_t), st);
        det_bag_of_kernel<<<(unsigned)((pb.nbags + 7) / 8), 256, 0, st>>>(ka, bag_of);
    }
    det_keys_kernel<<<(unsigned)((nb + 255) / 256), 256, 0, st>>>(ka, bag_of, kA, vA, nb);

    const SortPlan sp = make_plan(nb);
    const uint32_t bits = bits_for(mp.m);
    const uint32_t npass = (bits + 7) / 8;
    const uint32_t bpp = (bits + npass - 1) / npass;
    for (uint32_t pass = 0; pass < npass; ++pass) {
        const uint32_t shift = pass * bpp;
        const uint32_t width = bits - shift < bpp ? bits - shift : bpp;
        const uint32_t mask = (1u << width) - 1u;
        sort_count_kernel<<<sp.grid, kSortThreads, 0, st>>>(kA, counts, nb, sp.tiles, shift, mask);
        sort_scan_kernel<<<1, 1024, 0, st>>>(counts, (uint32_t)kRadix * sp.grid);
        sort_scatter_kernel<<<sp.grid, kSortThreads, 0, st>>>(kA, vA, kB, vB, counts, nb, sp.tiles,
                                                             shift, mask);
        uint32_t* t = kA; kA = kB; kB = t;
        t = vA; vA = vB; vB = t;
    }

    ApplyArgs aa{mp, grad_out, pb.indices, target, lr, nb, pb.status};
    uint32_t log2Zp = 0;
    while ((1u << log2Zp) < mp.Z) ++log2Zp;
    const uint64_t threads = nb << log2Zp;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
#define ROBE_DET_LAUNCH(SIGN, SGD)                                                        \
    do {                                                                                  \
        det_apply_kernel<SIGN, SGD><<<blocks, 256, 0, st>>>(aa, kA, vA, bag_of, log2Zp);   \
        if (mp.Z > 1) det_apply_low_kernel<SIGN, SGD><<<1, 128, 0, st>>>(aa, kA, vA, bag_of); \
    } while (0)
    if (pb.sign) {
        if (sgd) ROBE_DET_LAUNCH(true, true); else ROBE_DET_LAUNCH(true, false);
    } else {
        if (sgd) ROBE_DET_LAUNCH(false, true); else ROBE_DET_LAUNCH(false, false);
    }
#undef ROBE_DET_LAUNCH
    return cudaGetLastError();
}

}  // namespace robe
