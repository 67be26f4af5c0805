// Pieces shared by the staged forward and backward kernels: bag bounds, the warp-private
// staging area, and the hash phase that fills it (Section 3.2, h equation).
#pragma once
#include "robe_device.cuh"

namespace robe {

__device__ __forceinline__ int64_t clamp64(int64_t v, int64_t lo, int64_t hi) {
    return v < lo ? lo : (v > hi ? hi : v);
}

// ids of bag k: indices[lo, hi); malformed offsets are clamped so no read leaves indices[].
__device__ __forceinline__ void bag_range(const int64_t* offsets, int64_t nnz, int64_t k,
                                          int64_t& lo, int64_t& hi) {
    if (offsets == nullptr) {
        lo = k;
        hi = k + 1;
    } else {
        lo = clamp64(__ldg(offsets + k), 0, nnz);
        hi = clamp64(__ldg(offsets + k + 1), lo, nnz);
    }
}

constexpr int kStageEntries = 256;  // block starts per warp
constexpr int kStageIds = 64;       // ids per warp batch

// The block starts of a batch are kept chunk-major: start[c * stride + t] is the start of chunk c
// of the t-th id of the batch, stride = ids per batch.  A lane that owns element i of every row
// then reads one column, start[chunk(i) * stride + t] for t = 0, 1, ..: consecutive words.
struct StageSmem {
    uint64_t cterm[128];               // (C_h * c) mod P, c < C (d <= 128)
    uint64_t base[8][kStageIds];       // per warp: hash base of each staged id
    uint32_t start[8][kStageEntries];  // per warp: block starts, chunk-major
    uint32_t piece[8][kStageIds];      // per warp, rows clubbed into one block only: (x mod R) d
};

// ids a warp stages per batch: as many as fit the staging area (and at least one)
inline uint32_t staged_ids_per_batch(const MapParams& mp, bool bags, bool sign) {
    uint32_t cap = kStageEntries / mp.C;
    const uint32_t idcap = sign ? kStageIds / 2 : kStageIds;
    if (cap > idcap) cap = idcap;
    if (cap < 1) cap = 1;
    if (!bags) {
        // one-hot: rows per warp; enough pairs to fill the lanes twice, not more, so that small
        // batches still spread over many warps
        uint32_t want = (64 + mp.C - 1) / mp.C;
        if (want < 1) want = 1;
        if (cap > want) cap = want;
    }
    return cap;
}

inline uint32_t chunk_magic(const MapParams& mp) { return ((1u << 20) + mp.C - 1) / mp.C; }

// CTA-wide, once per kernel: the per-chunk hash terms.  Contains a __syncthreads.
__device__ __forceinline__ void stage_init(StageSmem& sm, const MapParams& mp) {
    if (threadIdx.x < mp.C) sm.cterm[threadIdx.x] = mulmod_p61_u32(mp.h.C, threadIdx.x);
    __syncthreads();
}

// Where the hash phase also leaves the block starts for a later sort-based backward of the same
// ids: keys[q] = h(e, x_p, c) and vals[q] for block q = p*C + c, vals[q] = q when the sign hash is
// on, else the position bag*d + c*Z of the block's first gradient element.  keys == nullptr: not
// kept.  `bag` is the warp's bag in pooled mode (one-hot: row p is bag p).
struct KeepBlocks {
    uint32_t* keys;
    uint32_t* vals;
    uint64_t bag;
};

// Hash phase of one batch of cnt ids starting at position p0 (warp-collective).
//   step 1: one id per lane          -> base_s[t] = (A e + B x + D) mod P  (and the sign base)
//   step 2: one (id, chunk) per lane -> start_s[c*stride + t] = h(e, x, c)
// In pooled mode tterm/gterm are the bag's table terms; in one-hot mode the table of row
// p0+t is (p0+t) mod T.  The sign base shares the upper half of base_s (the batch is halved
// when the sign is on).  Returns (warp-uniform) whether some block of the batch may run past
// the end of the array, i.e. whether the gather has to wrap slot numbers at all.
template <bool SIGN, bool BAGS>
__device__ __forceinline__ bool stage_batch(StageSmem& sm, const MapParams& mp,
                                            const IdList& indices, int64_t p0, uint32_t cnt,
                                            uint32_t stride, uint64_t tterm, uint64_t gterm,
                                            uint32_t cmagic, uint32_t w, uint32_t lane,
                                            const KeepBlocks keep = KeepBlocks{nullptr, nullptr, 0}) {
    uint64_t* base_s = sm.base[w];
    uint64_t* gbase_s = base_s + kStageIds / 2;
    uint32_t* start_s = sm.start[w];
    for (uint32_t t = lane; t < cnt; t += 32) {
        const uint64_t x = (uint64_t)indices.load(p0 + t);
        uint64_t xh = x;  // what the location hash sees in place of the id
        if (mp.R > 1) {   // R rows share a block: hashed by floor(x/R), row x starts (x mod R) d in
            xh = x / mp.R;
            sm.piece[w][t] = (uint32_t)(x - xh * mp.R) * mp.d;
        }
        uint64_t tt = tterm, gt = gterm;
        if (!BAGS) {
            const uint32_t e = table_of_bag((uint64_t)(p0 + t), mp);
            tt = table_term(mp.h, e);
            if (SIGN) gt = table_term(mp.g, e);
        }
        base_s[t] = addmod_p61(tt, mulmod_p61_any(mp.h.B, xh));
        if (SIGN) gbase_s[t] = addmod_p61(gt, mulmod_p61_any(mp.g.B, x));
    }
    __syncwarp();
    const uint32_t entries = cnt * mp.C;
    const uint32_t last_fit = mp.m - mp.Z;  // a block starting beyond this reaches the array end
    bool wraps = false;
    for (uint32_t t = lane; t < entries; t += 32) {
        const uint32_t idl = (t * cmagic) >> 20;  // t / C, exact for t < 8192
        const uint32_t c = t - idl * mp.C;
        uint32_t s = mod_m(addmod_p61(base_s[idl], sm.cterm[c]), mp.m, mp.mu);
        if (mp.R > 1) {
            const uint64_t j = (uint64_t)s + sm.piece[w][idl];  // both below m
            s = (uint32_t)(j >= mp.m ? j - mp.m : j);
        }
        start_s[c * stride + idl] = s;
        wraps |= s > last_fit;
        if (keep.keys != nullptr) {  // consecutive lanes, consecutive words
            const uint64_t q = (uint64_t)p0 * mp.C + t;
            const uint64_t bag = BAGS ? keep.bag : (uint64_t)p0 + idl;
            keep.keys[q] = s;
            keep.vals[q] = SIGN ? (uint32_t)q : (uint32_t)(bag * mp.d + c * mp.Z);
        }
    }
    const bool any = __any_sync(0xFFFFFFFFu, wraps);
    __syncwarp();  // the stores above are visible to the whole warp from here on
    return any;
}

}  // namespace robe
