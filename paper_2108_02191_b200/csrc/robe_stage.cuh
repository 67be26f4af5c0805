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

// Resident CTAs of 256 threads per SM that the staged kernels' register budget is set for.  Rows of up
// to 64 elements come in two builds: 8 CTAs (32 registers; the kernels then spill 8-24 bytes per
// thread) for arrays of L2 size, where the gather is bound by L2 latency and the extra warps pay
// (2-8 % measured on B200), and 6 CTAs (40 registers, no spill) for arrays in HBM, where occupancy buys
// nothing and the spill traffic costs DRAM bandwidth (cfg 4 forward 0.895 -> 0.864 ms).  Rows of up to
// 128 elements: 6 CTAs (42 registers).  With the sign hash on: 4 CTAs (it needs the registers).
constexpr int kStagedCtasL2 = 8, kStagedCtasHbm = 6, kStagedCtasWide = 6, kStagedCtasSign = 4;
constexpr uint64_t kL2SizedBytes = 192ull << 20;  // arrays up to this size count as "of L2 size"

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
// (Storing the starts alone and deriving the payloads in the first sort pass - from q and one bag
// word per id - was measured: it saves 0.1 GB of writes per cfg 4 step and 8 us in the forward, and
// costs 50-60 us in the scatter pass, which is bound by latency and instruction issue, not by bytes.)
struct KeepBlocks {
    uint32_t* keys;
    uint32_t* vals;
    uint64_t bag;
    uint64_t nb;  // number of blocks of the call (read by the debug build's index check only)
};

// Hash phase of one batch of cnt ids starting at position p0 (warp-collective); the t-th id of the
// batch sits at position p0 + t * pstride (pstride = 1 except where a kernel picks the rows of one
// table out of a sample-major one-hot batch; such a kernel keeps no block starts).
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
                                            const KeepBlocks keep = KeepBlocks{nullptr, nullptr, 0, 0},
                                            int64_t pstride = 1) {
    uint64_t* base_s = sm.base[w];
    uint64_t* gbase_s = base_s + kStageIds / 2;
    uint32_t* start_s = sm.start[w];
    for (uint32_t t = lane; t < cnt; t += 32) {
        const uint64_t x = (uint64_t)indices.load(p0 + (int64_t)t * pstride);
        uint64_t xh = x;  // what the location hash sees in place of the id
        if (mp.R > 1) {   // R rows share a block: hashed by floor(x/R), row x starts (x mod R) d in
            xh = x / mp.R;
            sm.piece[w][t] = (uint32_t)(x - xh * mp.R) * mp.d;
        }
        uint64_t tt = tterm, gt = gterm;
        if (!BAGS) {
            const uint32_t e = table_of_bag((uint64_t)(p0 + (int64_t)t * pstride), mp);
            tt = table_term(mp.h, e);
            if (SIGN) gt = table_term(mp.g, e);
        }
        if (!ROBE_CHK(t < (uint32_t)(SIGN ? kStageIds / 2 : kStageIds), ROBE_DBG_SHARED)) continue;
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
        if (ROBE_CHK(c * stride + idl < (uint32_t)kStageEntries, ROBE_DBG_SHARED)) start_s[c * stride + idl] = s;
        wraps |= s > last_fit;
        if (keep.keys != nullptr &&
            ROBE_CHK((uint64_t)p0 * mp.C + t < keep.nb, ROBE_DBG_SORT_POS)) {  // consecutive lanes, consecutive words
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

// ---- lane-hashed kernels (short blocks): every lane hashes the chunks of its own elements ----
//
// With base = (A e + B x + D) mod P and cterm = (C c) mod P, both known mod m as well,
//     h = ((base + cterm) mod P) mod m
//       = (base mod m + cterm mod m + [base + cterm >= P] (m - P mod m)) mod m
// (exact: subtracting P from the sum subtracts P mod m from its residue), i.e. one 64-bit compare,
// two additions and two conditional subtractions per chunk instead of a 128-bit product.  A lane
// owns elements lane, lane + 32, .. of every row; LaneChunks holds, per owned element, the chunk's
// term mod P and mod m and the element's offset inside the chunk.
constexpr int kRowTables = 512;  // tables whose (A e + D) mod P term the kernels keep in shared memory

template <int EPL>
struct LaneChunks {
    uint64_t cterm[EPL];
    uint32_t ct[EPL], off[EPL];
    bool live[EPL];
    uint32_t m, padj;  // padj = m - P mod m

    __device__ __forceinline__ void init(const MapParams& mp, uint32_t lane, uint32_t padj_) {
        m = mp.m;
        padj = padj_;
#pragma unroll
        for (int u = 0; u < EPL; ++u) {
            uint32_t i = lane + 32u * u;
            live[u] = i < mp.d;
            if (!live[u]) i = mp.d - 1;
            uint32_t chk;
            chunk_of(mp, i, chk, off[u]);
            cterm[u] = mulmod_p61_u32(mp.h.C, chk);
            ct[u] = mod_m(cterm[u], mp.m, mp.mu);
        }
    }

    // slot of owned element u of the id whose shared part is (bm = base mod m, thr = P - base);
    // M30: m < 2^30, so that the three residues add up inside 32 bits
    template <bool M30>
    __device__ __forceinline__ uint32_t slot(int u, uint32_t bm, uint64_t thr) const {
        const uint32_t adj = cterm[u] >= thr ? padj : 0u;
        if (M30) {
            uint32_t s = bm + ct[u] + adj;
            if (s >= m) s -= m;
            if (s >= m) s -= m;
            s += off[u];
            if (s >= m) s -= m;
            return s;
        }
        uint64_t s = (uint64_t)bm + ct[u] + adj;
        if (s >= m) s -= m;
        if (s >= m) s -= m;
        s += off[u];
        if (s >= m) s -= m;
        return (uint32_t)s;
    }
};

// (A e + D) mod P of the table of bag `bag`, from the shared-memory table where it reaches
__device__ __forceinline__ uint64_t lane_table_term(const uint64_t* tt_s, const MapParams& mp, uint64_t bag) {
    const uint32_t e = table_of_bag(bag, mp);
    return e < (uint32_t)kRowTables ? tt_s[e] : table_term(mp.h, e);
}

// The shared part of the hash of one id, in the form LaneChunks::slot takes it.
__device__ __forceinline__ void lane_id_base(const MapParams& mp, uint64_t tterm, uint64_t x, uint32_t& bm,
                                             uint64_t& thr) {
    const uint64_t base = addmod_p61(tterm, mulmod_p61_any(mp.h.B, x));
    bm = mod_m(base, mp.m, mp.mu);
    thr = kP61 - base;
}

inline uint32_t lane_padj(const MapParams& mp) { return mp.m - (uint32_t)(kP61 % mp.m); }

// persistent grid of the lane-hashed kernels: a few CTAs of 8 warps per SM, fewer for little work
inline unsigned lane_grid(int64_t units) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    (void)cudaGetLastError();
    int64_t blocks = (units + 7) / 8;
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    return (unsigned)(blocks < 1 ? 1 : blocks);
}

}  // namespace robe
