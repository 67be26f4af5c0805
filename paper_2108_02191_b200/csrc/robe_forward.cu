// Forward lookup kernels (Section 3.2 forward: the embedding is the concatenation of
// ceil(d/Z) blocks M[h(e,x,c) : h(e,x,c)+Z] read circularly; Section 3.1 for the optional
// element-wise sign).  Sum pooling over a bag is sequential in fp32 in bag order.
//
// Two kernels:
//   fwd_direct_kernel  any Z, any d: every lane hashes the chunk of its own element.
//   fwd_staged_kernel  d <= 128: a warp first evaluates the block starts of a whole batch of
//                      ids (one (id, chunk) pair per lane) into a warp-private staging area in
//                      shared memory, then gathers without further integer work, so the hash
//                      cost per id does not depend on how many lanes read a block.
#include "robe_internal.h"
#include "robe_stage.cuh"

namespace robe {

struct FwdArgs {
    MapParams mp;
    const void* array;
    IdList indices;
    const int64_t* offsets;
    float* out;
    int64_t nbags;
    int64_t nnz;
    const int32_t* status;
    uint32_t* keep_keys;  // block starts and payloads kept for the backward, or nullptr
    uint32_t* keep_vals;
};

// Kept block starts, pooled input: id positions before the first bag or after the last one (offsets
// that break the contract offsets[0] = 0, offsets[nbags] = nnz) belong to no warp of the forward
// kernel; they get block start 0 and bag 0 here, so that the backward reads nothing stale.  With
// well-formed offsets there is nothing to do.  (A kernel of its own: inside the gather kernel these
// two loops cost registers that its occupancy has no room for.)
__global__ void __launch_bounds__(256) keep_gaps_kernel(FwdArgs a) {
    int64_t lo, hi, lo_last, hi_last;
    bag_range(a.offsets, a.nnz, 0, lo, hi);
    bag_range(a.offsets, a.nnz, a.nbags - 1, lo_last, hi_last);
    const int64_t C = (int64_t)a.mp.C;
    const int64_t step = (int64_t)gridDim.x * 256, t0 = (int64_t)blockIdx.x * 256 + threadIdx.x;
    for (int64_t q = t0; q < lo * C; q += step) a.keep_keys[q] = a.keep_vals[q] = 0;
    for (int64_t q = hi_last * C + t0; q < a.nnz * C; q += step) a.keep_keys[q] = a.keep_vals[q] = 0;
}

template <int DT, bool SIGN>
__global__ void __launch_bounds__(256) fwd_direct_kernel(FwdArgs a) {
    const int64_t k = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    if (k >= a.nbags) return;
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    int64_t lo, hi;
    bag_range(a.offsets, a.nnz, k, lo, hi);
    const uint32_t e = table_of_bag((uint64_t)k, mp);
    for (uint32_t i = lane; i < mp.d; i += 32) {
        uint32_t c, o;
        chunk_of(mp, i, c, o);
        float acc = 0.0f;
        for (int64_t p = lo; p < hi; ++p) {
            const uint64_t x = (uint64_t)a.indices.load(p);
            uint32_t j = id_block_start(mp, e, x, c) + o;  // < m + d <= 2^32
            if (j >= mp.m) j -= mp.m;
            float v = 0.0f;
            if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) v = load_elem<DT>(a.array, j);
            if (SIGN) v = sign_of(mp, hash_base(mp.g, e, x), i) * v;
            acc = (p == lo) ? v : acc + v;
        }
        __stcs(a.out + k * mp.d + i, acc);
    }
}

// Staged kernel (any Z, d <= 128).  One warp serves one bag (pooled) or one group of
// consecutive rows (one-hot).  It works in two phases per batch of ids, with a warp-private
// staging area in shared memory and only __syncwarp between the phases:
//   hash phase    lanes take the ids of the batch, one id per lane, and store (A e + B x + D)
//                 mod P; then lanes take the (id, chunk) pairs of the batch, 32 at a time, and
//                 store the block starts h(e,x,c);
//   gather phase  lane l owns elements l, l+32, ...; it reads its block start from shared
//                 memory, adds its in-block offset (wrapping only if some block of the batch
//                 reaches the array end), and loads; the loads of U ids are issued before the
//                 first add.
// EPL = elements per lane (d <= 32*EPL).  FULLD: d == 32*EPL (no lane is past the row end).

// Loads of one group of n <= U ids of the staged batch, ids g0 .. g0+n-1.  WRAP: slot numbers
// are wrapped at the array end; TAIL: n may be below U.
template <int EPL, int DT, bool SIGN, int U, bool WRAP, bool TAIL>
__device__ __forceinline__ void gather_group(const FwdArgs& a, const uint32_t* const (&col)[EPL],
                                             const uint32_t (&off)[EPL], const bool (&live)[EPL],
                                             const uint64_t* gbase_s, uint32_t g0, uint32_t n,
                                             uint32_t lane, float (&v)[U][EPL]) {
    const MapParams& mp = a.mp;
#pragma unroll
    for (int gg = 0; gg < U; ++gg) {
        const bool on = !TAIL || (uint32_t)gg < n;  // warp-uniform
#pragma unroll
        for (int u = 0; u < EPL; ++u) {
            float val = 0.0f;
            if (on && live[u]) {
                uint32_t j = col[u][g0 + gg] + off[u];  // < m + d <= 2^32
                if (WRAP && j >= mp.m) j -= mp.m;
                if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) val = gather_elem<DT>(a.array, j);
                if (SIGN) val = sign_of(mp, gbase_s[g0 + gg], lane + 32u * u) * val;
            }
            v[gg][u] = val;
        }
    }
}

// Gather phase of one staged batch: pooled rows are added to acc in id order, one-hot rows are
// stored straight to the output.
template <int EPL, int DT, bool SIGN, bool BAGS, int U, bool WRAP>
__device__ __forceinline__ void gather_batch(const FwdArgs& a, const uint32_t* const (&col)[EPL],
                                             const uint32_t (&off)[EPL], const bool (&live)[EPL],
                                             const uint64_t* gbase_s, uint32_t cnt, int64_t p0,
                                             uint32_t lane, float (&acc)[EPL]) {
    const MapParams& mp = a.mp;
    uint32_t g0 = 0;
    for (; g0 + U <= cnt; g0 += U) {
        float v[U][EPL];
        gather_group<EPL, DT, SIGN, U, WRAP, false>(a, col, off, live, gbase_s, g0, U, lane, v);
        if (BAGS) {
#pragma unroll
            for (int gg = 0; gg < U; ++gg)
#pragma unroll
                for (int u = 0; u < EPL; ++u) acc[u] = acc[u] + v[gg][u];
        } else {
#pragma unroll
            for (int gg = 0; gg < U; ++gg) {
                float* orow = a.out + (p0 + g0 + gg) * (int64_t)mp.d;
#pragma unroll
                for (int u = 0; u < EPL; ++u)
                    if (live[u]) __stcs(orow + lane + 32u * u, v[gg][u]);
            }
        }
    }
    if (g0 < cnt) {
        const uint32_t n = cnt - g0;
        float v[U][EPL];
        gather_group<EPL, DT, SIGN, U, WRAP, true>(a, col, off, live, gbase_s, g0, n, lane, v);
        if (BAGS) {
#pragma unroll
            for (int gg = 0; gg < U; ++gg)
                if ((uint32_t)gg < n) {
#pragma unroll
                    for (int u = 0; u < EPL; ++u) acc[u] = acc[u] + v[gg][u];
                }
        } else {
#pragma unroll
            for (int gg = 0; gg < U; ++gg)
                if ((uint32_t)gg < n) {
                    float* orow = a.out + (p0 + g0 + gg) * (int64_t)mp.d;
#pragma unroll
                    for (int u = 0; u < EPL; ++u)
                        if (live[u]) __stcs(orow + lane + 32u * u, v[gg][u]);
                }
        }
    }
}

template <int EPL, int DT, bool SIGN, bool BAGS, bool FULLD, int MINB, int U>
__global__ void __launch_bounds__(256, MINB)
fwd_staged_kernel(FwdArgs a, uint32_t ids_per_batch, uint32_t cmagic) {
    __shared__ StageSmem sm;
    const MapParams& mp = a.mp;
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t warp = (int64_t)blockIdx.x * 8 + w;

    stage_init(sm, mp);
    if (a.status != nullptr && *a.status != 0) return;

    int64_t lo, hi;
    uint64_t tterm = 0, gterm = 0;
    if (BAGS) {
        if (warp >= a.nbags) return;
        bag_range(a.offsets, a.nnz, warp, lo, hi);
        const uint32_t e_bag = table_of_bag((uint64_t)warp, mp);
        tterm = table_term(mp.h, e_bag);
        if (SIGN) gterm = table_term(mp.g, e_bag);
    } else {
        lo = warp * (int64_t)ids_per_batch;  // this warp serves rows [lo, lo + ids_per_batch)
        if (lo >= a.nbags) return;
        hi = lo + ids_per_batch < a.nbags ? lo + ids_per_batch : a.nbags;
    }

    // per-lane constants of the gather: element i = lane + 32u, its in-block offset, and the
    // column of the staging area that holds the starts of its chunk
    uint32_t off[EPL];
    const uint32_t* col[EPL];
    bool live[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) {
        uint32_t i = lane + 32u * u;
        live[u] = FULLD || i < mp.d;
        if (!live[u]) i = mp.d - 1;
        uint32_t chk;
        chunk_of(mp, i, chk, off[u]);
        col[u] = sm.start[w] + chk * ids_per_batch;
    }
    const uint64_t* gbase_s = sm.base[w] + kStageIds / 2;  // sign-hash bases (sign on only)

    // -0 + v == v for every v (also v = -0): starting from -0 makes the first term initialise
    // the sum exactly as the definition says
    float acc[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) acc[u] = -0.0f;

    for (int64_t p0 = lo; p0 < hi; p0 += ids_per_batch) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)ids_per_batch ? (hi - p0)
                                                                            : (int64_t)ids_per_batch);
        const bool wraps = stage_batch<SIGN, BAGS>(sm, mp, a.indices, p0, cnt, ids_per_batch, tterm,
                                                   gterm, cmagic, w, lane,
                                                   KeepBlocks{a.keep_keys, a.keep_vals, (uint64_t)warp, (uint64_t)a.nnz * mp.C});
        if (wraps)
            gather_batch<EPL, DT, SIGN, BAGS, U, true>(a, col, off, live, gbase_s, cnt, p0, lane, acc);
        else
            gather_batch<EPL, DT, SIGN, BAGS, U, false>(a, col, off, live, gbase_s, cnt, p0, lane, acc);
        __syncwarp();  // the staging area is rewritten by the next batch
    }
    if (BAGS) {
        float* orow = a.out + warp * (int64_t)mp.d;
        const bool empty = hi <= lo;
#pragma unroll
        for (int u = 0; u < EPL; ++u)
            if (live[u]) __stcs(orow + lane + 32u * u, empty ? 0.0f : acc[u]);
    }
}

// Vector kernel: fp32 array, d, Z and m multiples of four, d <= 128.  The staging and the hash
// phase are those of the staged kernel; the gather reads 16 bytes per load.  A block starts at
// an arbitrary element, so its elements 4k .. 4k+3 (output vector k of the row) lie in the two
// ALIGNED 16-byte pieces around them: the lane loads both (only the first when the block start is
// itself a multiple of four) and shifts the eight values by (start mod 4) in registers.  m is a
// multiple of four, so an aligned piece never straddles the end of the array and the wrap-around
// is a subtraction on the piece's slot number.  d/4 lanes serve one id; with d <= 64 the warp
// serves 32 / (d/4) ids per load instruction, and the pooled sum still adds the ids in bag order:
// the lanes of the first id hold the sum and fetch the other ids' vectors by shuffle, in order.
__device__ __forceinline__ float4 ldg_f4_64B(const float* p) {
    float4 v;
    asm("ld.global.nc.L2::64B.v4.f32 {%0, %1, %2, %3}, [%4];"
        : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
        : "l"(p));
    return v;
}

// elements r .. r+3 of the eight values (lo, hi), r = 0 .. 3
__device__ __forceinline__ float4 realign4(const float4 lo, const float4 hi, uint32_t r) {
    float e0 = lo.x, e1 = lo.y, e2 = lo.z, e3 = lo.w, e4 = hi.x, e5 = hi.y, e6 = hi.z;
    if (r & 2u) { e0 = e2; e1 = e3; e2 = e4; e3 = e5; e4 = e6; }
    if (r & 1u) { e0 = e1; e1 = e2; e2 = e3; e3 = e4; }
    return make_float4(e0, e1, e2, e3);
}

template <bool BAGS, bool WRAP, int U>
__device__ __forceinline__ void vec_gather_batch(const FwdArgs& a, const uint32_t* col, uint32_t o,
                                                 uint32_t cnt, int64_t p0, uint32_t lpi, uint32_t ipi,
                                                 uint32_t grp, uint32_t k, bool lane_on, float4& acc) {
    const MapParams& mp = a.mp;
    const float* array = (const float*)a.array;
    for (uint32_t g0 = 0; g0 < cnt; g0 += ipi * U) {
        float4 v[U];
#pragma unroll
        for (int gg = 0; gg < U; ++gg) {
            const uint32_t t = g0 + gg * ipi + grp;
            v[gg] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (lane_on && t < cnt) {
                const uint32_t pos = col[t] + o;  // first slot of the vector, < m + d <= 2^32
                const uint32_t r = pos & 3u;
                uint32_t a0 = pos & ~3u;
                if (WRAP && a0 >= mp.m) a0 -= mp.m;
                if (!ROBE_CHK(a0 < mp.m && (r == 0 || WRAP || a0 + 4u < mp.m), ROBE_DBG_ARRAY_SLOT)) continue;
                const float4 lo = ldg_f4_64B(array + a0);
                float4 hi = lo;
                if (r != 0) {
                    uint32_t a1 = a0 + 4u;
                    if (WRAP && a1 >= mp.m) a1 -= mp.m;
                    hi = ldg_f4_64B(array + a1);
                }
                v[gg] = realign4(lo, hi, r);
            }
        }
        if (BAGS) {
#pragma unroll
            for (int gg = 0; gg < U; ++gg) {
                for (uint32_t gs = 0; gs < ipi; ++gs) {
                    if (g0 + gg * ipi + gs >= cnt) break;  // warp-uniform
                    float4 x = v[gg];
                    if (gs != 0) {  // the vector of a later id of this load: from its lanes
                        const int src = (int)(k + gs * lpi);
                        x.x = __shfl_sync(0xFFFFFFFFu, v[gg].x, src);
                        x.y = __shfl_sync(0xFFFFFFFFu, v[gg].y, src);
                        x.z = __shfl_sync(0xFFFFFFFFu, v[gg].z, src);
                        x.w = __shfl_sync(0xFFFFFFFFu, v[gg].w, src);
                    }
                    acc.x = acc.x + x.x;
                    acc.y = acc.y + x.y;
                    acc.z = acc.z + x.z;
                    acc.w = acc.w + x.w;
                }
            }
        } else {
#pragma unroll
            for (int gg = 0; gg < U; ++gg) {
                const uint32_t t = g0 + gg * ipi + grp;
                if (lane_on && t < cnt)
                    __stcs(reinterpret_cast<float4*>(a.out + (p0 + t) * (int64_t)mp.d) + k, v[gg]);
            }
        }
    }
}

template <bool BAGS, int U>
__global__ void __launch_bounds__(256, 5)
fwd_vec_kernel(FwdArgs a, uint32_t ids_per_batch, uint32_t cmagic) {
    __shared__ StageSmem sm;
    const MapParams& mp = a.mp;
    const uint32_t lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t warp = (int64_t)blockIdx.x * 8 + w;

    stage_init(sm, mp);
    if (a.status != nullptr && *a.status != 0) return;

    int64_t lo, hi;
    uint64_t tterm = 0;
    if (BAGS) {
        if (warp >= a.nbags) return;
        bag_range(a.offsets, a.nnz, warp, lo, hi);
        tterm = table_term(mp.h, table_of_bag((uint64_t)warp, mp));
    } else {
        lo = warp * (int64_t)ids_per_batch;
        if (lo >= a.nbags) return;
        hi = lo + ids_per_batch < a.nbags ? lo + ids_per_batch : a.nbags;
    }

    const uint32_t lpi = mp.d >> 2;   // lanes per id = output vectors per row
    const uint32_t ipi = 32u / lpi;   // ids per load instruction
    const uint32_t grp = lane / lpi;  // which of them this lane reads
    const uint32_t k = lane - grp * lpi;
    const bool lane_on = grp < ipi;
    uint32_t chk, o;
    chunk_of(mp, 4u * k, chk, o);
    const uint32_t* col = sm.start[w] + chk * ids_per_batch;

    float4 acc = make_float4(-0.0f, -0.0f, -0.0f, -0.0f);  // -0 + v == v: the first term initialises
    for (int64_t p0 = lo; p0 < hi; p0 += ids_per_batch) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)ids_per_batch ? (hi - p0)
                                                                            : (int64_t)ids_per_batch);
        const bool wraps = stage_batch<false, BAGS>(sm, mp, a.indices, p0, cnt, ids_per_batch, tterm, 0,
                                                    cmagic, w, lane,
                                                    KeepBlocks{a.keep_keys, a.keep_vals, (uint64_t)warp, (uint64_t)a.nnz * mp.C});
        if (wraps)
            vec_gather_batch<BAGS, true, U>(a, col, o, cnt, p0, lpi, ipi, grp, k, lane_on, acc);
        else
            vec_gather_batch<BAGS, false, U>(a, col, o, cnt, p0, lpi, ipi, grp, k, lane_on, acc);
        __syncwarp();
    }
    if (BAGS && grp == 0) {
        const bool empty = hi <= lo;
        if (empty) acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        __stcs(reinterpret_cast<float4*>(a.out + warp * (int64_t)mp.d) + k, acc);
    }
}

// what the vector kernel asks of a call
static bool vec_kernel_ok(const Problem& pb, const float* out) {
    const MapParams& mp = pb.mp;
    return pb.dtype == 0 && pb.sign == 0 && mp.d <= 128 && mp.d % 4 == 0 && mp.Z % 4 == 0 && mp.m % 4 == 0 &&
           ((uintptr_t)out & 15u) == 0 && ((uintptr_t)pb.array & 15u) == 0;
}

static void launch_vec(const FwdArgs& a, bool bags, cudaStream_t st) {
    const uint32_t ipb = staged_ids_per_batch(a.mp, bags, false);
    const uint32_t cmagic = chunk_magic(a.mp);
    const int64_t warps = bags ? a.nbags : (a.nbags + ipb - 1) / ipb;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags) fwd_vec_kernel<true, 4><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
    else fwd_vec_kernel<false, 4><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
}

// Ids whose loads are in flight together (U) and resident CTAs per SM the register budget is set
// for (MINB, see kStagedCtas*).  Measured on B200: the time of the HBM-resident gather does not move
// between 4 and 16 ids in flight - the random 64-byte requests themselves are the limit.

template <int EPL, int DT, bool SIGN, bool FULLD, int MINB>
static void launch_staged_minb(const FwdArgs& a, bool bags, cudaStream_t st) {
    constexpr int UB = (EPL == 4) ? 2 : 4;
    constexpr int UO = (EPL == 4) ? 2 : 4;
    const uint32_t ipb = staged_ids_per_batch(a.mp, bags, SIGN);
    const uint32_t cmagic = chunk_magic(a.mp);
    const int64_t warps = bags ? a.nbags : (a.nbags + ipb - 1) / ipb;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags)
        fwd_staged_kernel<EPL, DT, SIGN, true, FULLD, MINB, UB><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
    else
        fwd_staged_kernel<EPL, DT, SIGN, false, FULLD, MINB, UO><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
}

template <int EPL, int DT, bool SIGN, bool FULLD>
static void launch_staged(const FwdArgs& a, bool bags, cudaStream_t st) {
    const bool l2_sized = (uint64_t)a.mp.m * (DT == 0 ? 4u : 2u) <= kL2SizedBytes;
    if constexpr (SIGN) launch_staged_minb<EPL, DT, SIGN, FULLD, kStagedCtasSign>(a, bags, st);
    else if constexpr (EPL == 4) launch_staged_minb<EPL, DT, SIGN, FULLD, kStagedCtasWide>(a, bags, st);
    else if (l2_sized) launch_staged_minb<EPL, DT, SIGN, FULLD, kStagedCtasL2>(a, bags, st);
    else launch_staged_minb<EPL, DT, SIGN, FULLD, kStagedCtasHbm>(a, bags, st);
}

template <int EPL, int DT>
static void launch_staged_flags(const FwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    const bool fulld = a.mp.d == 32u * EPL;
    if (sign) {  // the sign hash is off in every timed configuration: one generic variant
        launch_staged<EPL, DT, true, false>(a, bags, st);
    } else if (fulld) {
        launch_staged<EPL, DT, false, true>(a, bags, st);
    } else {
        launch_staged<EPL, DT, false, false>(a, bags, st);
    }
}

template <int DT>
static void launch_staged_epl(const FwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    if (a.mp.d <= 32)
        launch_staged_flags<1, DT>(a, bags, sign, st);
    else if (a.mp.d <= 64)
        launch_staged_flags<2, DT>(a, bags, sign, st);
    else
        launch_staged_flags<4, DT>(a, bags, sign, st);
}

// Lane-hashed kernel for short blocks (Z <= 2 by default; any Z <= d whose lanes can afford to hash
// their own chunks).  With d/Z chunks per id as numerous as the elements themselves, staging the
// block starts in shared memory buys nothing: every lane owns elements lane, lane+32, .. of every
// row and hashes exactly the chunks of those elements, in registers (LaneChunks).  Per id the shared
// part of the hash is evaluated once, by one lane, 32 ids at a time, and handed round by shuffle.
// Warps are persistent: the per-lane chunk constants are set up once and serve every row the
// warp takes (rows in groups of 32, or one bag after another).
template <int EPL, int DT, bool BAGS, bool M30, int U>
__global__ void __launch_bounds__(256, 4)
fwd_lanehash_kernel(FwdArgs a, uint32_t padj) {
    __shared__ uint64_t tt_s[kRowTables];
    const MapParams& mp = a.mp;
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t e = threadIdx.x; e < mp.T && e < (uint32_t)kRowTables; e += 256) tt_s[e] = table_term(mp.h, e);
    __syncthreads();
    if (a.status != nullptr && *a.status != 0) return;

    LaneChunks<EPL> lc;
    lc.init(mp, lane, padj);

    // the loads of U ids (the owned elements of each) are issued together
    auto gather_ids = [&](uint32_t bm, uint64_t thr, uint32_t g0, uint32_t n, float (&v)[U][EPL]) {
#pragma unroll
        for (int gg = 0; gg < U; ++gg) {
            const int src = (int)(g0 + gg < n ? g0 + gg : n - 1);
            const uint32_t bm_g = __shfl_sync(0xFFFFFFFFu, bm, src);
            const uint64_t thr_g = __shfl_sync(0xFFFFFFFFu, thr, src);
#pragma unroll
            for (int u = 0; u < EPL; ++u) {
                v[gg][u] = 0.0f;
                if (lc.live[u]) {
                    const uint32_t j = lc.template slot<M30>(u, bm_g, thr_g);
                    if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) v[gg][u] = gather_elem<DT>(a.array, j);
                }
            }
        }
    };

    const int64_t nwarps = (int64_t)gridDim.x * 8;
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (!BAGS) {
        for (int64_t r0 = gw * 32; r0 < a.nbags; r0 += nwarps * 32) {
            const int64_t row = r0 + lane;
            uint32_t bm = 0;
            uint64_t thr = kP61;
            if (row < a.nbags)
                lane_id_base(mp, lane_table_term(tt_s, mp, (uint64_t)row), (uint64_t)a.indices.load(row), bm, thr);
            const uint32_t n = (uint32_t)(a.nbags - r0 < 32 ? a.nbags - r0 : 32);
            for (uint32_t g0 = 0; g0 < n; g0 += U) {
                float v[U][EPL];
                gather_ids(bm, thr, g0, n, v);
#pragma unroll
                for (int gg = 0; gg < U; ++gg) {
                    if (g0 + gg < n) {
                        float* orow = a.out + (r0 + g0 + gg) * (int64_t)mp.d;
#pragma unroll
                        for (int u = 0; u < EPL; ++u)
                            if (lc.live[u]) __stcs(orow + lane + 32u * u, v[gg][u]);
                    }
                }
            }
        }
    } else {
        for (int64_t bag = gw; bag < a.nbags; bag += nwarps) {
            int64_t lo, hi;
            bag_range(a.offsets, a.nnz, bag, lo, hi);
            const uint64_t tterm = lane_table_term(tt_s, mp, (uint64_t)bag);
            float acc[EPL];
#pragma unroll
            for (int u = 0; u < EPL; ++u) acc[u] = -0.0f;  // -0 + v == v: the first term initialises
            for (int64_t p0 = lo; p0 < hi; p0 += 32) {
                uint32_t bm = 0;
                uint64_t thr = kP61;
                if (p0 + lane < hi) lane_id_base(mp, tterm, (uint64_t)a.indices.load(p0 + lane), bm, thr);
                const uint32_t n = (uint32_t)(hi - p0 < 32 ? hi - p0 : 32);
                for (uint32_t g0 = 0; g0 < n; g0 += U) {
                    float v[U][EPL];
                    gather_ids(bm, thr, g0, n, v);
#pragma unroll
                    for (int gg = 0; gg < U; ++gg)
                        if (g0 + gg < n) {
#pragma unroll
                            for (int u = 0; u < EPL; ++u) acc[u] = acc[u] + v[gg][u];
                        }
                }
            }
            float* orow = a.out + bag * (int64_t)mp.d;
#pragma unroll
            for (int u = 0; u < EPL; ++u)
                if (lc.live[u]) __stcs(orow + lane + 32u * u, hi <= lo ? 0.0f : acc[u]);
        }
    }
}

// what the lane-hashed kernel asks of a call: plain blocks (no rows clubbed into one), sign off
static bool lanehash_ok(const Problem& pb) { return pb.sign == 0 && pb.mp.R == 1 && pb.mp.d <= 128; }

template <int EPL, int DT>
static void launch_lanehash_m(const FwdArgs& a, bool bags, cudaStream_t st) {
    const unsigned blocks = lane_grid(bags ? a.nbags : (a.nbags + 31) / 32);
    const uint32_t padj = lane_padj(a.mp);
    const bool m30 = a.mp.m < (1u << 30);
    constexpr int U = EPL == 4 ? 2 : 4;
    if (bags) {
        if (m30) fwd_lanehash_kernel<EPL, DT, true, true, U><<<blocks, 256, 0, st>>>(a, padj);
        else fwd_lanehash_kernel<EPL, DT, true, false, U><<<blocks, 256, 0, st>>>(a, padj);
    } else {
        if (m30) fwd_lanehash_kernel<EPL, DT, false, true, U><<<blocks, 256, 0, st>>>(a, padj);
        else fwd_lanehash_kernel<EPL, DT, false, false, U><<<blocks, 256, 0, st>>>(a, padj);
    }
}

template <int DT>
static void launch_lanehash(const FwdArgs& a, bool bags, cudaStream_t st) {
    if (a.mp.d <= 32) launch_lanehash_m<1, DT>(a, bags, st);
    else if (a.mp.d <= 64) launch_lanehash_m<2, DT>(a, bags, st);
    else launch_lanehash_m<4, DT>(a, bags, st);
}

cudaError_t launch_forward(const Problem& pb, float* out, int variant, cudaStream_t st,
                           uint32_t* keep_keys, uint32_t* keep_vals, bool* kept) {
    if (kept != nullptr) *kept = false;
    if (pb.nbags == 0) return cudaSuccess;
    FwdArgs a{pb.mp, pb.array, pb.indices, pb.offsets, out, pb.nbags, pb.nnz, pb.status, keep_keys,
              keep_vals};
    const bool bags = pb.offsets != nullptr;
    const bool warp_ok = pb.mp.d <= 128;
    if (variant == 2 && !warp_ok) return cudaErrorInvalidValue;
    if (variant == 3) {  // the kernel with 16-byte loads
        if (!vec_kernel_ok(pb, out)) return cudaErrorInvalidValue;
        if (kept != nullptr) *kept = keep_keys != nullptr;
        if (bags && keep_keys != nullptr) keep_gaps_kernel<<<8, 256, 0, st>>>(a);
        launch_vec(a, bags, st);
        return cudaGetLastError();
    }
    // Short blocks: every lane hashes its own chunks (keeps nothing for a sort-based backward).
    // Automatic for arrays of L2 size, where the staged kernel is bound by its instruction count
    // (measured on B200, Z = 1 / 2: 1 MB array 2.27 -> 1.72 ms / 1.72 -> 1.00 ms, 100 MB 3.59 -> 3.40 /
    // 2.14 -> 2.09); on a 10 GB array the staged kernel's higher occupancy keeps more DRAM requests
    // in flight and stays ahead (9.5 vs 10.2 ms), so it keeps those.
    const bool l2_sized = (uint64_t)pb.mp.m * (pb.dtype == 0 ? 4u : 2u) <= kL2SizedBytes;
    if (variant == 4 || (variant == 0 && pb.mp.Z <= 2 && l2_sized && lanehash_ok(pb) && keep_keys == nullptr)) {
        if (!lanehash_ok(pb)) return cudaErrorInvalidValue;
        if (pb.dtype == 0) launch_lanehash<0>(a, bags, st);
        else launch_lanehash<1>(a, bags, st);
        return cudaGetLastError();
    }
    const bool use_warp = variant == 2 || (variant == 0 && warp_ok);
    if (use_warp) {
        if (kept != nullptr) *kept = keep_keys != nullptr;  // (the direct kernel keeps nothing)
        if (bags && keep_keys != nullptr) keep_gaps_kernel<<<8, 256, 0, st>>>(a);
        if (pb.dtype == 0) launch_staged_epl<0>(a, bags, pb.sign != 0, st);
        else launch_staged_epl<1>(a, bags, pb.sign != 0, st);
    } else {
        const unsigned blocks = (unsigned)((pb.nbags + 7) / 8);
        if (pb.dtype == 0) {
            if (pb.sign) fwd_direct_kernel<0, true><<<blocks, 256, 0, st>>>(a);
            else fwd_direct_kernel<0, false><<<blocks, 256, 0, st>>>(a);
        } else {
            if (pb.sign) fwd_direct_kernel<1, true><<<blocks, 256, 0, st>>>(a);
            else fwd_direct_kernel<1, false><<<blocks, 256, 0, st>>>(a);
        }
    }
    return cudaGetLastError();
}

}  // namespace robe
