// Atomic backward (Section 3.1 backward equation): every element of the output gradient
// is added, with its sign, into the array slot it was read from in the forward pass:
//   delta[idx(e,x,i)] += g(e,x,i) * grad_out[bag, i]      for every id x of every bag.
// `target` is either a dense fp32 gradient array (scale = 1) or the parameter array
// itself (scale = -lr: the SGD step fused into the scatter).  fp32 reductions in global
// memory (red.global.add.f32); the order of the additions is not fixed.
//
// Same two shapes as the forward: a direct kernel for any (Z, d) and a staged kernel
// (d <= 128) that evaluates the block starts of a batch of ids into shared memory first.
#include "robe_internal.h"
#include "robe_stage.cuh"

namespace robe {

struct BwdArgs {
    MapParams mp;
    const float* grad_out;
    IdList indices;
    const int64_t* offsets;
    float* target;
    float scale;
    int64_t nbags;
    int64_t nnz;
    const int32_t* status;
    int l2_keep;  // the reductions carry the L2 "keep" policy
};


template <bool SIGN>
__global__ void __launch_bounds__(256) bwd_atomic_direct_kernel(BwdArgs a) {
    const int64_t k = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    if (k >= a.nbags) return;
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    int64_t lo, hi;
    bag_range(a.offsets, a.nnz, k, lo, hi);
    const uint32_t e = table_of_bag((uint64_t)k, mp);
    const uint64_t pol = l2_keep_policy(a.l2_keep != 0);
    for (uint32_t i = lane; i < mp.d; i += 32) {
        uint32_t c, o;
        chunk_of(mp, i, c, o);
        const float gv = __ldcs(a.grad_out + k * mp.d + i) * a.scale;
        for (int64_t p = lo; p < hi; ++p) {
            const uint64_t x = (uint64_t)a.indices.load(p);
            uint32_t j = id_block_start(mp, e, x, c) + o;
            if (j >= mp.m) j -= mp.m;
            float t = gv;
            if (SIGN) t = sign_of(mp, hash_base(mp.g, e, x), i) * t;
            if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) red_add(a.target + j, t, pol);
        }
    }
}

// Staged kernel (any Z, d <= 128): same two phases as the staged forward kernel - the warp
// first evaluates the block starts of a batch of ids into its shared-memory staging area, then
// every lane issues one fp32 reduction per (id, element) it owns.  The gradient row of a bag is
// read once and kept in registers for all ids of the bag.
//
// MERGE (one-hot input, sign off): a warp takes up to 64 rows of ONE table - every T-th row of a
// sample-major batch, consecutive rows of a table-major one; neighbouring warps take different
// tables, so that the reductions of a hot id do not all arrive at once - and groups the rows whose
// hash base (A e + B x + D) mod P is the same, i.e. the repeats of an id (a Zipf batch puts 8-16 %
// of a table's lookups on its top id): such rows address the same slots in every chunk.  The first
// row of a group sums the gradient rows of the whole group in registers and issues ONE reduction
// per element where the plain kernel issues one per occurrence.
template <int EPL, bool SIGN, bool BAGS, bool FULLD, int MINB, bool MERGE = false>
__global__ void __launch_bounds__(256, MINB)
bwd_atomic_staged_kernel(BwdArgs a, uint32_t ids_per_batch, uint32_t cmagic) {
    __shared__ StageSmem sm;
    __shared__ uint32_t dup_s[MERGE ? 8 : 1][kStageIds];
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
    } else if (!MERGE) {
        lo = warp * (int64_t)ids_per_batch;
        if (lo >= a.nbags) return;
        hi = lo + ids_per_batch < a.nbags ? lo + ids_per_batch : a.nbags;
    }
    // MERGE: warp -> (table e, ids_per_batch consecutive samples from n0 on); the t-th row of the
    // batch is bag number p0 + t * pstride
    int64_t pstride = 1;
    if (MERGE) {
        const int64_t batch = a.nbags / mp.T;
        const uint32_t e = (uint32_t)(warp % mp.T);
        const int64_t n0 = (warp / mp.T) * (int64_t)ids_per_batch;
        if (n0 >= batch) return;
        const int64_t cnt = n0 + ids_per_batch < batch ? ids_per_batch : batch - n0;
        if (mp.B != 0) {  // table-major: the rows of table e lie side by side
            lo = (int64_t)e * batch + n0;
            hi = lo + cnt;
        } else {
            pstride = mp.T;
            lo = n0 * mp.T + e;
            hi = lo + cnt * pstride;  // (one batch: the loop below runs once)
        }
    }

    uint32_t off[EPL], chk[EPL];
    bool live[EPL];
    float gv[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) {
        uint32_t i = lane + 32u * u;
        live[u] = FULLD || i < mp.d;
        if (!live[u]) i = mp.d - 1;
        chunk_of(mp, i, chk[u], off[u]);
        gv[u] = 0.0f;
        if (BAGS && live[u]) gv[u] = __ldcs(a.grad_out + warp * (int64_t)mp.d + i) * a.scale;
    }
    const uint32_t* start_s = sm.start[w];
    const uint64_t* gbase_s = sm.base[w] + kStageIds / 2;
    const uint64_t pol = l2_keep_policy(a.l2_keep != 0);

    for (int64_t p0 = lo; p0 < hi; p0 += (int64_t)ids_per_batch * pstride) {
        const int64_t left = (hi - p0 + pstride - 1) / pstride;
        const uint32_t cnt = (uint32_t)(left < (int64_t)ids_per_batch ? left : (int64_t)ids_per_batch);
        stage_batch<SIGN, BAGS>(sm, mp, a.indices, p0, cnt, ids_per_batch, tterm, gterm, cmagic, w, lane,
                                KeepBlocks{nullptr, nullptr, 0, 0}, pstride);
        if (MERGE) {
            for (uint32_t t0 = 0; t0 < cnt; t0 += 32) {
                const uint32_t t = t0 + lane;
                const uint32_t part = __ballot_sync(0xFFFFFFFFu, t < cnt);
                if (t < cnt) {
                    // (rows clubbed into one block share a hash base without sharing slots: no merge)
                    const uint32_t same = mp.R > 1 ? (1u << lane) : __match_any_sync(part, sm.base[w][t]);
                    dup_s[w][t] = ((same & ((1u << lane) - 1u)) == 0) ? same : 0u;
                }
            }
            __syncwarp();
        }
        for (uint32_t g = 0; g < cnt; ++g) {
            if (MERGE) {
                const uint32_t mk = dup_s[w][g];  // warp-uniform
                if (mk == 0) continue;            // an earlier row of the batch adds this one's gradient too
#pragma unroll
                for (int u = 0; u < EPL; ++u) gv[u] = 0.0f;
                for (uint32_t rest = mk; rest != 0; rest &= rest - 1) {
                    const int64_t row = p0 + (int64_t)((g & ~31u) + (uint32_t)(__ffs((int)rest) - 1)) * pstride;
#pragma unroll
                    for (int u = 0; u < EPL; ++u)
                        if (live[u]) gv[u] += __ldcs(a.grad_out + row * (int64_t)mp.d + lane + 32u * u);
                }
#pragma unroll
                for (int u = 0; u < EPL; ++u) gv[u] *= a.scale;
            } else if (!BAGS) {
#pragma unroll
                for (int u = 0; u < EPL; ++u)
                    if (live[u])
                        gv[u] = __ldcs(a.grad_out + (p0 + g) * (int64_t)mp.d + lane + 32u * u) * a.scale;
            }
#pragma unroll
            for (int u = 0; u < EPL; ++u) {
                uint32_t j = start_s[chk[u] * ids_per_batch + g] + off[u];
                if (j >= mp.m) j -= mp.m;
                if (live[u] && ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) {
                    float t = gv[u];
                    if (SIGN) t = sign_of(mp, gbase_s[g], lane + 32u * u) * t;
                    red_add(a.target + j, t, pol);
                }
            }
        }
        __syncwarp();
    }
}

// Vector kernel: d, Z and m multiples of four, d <= 128, sign off.  d/4 lanes serve one id, lane k
// owning the four gradient elements 4k .. 4k+3 of the row (one 16-byte load per bag, or per row).
// Their slots start at an arbitrary element, so they straddle two ALIGNED groups of four slots;
// the lane therefore adds into the upper of the two, with ONE 16-byte reduction
// (red.global.add.v4.f32), its own last elements followed by the first elements of the row's next
// vector - shifted into place in registers.  What is left over at the two ends of a block goes out
// as at most three scalar reductions by the block's first and last lane.  A block start that is a
// multiple of four needs no shift.
//
// MERGE (one-hot input): ids of a staged batch with the same hash base (A e + B x + D) mod P - the
// same id of the same table, as a Zipf batch repeats its hot ids - address the same slots in every
// chunk.  __match_any_sync groups them, the group's first id sums the gradient rows of all of them
// in registers and issues one reduction where the plain kernel issues one per occurrence.
__device__ __forceinline__ void red_add_v4(float* p, const float4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 :
                 : "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}

// elements r .. r+3 of the eight values (lo, hi), r = 0 .. 3
__device__ __forceinline__ float4 shift4(const float4 lo, const float4 hi, uint32_t r) {
    float e0 = lo.x, e1 = lo.y, e2 = lo.z, e3 = lo.w, e4 = hi.x, e5 = hi.y, e6 = hi.z;
    if (r & 2u) { e0 = e2; e1 = e3; e2 = e4; e3 = e5; e4 = e6; }
    if (r & 1u) { e0 = e1; e1 = e2; e2 = e3; e3 = e4; }
    return make_float4(e0, e1, e2, e3);
}

__device__ __forceinline__ float4 scaled(const float4 v, float s) {
    return make_float4(v.x * s, v.y * s, v.z * s, v.w * s);
}

// The reductions of one (id, vector): gk = the lane's four gradient elements, gn = the four after
// them (zeros when the lane's vector is the last of its block), pos = slot of gk.x.
template <bool WRAP>
__device__ __forceinline__ void vec_scatter(float* target, uint32_t m, uint32_t pos, const float4 gk,
                                            const float4 gn, bool first_in_block, bool last_in_block) {
    const uint32_t r = pos & 3u;
    uint32_t a0 = pos & ~3u;
    // the slots below are pos .. pos + 3 (first and last lanes of a block, or no shift) or up to
    // pos + 7 - r; without WRAP the staged batch was found to keep all its blocks inside the array
    if (!ROBE_CHK((uint64_t)pos + ((r == 0 || last_in_block) ? 3u : 7u - r) < (WRAP ? 2ull * m : (uint64_t)m),
                  ROBE_DBG_ARRAY_SLOT))
        return;
    if (r == 0) {
        if (WRAP && a0 >= m) a0 -= m;
        red_add_v4(target + a0, gk);
        return;
    }
    if (first_in_block) {  // slots pos .. pos + 3 - r lie below the first full group
        uint32_t j = pos;
        if (WRAP && j >= m) j -= m;
        atomicAdd(target + j, gk.x);
        if (r <= 2) {
            j = pos + 1;
            if (WRAP && j >= m) j -= m;
            atomicAdd(target + j, gk.y);
        }
        if (r == 1) {
            j = pos + 2;
            if (WRAP && j >= m) j -= m;
            atomicAdd(target + j, gk.z);
        }
    }
    uint32_t a1 = a0 + 4u;
    if (WRAP && a1 >= m) a1 -= m;  // m is a multiple of four: the whole group wraps together
    const float4 v = shift4(gk, gn, 4u - r);
    if (!last_in_block) {
        red_add_v4(target + a1, v);
    } else {  // r elements past the last full group
        atomicAdd(target + a1, v.x);
        if (r >= 2) atomicAdd(target + a1 + 1, v.y);
        if (r == 3) atomicAdd(target + a1 + 2, v.z);
    }
}

template <bool BAGS, bool MERGE, bool WRAP>
__device__ __forceinline__ void vec_scatter_batch(const BwdArgs& a, const uint32_t* col,
                                                  const uint32_t* dup, uint32_t o, uint32_t cnt,
                                                  int64_t p0, uint32_t lpi, uint32_t ipi, uint32_t grp,
                                                  uint32_t k, bool lane_on, bool first_in_block,
                                                  bool last_in_block, float4 gk, float4 gn) {
    const MapParams& mp = a.mp;
    for (uint32_t g0 = 0; g0 < cnt; g0 += ipi) {
        const uint32_t t = g0 + grp;
        if (!lane_on || t >= cnt) continue;
        if (!BAGS) {
            const float4* rows = reinterpret_cast<const float4*>(a.grad_out);
            const uint32_t vpr = mp.d >> 2;  // vectors per row
            if (MERGE) {
                const uint32_t mk = dup[t];
                if (mk == 0) continue;  // an earlier id of the batch adds this one's row too
                gk = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                gn = gk;
                for (uint32_t rest = mk; rest != 0; rest &= rest - 1) {
                    const int64_t row = p0 + (t & ~31u) + (uint32_t)(__ffs((int)rest) - 1);
                    const float4 x = __ldcs(rows + row * vpr + k);
                    gk.x += x.x; gk.y += x.y; gk.z += x.z; gk.w += x.w;
                    if (!last_in_block) {
                        const float4 y = __ldcs(rows + row * vpr + k + 1);
                        gn.x += y.x; gn.y += y.y; gn.z += y.z; gn.w += y.w;
                    }
                }
            } else {
                const int64_t row = p0 + t;
                gk = __ldcs(rows + row * vpr + k);
                gn = last_in_block ? make_float4(0.0f, 0.0f, 0.0f, 0.0f) : __ldcs(rows + row * vpr + k + 1);
            }
            gk = scaled(gk, a.scale);
            gn = scaled(gn, a.scale);
        }
        vec_scatter<WRAP>(a.target, mp.m, col[t] + o, gk, gn, first_in_block, last_in_block);
    }
}

template <bool BAGS, bool MERGE>
__global__ void __launch_bounds__(256, 5)
bwd_atomic_vec_kernel(BwdArgs a, uint32_t ids_per_batch, uint32_t cmagic) {
    __shared__ StageSmem sm;
    __shared__ uint32_t dup_s[MERGE ? 8 : 1][kStageIds];
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

    const uint32_t lpi = mp.d >> 2, ipi = 32u / lpi, grp = lane / lpi, k = lane - grp * lpi;
    const bool lane_on = grp < ipi;
    uint32_t chk, o;
    chunk_of(mp, 4u * k, chk, o);
    const bool first_in_block = o == 0;
    const bool last_in_block = o + 4u == mp.Z || 4u * k + 4u == mp.d;
    const uint32_t* col = sm.start[w] + chk * ids_per_batch;

    float4 gk = make_float4(0.0f, 0.0f, 0.0f, 0.0f), gn = gk;
    if (BAGS && lane_on) {  // the bag's gradient row: once for all its ids
        const float4* row = reinterpret_cast<const float4*>(a.grad_out + warp * (int64_t)mp.d);
        gk = scaled(__ldcs(row + k), a.scale);
        if (!last_in_block) gn = scaled(__ldcs(row + k + 1), a.scale);
    }

    for (int64_t p0 = lo; p0 < hi; p0 += ids_per_batch) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)ids_per_batch ? (hi - p0)
                                                                            : (int64_t)ids_per_batch);
        const bool wraps = stage_batch<false, BAGS>(sm, mp, a.indices, p0, cnt, ids_per_batch, tterm, 0,
                                                    cmagic, w, lane);
        if (MERGE) {
            for (uint32_t t0 = 0; t0 < cnt; t0 += 32) {
                const uint32_t t = t0 + lane;
                const uint32_t part = __ballot_sync(0xFFFFFFFFu, t < cnt);
                if (t < cnt) {
                    // (rows clubbed into one block share a hash base without sharing slots: no merge)
                    const uint32_t same = mp.R > 1 ? (1u << lane) : __match_any_sync(part, sm.base[w][t]);
                    dup_s[w][t] = ((same & ((1u << lane) - 1u)) == 0) ? same : 0u;
                }
            }
            __syncwarp();
        }
        const uint32_t* dup = MERGE ? dup_s[w] : nullptr;
        if (wraps)
            vec_scatter_batch<BAGS, MERGE, true>(a, col, dup, o, cnt, p0, lpi, ipi, grp, k, lane_on,
                                                 first_in_block, last_in_block, gk, gn);
        else
            vec_scatter_batch<BAGS, MERGE, false>(a, col, dup, o, cnt, p0, lpi, ipi, grp, k, lane_on,
                                                  first_in_block, last_in_block, gk, gn);
        __syncwarp();
    }
}

// Lane-hashed kernel for short blocks (the mirror of the forward's): every lane hashes the chunks
// of its own elements in registers and issues one reduction per (id, owned element); persistent
// warps, 32 ids' shared hash parts evaluated at a time and handed round by shuffle.
template <int EPL, bool BAGS, bool M30>
__global__ void __launch_bounds__(256, 4)
bwd_atomic_lanehash_kernel(BwdArgs a, uint32_t padj) {
    __shared__ uint64_t tt_s[kRowTables];
    const MapParams& mp = a.mp;
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t e = threadIdx.x; e < mp.T && e < (uint32_t)kRowTables; e += 256) tt_s[e] = table_term(mp.h, e);
    __syncthreads();
    if (a.status != nullptr && *a.status != 0) return;

    LaneChunks<EPL> lc;
    lc.init(mp, lane, padj);
    const uint64_t pol = l2_keep_policy(a.l2_keep != 0);
    const int64_t nwarps = (int64_t)gridDim.x * 8;
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);

    auto scatter_id = [&](uint32_t bm, uint64_t thr, int src, const float (&gv)[EPL]) {
        const uint32_t bm_g = __shfl_sync(0xFFFFFFFFu, bm, src);
        const uint64_t thr_g = __shfl_sync(0xFFFFFFFFu, thr, src);
#pragma unroll
        for (int u = 0; u < EPL; ++u)
            if (lc.live[u]) {
                const uint32_t j = lc.template slot<M30>(u, bm_g, thr_g);
                if (ROBE_CHK(j < mp.m, ROBE_DBG_ARRAY_SLOT)) red_add(a.target + j, gv[u], pol);
            }
    };

    if (!BAGS) {
        for (int64_t r0 = gw * 32; r0 < a.nbags; r0 += nwarps * 32) {
            const int64_t row = r0 + lane;
            uint32_t bm = 0;
            uint64_t thr = kP61;
            if (row < a.nbags)
                lane_id_base(mp, lane_table_term(tt_s, mp, (uint64_t)row), (uint64_t)a.indices.load(row), bm, thr);
            const uint32_t n = (uint32_t)(a.nbags - r0 < 32 ? a.nbags - r0 : 32);
            for (uint32_t g = 0; g < n; g += 2) {  // the gradient rows of two ids are fetched together
                float gv[2][EPL];
#pragma unroll
                for (int gg = 0; gg < 2; ++gg)
#pragma unroll
                    for (int u = 0; u < EPL; ++u) {
                        gv[gg][u] = 0.0f;
                        if (g + gg < n && lc.live[u])
                            gv[gg][u] = __ldcs(a.grad_out + (r0 + g + gg) * (int64_t)mp.d + lane + 32u * u) * a.scale;
                    }
                scatter_id(bm, thr, (int)g, gv[0]);
                if (g + 1 < n) scatter_id(bm, thr, (int)g + 1, gv[1]);
            }
        }
    } else {
        for (int64_t bag = gw; bag < a.nbags; bag += nwarps) {
            int64_t lo, hi;
            bag_range(a.offsets, a.nnz, bag, lo, hi);
            if (hi <= lo) continue;
            const uint64_t tterm = lane_table_term(tt_s, mp, (uint64_t)bag);
            float gv[EPL];
#pragma unroll
            for (int u = 0; u < EPL; ++u) {
                gv[u] = 0.0f;
                if (lc.live[u]) gv[u] = __ldcs(a.grad_out + bag * (int64_t)mp.d + lane + 32u * u) * a.scale;
            }
            for (int64_t p0 = lo; p0 < hi; p0 += 32) {
                uint32_t bm = 0;
                uint64_t thr = kP61;
                if (p0 + lane < hi) lane_id_base(mp, tterm, (uint64_t)a.indices.load(p0 + lane), bm, thr);
                const uint32_t n = (uint32_t)(hi - p0 < 32 ? hi - p0 : 32);
                for (uint32_t g = 0; g < n; ++g) scatter_id(bm, thr, (int)g, gv);
            }
        }
    }
}

template <int EPL>
static void launch_bwd_lanehash_m(const BwdArgs& a, bool bags, cudaStream_t st) {
    const unsigned blocks = lane_grid(bags ? a.nbags : (a.nbags + 31) / 32);
    const uint32_t padj = lane_padj(a.mp);
    const bool m30 = a.mp.m < (1u << 30);
    if (bags) {
        if (m30) bwd_atomic_lanehash_kernel<EPL, true, true><<<blocks, 256, 0, st>>>(a, padj);
        else bwd_atomic_lanehash_kernel<EPL, true, false><<<blocks, 256, 0, st>>>(a, padj);
    } else {
        if (m30) bwd_atomic_lanehash_kernel<EPL, false, true><<<blocks, 256, 0, st>>>(a, padj);
        else bwd_atomic_lanehash_kernel<EPL, false, false><<<blocks, 256, 0, st>>>(a, padj);
    }
}

static void launch_bwd_lanehash(const BwdArgs& a, bool bags, cudaStream_t st) {
    if (a.mp.d <= 32) launch_bwd_lanehash_m<1>(a, bags, st);
    else if (a.mp.d <= 64) launch_bwd_lanehash_m<2>(a, bags, st);
    else launch_bwd_lanehash_m<4>(a, bags, st);
}

// what the vector kernels ask of a call
static bool bwd_vec_ok(const Problem& pb, const float* grad_out, const float* target) {
    const MapParams& mp = pb.mp;
    return pb.sign == 0 && mp.d <= 128 && mp.d % 4 == 0 && mp.Z % 4 == 0 && mp.m % 4 == 0 &&
           ((uintptr_t)grad_out & 15u) == 0 && ((uintptr_t)target & 15u) == 0;
}

template <int EPL, bool SIGN, bool FULLD, int MINB>
static void launch_bwd_staged_minb(const BwdArgs& a, bool bags, cudaStream_t st) {
    const uint32_t ipb = staged_ids_per_batch(a.mp, bags, SIGN);
    const uint32_t cmagic = chunk_magic(a.mp);
    const int64_t warps = bags ? a.nbags : (a.nbags + ipb - 1) / ipb;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags)
        bwd_atomic_staged_kernel<EPL, SIGN, true, FULLD, MINB><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
    else
        bwd_atomic_staged_kernel<EPL, SIGN, false, FULLD, MINB><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
}

template <int EPL, bool SIGN, bool FULLD>
static void launch_bwd_staged(const BwdArgs& a, bool bags, cudaStream_t st) {
    const bool l2_sized = (uint64_t)a.mp.m * 4u <= kL2SizedBytes;  // (see kStagedCtas*)
    if constexpr (SIGN) launch_bwd_staged_minb<EPL, SIGN, FULLD, kStagedCtasSign>(a, bags, st);
    else if constexpr (EPL == 4) launch_bwd_staged_minb<EPL, SIGN, FULLD, kStagedCtasWide>(a, bags, st);
    else if (l2_sized) launch_bwd_staged_minb<EPL, SIGN, FULLD, kStagedCtasL2>(a, bags, st);
    else launch_bwd_staged_minb<EPL, SIGN, FULLD, kStagedCtasHbm>(a, bags, st);
}

template <int EPL>
static void launch_bwd_staged_flags(const BwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    const bool fulld = a.mp.d == 32u * EPL;
    if (sign) launch_bwd_staged<EPL, true, false>(a, bags, st);
    else if (fulld) launch_bwd_staged<EPL, false, true>(a, bags, st);
    else launch_bwd_staged<EPL, false, false>(a, bags, st);
}

static void launch_bwd_staged_epl(const BwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    if (a.mp.d <= 32) launch_bwd_staged_flags<1>(a, bags, sign, st);
    else if (a.mp.d <= 64) launch_bwd_staged_flags<2>(a, bags, sign, st);
    else launch_bwd_staged_flags<4>(a, bags, sign, st);
}

cudaError_t launch_backward_atomic(const Problem& pb, const float* grad_out, float* target,
                                   float scale, int variant, cudaStream_t st) {
    if (pb.nbags == 0) return cudaSuccess;
    BwdArgs a{pb.mp, grad_out, pb.indices, pb.offsets, target, scale, pb.nbags, pb.nnz, pb.status, pb.l2_keep};
    const bool bags = pb.offsets != nullptr;
    const bool warp_ok = pb.mp.d <= 128;
    if (variant == 2 && !warp_ok) return cudaErrorInvalidValue;
    // Short blocks: every lane hashes its own chunks.  Never the automatic choice: unlike the forward,
    // the backward at Z <= 2 is bound by the reductions themselves, not by instruction issue (measured
    // on B200 against the staged kernel: 1 MB array Z=1 2.28 -> 2.45 ms, Z=2 1.61 -> 1.43 ms, 100 MB
    // 5.03 -> 5.66 / 3.24 -> 3.42 ms, Zipf ids Z=1 0.91 -> 0.97 ms).
    const bool lane_ok = pb.sign == 0 && pb.mp.R == 1 && warp_ok;
    if (variant == 6) {
        if (!lane_ok) return cudaErrorInvalidValue;
        launch_bwd_lanehash(a, bags, st);
        return cudaGetLastError();
    }
    if (variant == 5) {  // one-hot rows taken table by table, repeats of an id merged in the warp
        if (bags || pb.sign != 0 || !warp_ok || pb.nbags % pb.mp.T != 0) return cudaErrorInvalidValue;
        uint32_t ipb = (uint32_t)kStageEntries / a.mp.C;  // as many rows as the staging area holds
        if (ipb > (uint32_t)kStageIds) ipb = kStageIds;
        if (ipb < 1) ipb = 1;
        const int64_t batch = pb.nbags / pb.mp.T;
        const int64_t warps = ((batch + ipb - 1) / ipb) * pb.mp.T;
        const unsigned blocks = (unsigned)((warps + 7) / 8);
        const uint32_t cmagic = chunk_magic(a.mp);
        if (a.mp.d <= 32) bwd_atomic_staged_kernel<1, false, false, false, 6, true><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        else if (a.mp.d <= 64) bwd_atomic_staged_kernel<2, false, false, false, 6, true><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        else bwd_atomic_staged_kernel<4, false, false, false, 5, true><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        return cudaGetLastError();
    }
    if (variant == 3 || variant == 4) {  // 16-byte reductions; 4: duplicates of an id merged first
        if (!bwd_vec_ok(pb, grad_out, target)) return cudaErrorInvalidValue;
        const uint32_t ipb = staged_ids_per_batch(a.mp, bags, false);
        const uint32_t cmagic = chunk_magic(a.mp);
        const int64_t warps = bags ? a.nbags : (a.nbags + ipb - 1) / ipb;
        const unsigned blocks = (unsigned)((warps + 7) / 8);
        if (bags) bwd_atomic_vec_kernel<true, false><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        else if (variant == 4) bwd_atomic_vec_kernel<false, true><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        else bwd_atomic_vec_kernel<false, false><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
        return cudaGetLastError();
    }
    const bool use_warp = variant == 2 || (variant == 0 && warp_ok);
    if (use_warp) {
        launch_bwd_staged_epl(a, bags, pb.sign != 0, st);
    } else {
        const unsigned blocks = (unsigned)((pb.nbags + 7) / 8);
        if (pb.sign) bwd_atomic_direct_kernel<true><<<blocks, 256, 0, st>>>(a);
        else bwd_atomic_direct_kernel<false><<<blocks, 256, 0, st>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace robe
