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
            atomicAdd(a.target + j, t);
        }
    }
}

// Staged kernel (any Z, d <= 128): same two phases as the staged forward kernel - the warp
// first evaluates the block starts of a batch of ids into its shared-memory staging area, then
// every lane issues one fp32 reduction per (id, element) it owns.  The gradient row of a bag is
// read once and kept in registers for all ids of the bag.
template <int EPL, bool SIGN, bool BAGS, bool FULLD, int MINB>
__global__ void __launch_bounds__(256, MINB)
bwd_atomic_staged_kernel(BwdArgs a, uint32_t ids_per_batch, uint32_t cmagic) {
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
        lo = warp * (int64_t)ids_per_batch;
        if (lo >= a.nbags) return;
        hi = lo + ids_per_batch < a.nbags ? lo + ids_per_batch : a.nbags;
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

    for (int64_t p0 = lo; p0 < hi; p0 += ids_per_batch) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)ids_per_batch ? (hi - p0)
                                                                            : (int64_t)ids_per_batch);
        stage_batch<SIGN, BAGS>(sm, mp, a.indices, p0, cnt, ids_per_batch, tterm, gterm, cmagic, w, lane);
        for (uint32_t g = 0; g < cnt; ++g) {
            if (!BAGS) {
#pragma unroll
                for (int u = 0; u < EPL; ++u)
                    if (live[u])
                        gv[u] = __ldcs(a.grad_out + (p0 + g) * (int64_t)mp.d + lane + 32u * u) * a.scale;
            }
#pragma unroll
            for (int u = 0; u < EPL; ++u) {
                uint32_t j = start_s[chk[u] * ids_per_batch + g] + off[u];
                if (j >= mp.m) j -= mp.m;
                if (live[u]) {
                    float t = gv[u];
                    if (SIGN) t = sign_of(mp, gbase_s[g], lane + 32u * u) * t;
                    atomicAdd(a.target + j, t);
                }
            }
        }
        __syncwarp();
    }
}

template <int EPL, bool SIGN, bool FULLD>
static void launch_bwd_staged(const BwdArgs& a, bool bags, cudaStream_t st) {
    constexpr int MINB = (EPL == 4) ? 6 : 8;
    const uint32_t ipb = staged_ids_per_batch(a.mp, bags, SIGN);
    const uint32_t cmagic = chunk_magic(a.mp);
    const int64_t warps = bags ? a.nbags : (a.nbags + ipb - 1) / ipb;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags)
        bwd_atomic_staged_kernel<EPL, SIGN, true, FULLD, MINB><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
    else
        bwd_atomic_staged_kernel<EPL, SIGN, false, FULLD, MINB><<<blocks, 256, 0, st>>>(a, ipb, cmagic);
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
    BwdArgs a{pb.mp, grad_out, pb.indices, pb.offsets, target, scale, pb.nbags, pb.nnz, pb.status};
    const bool bags = pb.offsets != nullptr;
    const bool warp_ok = pb.mp.d <= 128;
    if (variant == 2 && !warp_ok) return cudaErrorInvalidValue;
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
