// Atomic backward (Section 3.1 backward equation): every element of the output gradient
// is added, with its sign, into the array slot it was read from in the forward pass:
//   delta[idx(e,x,i)] += g(e,x,i) * grad_out[bag, i]      for every id x of every bag.
// `target` is either a dense fp32 gradient array (scale = 1) or the parameter array
// itself (scale = -lr: the SGD step fused into the scatter).  fp32 reductions in global
// memory (red.global.add.f32); the order of the additions is not fixed.
//
// Same two shapes as the forward: a direct kernel for any (Z, d) and a warp kernel that
// evaluates 32 block starts per pass and distributes them by shuffles.
#include "robe_internal.h"

namespace robe {

struct BwdArgs {
    MapParams mp;
    const float* grad_out;
    const int64_t* indices;
    const int64_t* offsets;
    float* target;
    float scale;
    int64_t nbags;
    int64_t nnz;
    const int32_t* status;
};

__device__ __forceinline__ int64_t clamp64b(int64_t v, int64_t lo, int64_t hi) {
    return v < lo ? lo : (v > hi ? hi : v);
}

__device__ __forceinline__ void bag_range_b(const int64_t* offsets, int64_t nnz, int64_t k,
                                            int64_t& lo, int64_t& hi) {
    if (offsets == nullptr) {
        lo = k;
        hi = k + 1;
    } else {
        lo = clamp64b(__ldg(offsets + k), 0, nnz);
        hi = clamp64b(__ldg(offsets + k + 1), lo, nnz);
    }
}

template <bool SIGN>
__global__ void __launch_bounds__(256) bwd_atomic_direct_kernel(BwdArgs a) {
    const int64_t k = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    if (k >= a.nbags) return;
    if (a.status != nullptr && *a.status != 0) return;
    const MapParams& mp = a.mp;
    int64_t lo, hi;
    bag_range_b(a.offsets, a.nnz, k, lo, hi);
    const uint32_t e = table_of_bag((uint64_t)k, mp);
    for (uint32_t i = lane; i < mp.d; i += 32) {
        uint32_t c, o;
        chunk_of(mp, i, c, o);
        const float gv = __ldcs(a.grad_out + k * mp.d + i) * a.scale;
        for (int64_t p = lo; p < hi; ++p) {
            const uint64_t x = (uint64_t)__ldg(a.indices + p);
            uint32_t j = block_start(mp, hash_base(mp.h, e, x), c) + o;
            if (j >= mp.m) j -= mp.m;
            float t = gv;
            if (SIGN) t = sign_of(mp, hash_base(mp.g, e, x), i) * t;
            atomicAdd(a.target + j, t);
        }
    }
}

template <int EPL, bool SIGN, bool BAGS>
__global__ void __launch_bounds__(256) bwd_atomic_warp_kernel(BwdArgs a, uint32_t log2sub) {
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const MapParams& mp = a.mp;
    const int64_t warp = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t sub = 1u << log2sub;
    const uint32_t G = 32u >> log2sub;
    const uint32_t gl = lane >> log2sub;
    const uint32_t cl = lane & (sub - 1);

    if (a.status != nullptr && *a.status != 0) return;

    uint32_t off[EPL], src[EPL], slot[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) {
        uint32_t i = lane + 32u * u;
        if (i >= mp.d) i = mp.d - 1;
        uint32_t c = i >> mp.log2Z;
        off[u] = i & (mp.Z - 1);
        src[u] = c & (sub - 1);
        slot[u] = c >> 5;
    }

    int64_t lo, hi;
    uint32_t e_bag = 0;
    float gbag[EPL];
    if (BAGS) {
        if (warp >= a.nbags) return;
        bag_range_b(a.offsets, a.nnz, warp, lo, hi);
        e_bag = table_of_bag((uint64_t)warp, mp);
#pragma unroll
        for (int u = 0; u < EPL; ++u)
            gbag[u] = lane + 32u * u < mp.d
                          ? __ldcs(a.grad_out + warp * (int64_t)mp.d + lane + 32u * u) * a.scale
                          : 0.0f;
    } else {
        lo = warp * (int64_t)G;
        if (lo >= a.nbags) return;
        hi = lo + G < a.nbags ? lo + G : a.nbags;
    }

    for (int64_t p0 = lo; p0 < hi; p0 += G) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)G ? (hi - p0) : (int64_t)G);
        uint32_t st[4] = {0, 0, 0, 0};
        uint64_t gbase = 0;
        if (gl < cnt) {
            const int64_t p = p0 + gl;
            const uint64_t x = (uint64_t)__ldg(a.indices + p);
            const uint32_t e = BAGS ? e_bag : table_of_bag((uint64_t)p, mp);
            const uint64_t base = hash_base(mp.h, e, x);
            if (SIGN) gbase = hash_base(mp.g, e, x);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t c = cl + 32u * k;
                if (c < mp.C) st[k] = block_start(mp, base, c);
            }
        }
        for (uint32_t g = 0; g < cnt; ++g) {
            float gv[EPL];
            if (BAGS) {
#pragma unroll
                for (int u = 0; u < EPL; ++u) gv[u] = gbag[u];
            } else {
#pragma unroll
                for (int u = 0; u < EPL; ++u)
                    gv[u] = lane + 32u * u < mp.d
                                ? __ldcs(a.grad_out + (p0 + g) * (int64_t)mp.d + lane + 32u * u) *
                                      a.scale
                                : 0.0f;
            }
            uint64_t gb = 0;
            if (SIGN) gb = __shfl_sync(FULL, gbase, g << log2sub);
#pragma unroll
            for (int u = 0; u < EPL; ++u) {
                uint32_t mine = slot[u] == 0 ? st[0] : slot[u] == 1 ? st[1]
                              : slot[u] == 2 ? st[2] : st[3];
                uint32_t s = __shfl_sync(FULL, mine, (g << log2sub) + src[u]);
                uint32_t j = s + off[u];
                if (j >= mp.m) j -= mp.m;
                if (lane + 32u * u < mp.d) {
                    float t = gv[u];
                    if (SIGN) t = sign_of(mp, gb, lane + 32u * u) * t;
                    atomicAdd(a.target + j, t);
                }
            }
        }
    }
}

static uint32_t log2_sub_for_b(uint32_t C) {
    uint32_t l = 0;
    while ((1u << l) < C && l < 5) ++l;
    return l;
}

template <int EPL, bool SIGN>
static void launch_bwd_warp(const BwdArgs& a, bool bags, cudaStream_t st) {
    const uint32_t l2s = log2_sub_for_b(a.mp.C);
    const int64_t G = 32 >> l2s;
    const int64_t warps = bags ? a.nbags : (a.nbags + G - 1) / G;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags)
        bwd_atomic_warp_kernel<EPL, SIGN, true><<<blocks, 256, 0, st>>>(a, l2s);
    else
        bwd_atomic_warp_kernel<EPL, SIGN, false><<<blocks, 256, 0, st>>>(a, l2s);
}

template <bool SIGN>
static void launch_bwd_warp_epl(const BwdArgs& a, bool bags, cudaStream_t st) {
    if (a.mp.d <= 32)
        launch_bwd_warp<1, SIGN>(a, bags, st);
    else if (a.mp.d <= 64)
        launch_bwd_warp<2, SIGN>(a, bags, st);
    else
        launch_bwd_warp<4, SIGN>(a, bags, st);
}

cudaError_t launch_backward_atomic(const Problem& pb, const float* grad_out, float* target,
                                   float scale, int variant, cudaStream_t st) {
    if (pb.nbags == 0) return cudaSuccess;
    BwdArgs a{pb.mp, grad_out, pb.indices, pb.offsets, target, scale, pb.nbags, pb.nnz, pb.status};
    const bool bags = pb.offsets != nullptr;
    const bool warp_ok = pb.mp.log2Z != 0xFFFFFFFFu && pb.mp.d <= 128;
    if (variant == 2 && !warp_ok) return cudaErrorInvalidValue;
    const bool use_warp = variant == 2 || (variant == 0 && warp_ok);
    if (use_warp) {
        if (pb.sign) launch_bwd_warp_epl<true>(a, bags, st);
        else launch_bwd_warp_epl<false>(a, bags, st);
    } else {
        const unsigned blocks = (unsigned)((pb.nbags + 7) / 8);
        if (pb.sign) bwd_atomic_direct_kernel<true><<<blocks, 256, 0, st>>>(a);
        else bwd_atomic_direct_kernel<false><<<blocks, 256, 0, st>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace robe
