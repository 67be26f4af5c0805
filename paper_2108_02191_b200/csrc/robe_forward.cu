// Forward lookup kernels (Section 3.2 forward: the embedding is the concatenation of
// ceil(d/Z) blocks M[h(e,x,c) : h(e,x,c)+Z] read circularly; Section 3.1 for the optional
// element-wise sign).  Sum pooling over a bag is sequential in fp32 in bag order.
//
// Two kernels:
//   fwd_direct_kernel  any Z, any d: every lane hashes the chunk of its own element.
//   fwd_warp_kernel    Z a power of two and d <= 128: the 32 lanes of a warp first
//                      evaluate 32 block starts at once (several ids x chunks), then
//                      hand them to the lanes that gather through warp shuffles, so the
//                      hash cost per id does not depend on how many lanes read a block.
#include "robe_internal.h"

namespace robe {

struct FwdArgs {
    MapParams mp;
    const void* array;
    const int64_t* indices;
    const int64_t* offsets;
    float* out;
    int64_t nbags;
    int64_t nnz;
    const int32_t* status;
};

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
            const uint64_t x = (uint64_t)__ldg(a.indices + p);
            uint32_t j = block_start(mp, hash_base(mp.h, e, x), c) + o;  // < m + d <= 2^32
            if (j >= mp.m) j -= mp.m;
            float v = load_elem<DT>(a.array, j);
            if (SIGN) v = sign_of(mp, hash_base(mp.g, e, x), i) * v;
            acc = (p == lo) ? v : acc + v;
        }
        __stcs(a.out + k * mp.d + i, acc);
    }
}

// EPL   elements per lane (d <= 32*EPL)
// MULTI chunks per embedding C > 32: a lane holds up to four block starts (chunks cl + 32k)
// FULLD d == 32*EPL: no lane is ever past the end of the row
// U     ids whose loads are issued before the first add
template <int EPL, int DT, bool SIGN, bool BAGS, bool MULTI, bool FULLD>
__global__ void __launch_bounds__(256) fwd_warp_kernel(FwdArgs a, uint32_t log2sub) {
    constexpr int U = (EPL == 4) ? 2 : 4;
    constexpr int KS = MULTI ? 4 : 1;
    constexpr unsigned FULL = 0xFFFFFFFFu;
    const MapParams& mp = a.mp;
    const int64_t warp = ((int64_t)blockIdx.x * 256 + threadIdx.x) >> 5;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t sub = 1u << log2sub;   // lanes that hash one id: min(32, pow2ceil(C))
    const uint32_t G = 32u >> log2sub;    // ids hashed per pass
    const uint32_t gl = lane >> log2sub;  // which id of the pass this lane hashes
    const uint32_t cl = lane & (sub - 1); // which chunk (plus multiples of 32 when C > 32)

    if (a.status != nullptr && *a.status != 0) return;

    int64_t row0, lo, hi;
    uint64_t tterm = 0, gterm = 0;  // (A e + D) mod P of the bag's table (pooled mode)
    if (BAGS) {
        if (warp >= a.nbags) return;
        bag_range(a.offsets, a.nnz, warp, lo, hi);
        const uint32_t e_bag = table_of_bag((uint64_t)warp, mp);
        tterm = table_term(mp.h, e_bag);
        if (SIGN) gterm = table_term(mp.g, e_bag);
        row0 = warp;
    } else {
        row0 = warp * (int64_t)G;  // this warp serves rows [row0, row0 + G)
        if (row0 >= a.nbags) return;
        lo = row0;
        hi = row0 + G < a.nbags ? row0 + G : a.nbags;
    }

    // per-lane constants of the gather: element i = lane + 32u, its chunk and offset
    uint32_t off[EPL], src[EPL], slot[EPL];
    bool live[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) {
        uint32_t i = lane + 32u * u;
        live[u] = FULLD || i < mp.d;
        if (!live[u]) i = mp.d - 1;
        const uint32_t c = i >> mp.log2Z;
        off[u] = i & (mp.Z - 1);
        src[u] = c & (sub - 1);
        slot[u] = c >> 5;  // warp-uniform (non-zero only when C > 32)
    }
    // per-lane constants of the hash pass: (C_h * c) mod P for the chunks this lane evaluates
    uint64_t cterm[KS];
#pragma unroll
    for (int k = 0; k < KS; ++k) cterm[k] = mulmod_p61_u32(mp.h.C, cl + 32u * k);

    // -0 + v == v for every v (also for v = -0), so starting from -0 makes the first term
    // initialise the sum exactly as the definition says
    float acc[EPL];
#pragma unroll
    for (int u = 0; u < EPL; ++u) acc[u] = -0.0f;

    uint64_t x_next = 0;
    if (lo + gl < hi) x_next = (uint64_t)__ldg(a.indices + lo + gl);

    for (int64_t p0 = lo; p0 < hi; p0 += G) {
        const uint32_t cnt = (uint32_t)((hi - p0) < (int64_t)G ? (hi - p0) : (int64_t)G);
        // ---- hash pass: lane (gl, cl) evaluates the starts of id p0+gl, chunks cl (+32k)
        uint32_t st[KS];
        uint64_t gbase = 0;
        {
            const uint64_t x = x_next;
            if (p0 + G + gl < hi) x_next = (uint64_t)__ldg(a.indices + p0 + G + gl);
            uint64_t tt = tterm;
            if (!BAGS) {
                const uint32_t e = table_of_bag((uint64_t)(p0 + gl), mp);
                tt = table_term(mp.h, e);
                if (SIGN) gterm = table_term(mp.g, e);
            }
            const uint64_t base = addmod_p61(tt, mulmod_p61_any(mp.h.B, x));
            if (SIGN) gbase = addmod_p61(gterm, mulmod_p61_any(mp.g.B, x));
#pragma unroll
            for (int k = 0; k < KS; ++k)
                st[k] = mod_m(addmod_p61(base, cterm[k]), mp.m, mp.mu);
        }
        // ---- gather pass
        for (uint32_t g0 = 0; g0 < cnt; g0 += U) {
            float v[U][EPL];
#pragma unroll
            for (int gg = 0; gg < U; ++gg) {
                const uint32_t g = g0 + gg;           // warp-uniform
                const uint32_t gs = g < cnt ? g : cnt - 1;
                uint64_t gb = 0;
                if (SIGN) gb = __shfl_sync(FULL, gbase, gs << log2sub);
#pragma unroll
                for (int u = 0; u < EPL; ++u) {
                    uint32_t mine = st[0];
                    if (MULTI) mine = slot[u] == 0 ? st[0] : slot[u] == 1 ? st[1 % KS]
                                    : slot[u] == 2 ? st[2 % KS] : st[3 % KS];
                    const uint32_t s = __shfl_sync(FULL, mine, (gs << log2sub) + src[u]);
                    uint32_t j = s + off[u];
                    if (j >= mp.m) j -= mp.m;
                    float val = 0.0f;
                    if (g < cnt && live[u]) {
                        val = gather_elem<DT>(a.array, j);
                        if (SIGN) val = sign_of(mp, gb, lane + 32u * u) * val;
                    }
                    v[gg][u] = val;
                }
            }
            if (BAGS) {
#pragma unroll
                for (int gg = 0; gg < U; ++gg) {
                    if (g0 + gg < cnt) {
#pragma unroll
                        for (int u = 0; u < EPL; ++u) acc[u] = acc[u] + v[gg][u];
                    }
                }
            } else {
#pragma unroll
                for (int gg = 0; gg < U; ++gg) {
                    if (g0 + gg < cnt) {
                        float* orow = a.out + (p0 + g0 + gg) * (int64_t)mp.d;
#pragma unroll
                        for (int u = 0; u < EPL; ++u)
                            if (live[u]) __stcs(orow + lane + 32u * u, v[gg][u]);
                    }
                }
            }
        }
    }
    if (BAGS) {
        float* orow = a.out + row0 * (int64_t)mp.d;
        const bool empty = hi <= lo;
#pragma unroll
        for (int u = 0; u < EPL; ++u)
            if (live[u]) __stcs(orow + lane + 32u * u, empty ? 0.0f : acc[u]);
    }
}

static uint32_t log2_sub_for(uint32_t C) {
    uint32_t l = 0;
    while ((1u << l) < C && l < 5) ++l;
    return l;
}

template <int EPL, int DT, bool SIGN, bool MULTI, bool FULLD>
static void launch_warp(const FwdArgs& a, bool bags, cudaStream_t st) {
    const uint32_t l2s = log2_sub_for(a.mp.C);
    const int64_t G = 32 >> l2s;
    const int64_t warps = bags ? a.nbags : (a.nbags + G - 1) / G;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
    if (bags)
        fwd_warp_kernel<EPL, DT, SIGN, true, MULTI, FULLD><<<blocks, 256, 0, st>>>(a, l2s);
    else
        fwd_warp_kernel<EPL, DT, SIGN, false, MULTI, FULLD><<<blocks, 256, 0, st>>>(a, l2s);
}

template <int EPL, int DT>
static void launch_warp_flags(const FwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    const bool multi = a.mp.C > 32;
    const bool fulld = a.mp.d == 32u * EPL;
    if (sign) {  // the sign hash is off in every timed configuration: one generic variant
        launch_warp<EPL, DT, true, true, false>(a, bags, st);
        return;
    }
    if (EPL == 1) {  // d <= 32 means C <= 32
        if (fulld) launch_warp<EPL, DT, false, false, true>(a, bags, st);
        else launch_warp<EPL, DT, false, false, false>(a, bags, st);
        return;
    }
    if (multi) {
        if (fulld) launch_warp<EPL, DT, false, true, true>(a, bags, st);
        else launch_warp<EPL, DT, false, true, false>(a, bags, st);
    } else {
        if (fulld) launch_warp<EPL, DT, false, false, true>(a, bags, st);
        else launch_warp<EPL, DT, false, false, false>(a, bags, st);
    }
}

template <int DT>
static void launch_warp_epl(const FwdArgs& a, bool bags, bool sign, cudaStream_t st) {
    if (a.mp.d <= 32)
        launch_warp_flags<1, DT>(a, bags, sign, st);
    else if (a.mp.d <= 64)
        launch_warp_flags<2, DT>(a, bags, sign, st);
    else
        launch_warp_flags<4, DT>(a, bags, sign, st);
}

cudaError_t launch_forward(const Problem& pb, float* out, int variant, cudaStream_t st) {
    if (pb.nbags == 0) return cudaSuccess;
    FwdArgs a{pb.mp, pb.array, pb.indices, pb.offsets, out, pb.nbags, pb.nnz, pb.status};
    const bool bags = pb.offsets != nullptr;
    const bool warp_ok = pb.mp.log2Z != 0xFFFFFFFFu && pb.mp.d <= 128;
    if (variant == 2 && !warp_ok) return cudaErrorInvalidValue;
    const bool use_warp = variant == 2 || (variant == 0 && warp_ok);
    if (use_warp) {
        if (pb.dtype == 0) launch_warp_epl<0>(a, bags, pb.sign != 0, st);
        else launch_warp_epl<1>(a, bags, pb.sign != 0, st);
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
