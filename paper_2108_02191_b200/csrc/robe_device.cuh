// Device-side integer arithmetic of the ROBE-Z location mapping (Section 3.2:
// h(e,x,c) = ((A e + B x + C c + D) mod P) mod m, idx = (h + i mod Z) mod m) and of the
// optional sign hash (Section 3.1, g equation), for P = 2^61 - 1 and m < 2^32.
//
// Everything here is exact integer work, restructured for 32-bit integer ALUs:
//   * a product with a 61-bit constant is a 64x64->128 multiply folded with
//     2^61 = 1 (mod P);
//   * the per-(table,id) part of the sum is reduced once and the per-chunk part
//     C*c mod P is added afterwards (sums of residues, then one conditional subtract);
//   * "mod m" is a Barrett reduction with mu = floor(2^64 / m) and one correction.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace robe {

constexpr uint64_t kP61 = (1ull << 61) - 1ull;

// Index checks of the debug build (compiled with -DROBE_DEBUG as ONE translation unit, so that
// the word below exists once).  ROBE_CHK(cond, code) guards a computed index: in the debug build a
// false condition records `code` (the first one sticks) and the guarded access is skipped - no
// trap, no assert, the context stays usable; in the release build it is the constant `true` and
// costs nothing.  robe_debug_status() reads and clears the word.
// codes (the values the C header documents):
//   ROBE_DBG_ARRAY_SLOT  array / gradient slot >= m
//   ROBE_DBG_SORT_POS    sorted position or block number >= number of blocks
//   ROBE_DBG_SHARED      shared-memory index beyond its buffer
//   ROBE_DBG_GRAD_POS    position in grad_out beyond bags * d
//   ROBE_DBG_WINDOW      window number beyond the window tables
//   ROBE_DBG_LONG_WALK   hand-over record beyond the list
//   ROBE_DBG_SELFTEST    planted by robe_debug_selftest
#include "../../include/robe.h"
#ifdef ROBE_DEBUG
__device__ int32_t g_robe_debug_code;
__device__ __forceinline__ bool robe_dbg_ok(bool cond, int32_t code) {
    if (!cond) atomicCAS(&g_robe_debug_code, 0, code);
    return cond;
}
#define ROBE_CHK(cond, code) (::robe::robe_dbg_ok((cond), (code)))
#else
#define ROBE_CHK(cond, code) true
#endif

struct HashConsts {  // all < P
    uint64_t A, B, C, D;
};

// The ids of a call: int64 (default) or int32 elements, read through the read-only path.
struct IdList {
    const void* p;
    int i32;  // 0: int64_t elements, 1: int32_t elements
    __device__ __forceinline__ int64_t load(int64_t pos) const {
        return i32 ? (int64_t)__ldg((const int32_t*)p + pos) : __ldg((const int64_t*)p + pos);
    }
};

// Everything a kernel needs to map (e, x, c) to a block start.
struct MapParams {
    HashConsts h;      // location hash
    HashConsts g;      // sign hash
    uint64_t mu;       // floor(2^64 / m)  (2^64 - 1 when m == 1)
    uint32_t m;        // array length (m + d <= 2^32)
    uint32_t T;        // number of tables
    uint32_t d;        // embedding dimension
    uint32_t Z;        // block length the kernels work with: the block size, or d when rows are clubbed
    uint32_t R;        // rows clubbed into one block: block size / d when that exceeds 1, else 1
    uint32_t C;        // blocks per embedding = ceil(d / Z)
    uint32_t log2Z;    // valid when Z is a power of two, else 0xFFFFFFFF
    uint64_t tmagic;   // floor((2^64 - 1) / T) + 1, for k mod T with k < 2^32
    uint64_t bmagic;   // table-major bags: floor((2^64 - 1) / B) + 1, for k / B with k < 2^32
    uint32_t B;        // table-major bags: the batch size B of the call; 0 = sample-major bags
};

// (hi * 2^64 + lo) mod P for hi < 2^61.
__device__ __forceinline__ uint64_t fold_p61(uint64_t hi, uint64_t lo) {
    uint64_t v0 = lo & kP61;
    uint64_t v1 = ((lo >> 61) | (hi << 3)) & kP61;
    uint64_t v2 = hi >> 58;
    uint64_t s = v0 + v1 + v2;       // < 2^62 + 2^6
    s = (s & kP61) + (s >> 61);      // <= P + 2
    return s >= kP61 ? s - kP61 : s;
}

// (a * b) mod P, a < P, b any 64-bit value.
__device__ __forceinline__ uint64_t mulmod_p61(uint64_t a, uint64_t b) {
    return fold_p61(__umul64hi(a, b), a * b);
}

// (a * b) mod P, a < P, b < 2^32: the product has at most 93 bits.
__device__ __forceinline__ uint64_t mulmod_p61_u32(uint64_t a, uint32_t b) {
    uint64_t lo = (a & 0xFFFFFFFFull) * b;   // < 2^64
    uint64_t hi = (a >> 32) * b;             // < 2^61, weight 2^32
    // value = hi * 2^32 + lo ; split hi * 2^32 into 61-bit limbs
    uint64_t w0 = (hi << 32) & kP61;         // low 29 bits of hi, shifted
    uint64_t w1 = hi >> 29;                  // weight 2^61 = 1
    uint64_t s = (lo & kP61) + (lo >> 61) + w0 + w1;  // < 2^63
    s = (s & kP61) + (s >> 61);
    return s >= kP61 ? s - kP61 : s;
}

__device__ __forceinline__ uint64_t addmod_p61(uint64_t a, uint64_t b) {  // a, b < P
    uint64_t s = a + b;
    return s >= kP61 ? s - kP61 : s;
}

// t mod m for t < 2^64, m < 2^32 (mu = floor(2^64/m)): the quotient estimate is at most
// one too small, so one conditional subtract finishes it.
__device__ __forceinline__ uint32_t mod_m(uint64_t t, uint32_t m, uint64_t mu) {
    uint64_t q = __umul64hi(t, mu);
    uint64_t r = t - q * m;
    return (uint32_t)(r >= m ? r - m : r);
}

// Table of bag k.  Sample-major bags (k = n T + e): k mod T, by Lemire's fastmod with a 64-bit
// magic number for k < 2^32.  Table-major bags (k = e B + n, mp.B = B != 0): k / B, by the
// matching fastdiv.
__device__ __forceinline__ uint32_t table_of_bag(uint64_t k, const MapParams& mp) {
    if (mp.B != 0) {
        if (mp.B == 1) return (uint32_t)k;
        if (k >> 32) return (uint32_t)(k / mp.B);
        return (uint32_t)__umul64hi(mp.bmagic, k);
    }
    if (k >> 32) return (uint32_t)(k % mp.T);
    uint64_t low = mp.tmagic * (uint32_t)k;
    return (uint32_t)__umul64hi(low, (uint64_t)mp.T);
}

// (a * b) mod P, a < P, any b: ids below 2^32 (the common case) take the short product.
__device__ __forceinline__ uint64_t mulmod_p61_any(uint64_t a, uint64_t b) {
    return (b >> 32) == 0 ? mulmod_p61_u32(a, (uint32_t)b) : mulmod_p61(a, b);
}

// (A e + D) mod P : the part of the hash argument that depends on the table only.
__device__ __forceinline__ uint64_t table_term(const HashConsts& k, uint32_t e) {
    return addmod_p61(mulmod_p61_u32(k.A, e), k.D);
}

// (A e + B x + D) mod P : the part of the hash argument shared by all chunks of one id.
__device__ __forceinline__ uint64_t hash_base(const HashConsts& k, uint32_t e, uint64_t x) {
    uint64_t s = mulmod_p61_u32(k.A, e) + mulmod_p61(k.B, x) + k.D;  // < 3P < 2^63
    s = (s & kP61) + (s >> 61);
    return s >= kP61 ? s - kP61 : s;
}

// Block start h(e,x,c) given the base of (e,x).
__device__ __forceinline__ uint32_t block_start(const MapParams& mp, uint64_t base, uint32_t c) {
    uint64_t t = addmod_p61(base, mulmod_p61_u32(mp.h.C, c));
    return mod_m(t, mp.m, mp.mu);
}

// Start of block c of id x of table e, for every block size.  When R rows share one block
// (block size above d, Section 3.2 last paragraph) the block is hashed by (e, floor(x/R), 0) and
// row x is the piece that starts (x mod R) d slots into it.
__device__ __forceinline__ uint32_t id_block_start(const MapParams& mp, uint32_t e, uint64_t x,
                                                   uint32_t c) {
    if (mp.R > 1) {
        const uint64_t X = x / mp.R;
        const uint64_t j = (uint64_t)block_start(mp, hash_base(mp.h, e, X), 0) + (x - X * mp.R) * mp.d;
        return (uint32_t)(j >= mp.m ? j - mp.m : j);  // both terms are below m
    }
    return block_start(mp, hash_base(mp.h, e, x), c);
}

// Sign g(e,x,i) as +1.0f / -1.0f given the sign-hash base of (e,x).
__device__ __forceinline__ float sign_of(const MapParams& mp, uint64_t gbase, uint32_t i) {
    uint64_t t = addmod_p61(gbase, mulmod_p61_u32(mp.g.C, i));
    return (t & 1ull) ? 1.0f : -1.0f;
}

// chunk id and in-chunk offset of element i
__device__ __forceinline__ void chunk_of(const MapParams& mp, uint32_t i, uint32_t& c, uint32_t& o) {
    if (mp.log2Z != 0xFFFFFFFFu) {
        c = i >> mp.log2Z;
        o = i & (mp.Z - 1);
    } else {
        c = i / mp.Z;
        o = i - c * mp.Z;
    }
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) {
    return __uint_as_float((uint32_t)b << 16);
}

template <int DT>
__device__ __forceinline__ float load_elem(const void* array, uint32_t j) {
    if (DT == 0) return __ldg((const float*)array + j);
    return bf16_bits_to_float(__ldg((const unsigned short*)array + j));
}

// Array read of the gather kernels: read-only path, with the 64-byte L2 fetch hint.  Random
// Z-blocks gain nothing from the wider default fetch; measured on B200 this hint shortens a
// random 64-byte-block gather from a 1 GB array by about 13 %.
// L2 cache policy "keep": lines fetched under it are the last to be evicted.  For an array about
// the size of the L2 that shares it with gigabytes of streamed ids, output rows and gradients.
// 0 stands for "no policy" (createpolicy never returns 0 for evict_last).
__device__ __forceinline__ uint64_t l2_keep_policy(bool on) {
    uint64_t pol = 0;
    if (on) asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// fp32 reduction into global memory, with the L2 "keep" policy when pol != 0 (warp-uniform)
__device__ __forceinline__ void red_add(float* p, float v, uint64_t pol) {
    if (pol != 0)
        asm volatile("red.global.add.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
    else
        atomicAdd(p, v);
}

template <int DT>
__device__ __forceinline__ float gather_elem(const void* array, uint32_t j, uint64_t pol = 0) {
    if (pol != 0) {  // (warp-uniform)
        if (DT == 0) {
            float v;
            asm("ld.global.nc.L2::cache_hint.L2::64B.f32 %0, [%1], %2;"
                : "=f"(v)
                : "l"((const float*)array + j), "l"(pol));
            return v;
        }
        unsigned short b;
        asm("ld.global.nc.L2::cache_hint.L2::64B.u16 %0, [%1], %2;"
            : "=h"(b)
            : "l"((const unsigned short*)array + j), "l"(pol));
        return bf16_bits_to_float(b);
    }
    if (DT == 0) {
        float v;
        asm("ld.global.nc.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"((const float*)array + j));
        return v;
    }
    unsigned short b;
    asm("ld.global.nc.L2::64B.u16 %0, [%1];"
                 : "=h"(b)
                 : "l"((const unsigned short*)array + j));
    return bf16_bits_to_float(b);
}

}  // namespace robe
