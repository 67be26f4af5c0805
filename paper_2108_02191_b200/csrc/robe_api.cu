// C ABI of librobe.so: handle, options, argument checks, hash-constant draw, dispatch.
// The entry points are documented in include/robe.h.
#include <cmath>
#include <mutex>
#include <new>

#include "../../include/robe.h"
#include "robe_internal.h"

using namespace robe;

// Scratch of robe_backward_deterministic_static: part of the library image, so every device
// that loads the library holds these bytes until the process exits.  In host code this name
// is only a stand-in for the symbol; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char robe_static_scratch[ROBE_STATIC_SCRATCH_BYTES];

struct robe_ctx {
    uint64_t M;
    uint32_t Z, d, T;
    uint64_t consts[9];  // P, A_h, B_h, C_h, D_h, A_g, B_g, C_g, D_g
    MapParams mp;
    void* array;
    int dtype;
    int sign;
    int bwd_mode;
    int validate;
    int fwd_variant;
    int bwd_variant;
    int32_t* status_word;
    int index_type;
    int bag_layout;
    int l2_keep;
    // second stream of the deterministic backward, made at the first call that can use it
    bool side_tried;
    int side_device;  // the device the stream and events below belong to
    cudaStream_t side;
    cudaEvent_t fork_event, join_event;
};

namespace robe_api_detail {  // (named: the debug build compiles all sources as one translation unit)

// SplitMix64 (Steele, Lea, Flood): the stream the hash constants are drawn from.
uint64_t splitmix_next(uint64_t& s) {
    s += 0x9E3779B97F4A7C15ull;
    uint64_t z = s;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// Section 3.2: A_h, B_h, C_h in {1..P-1}, D_h in {0..P-1}; same ranges for the sign hash.
void draw_constants(uint64_t seed, uint64_t out[9]) {
    uint64_t s = seed;
    out[0] = kP61;
    for (int k = 1; k <= 8; ++k) {
        const bool additive = (k == 4 || k == 8);
        uint64_t v;
        do {
            v = splitmix_next(s) >> 3;
        } while (v >= kP61 || (!additive && v == 0));
        out[k] = v;
    }
}

__global__ void validate_kernel(IdList indices, const int64_t* offsets, int64_t nbags,
                                int64_t nnz, int32_t* status) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < nnz && indices.load(t) < 0) atomicCAS(status, ROBE_DEV_OK, ROBE_DEV_BAD_INDEX);
    if (offsets != nullptr && t <= nbags) {
        const int64_t o = offsets[t];
        bool bad = o < 0 || o > nnz;
        if (t == 0 && o != 0) bad = true;
        if (t == nbags && o != nnz) bad = true;
        if (t < nbags && offsets[t + 1] < o) bad = true;
        if (bad) atomicCAS(status, ROBE_DEV_OK, ROBE_DEV_BAD_OFFSETS);
    }
}

// status of a launch helper: a kernel variant that cannot take the call reports an invalid value
int launch_status(cudaError_t e) {
    if (e == cudaSuccess) return ROBE_OK;
    if (e == cudaErrorInvalidValue) return ROBE_ERR_UNSUPPORTED;
    (void)cudaGetLastError();
    return ROBE_ERR_CUDA;
}

bool check_sizes(robe_ctx* h, const void* indices, const int64_t* offsets, int64_t batch,
                 int64_t nnz) {
    if (h == nullptr || batch < 0 || nnz < 0) return false;
    if (nnz > 0 && indices == nullptr) return false;
    const int64_t nbags = batch * (int64_t)h->T;
    if (batch != 0 && nbags / batch != (int64_t)h->T) return false;  // overflow
    if (offsets == nullptr && nnz != nbags) return false;
    if (h->bag_layout == ROBE_BAGS_TABLE_MAJOR && batch >= (1ll << 32)) return false;  // B is kept in 32 bits
    return true;
}

Problem make_problem(robe_ctx* h, const void* indices, const int64_t* offsets, int64_t batch,
                     int64_t nnz) {
    Problem pb;
    pb.mp = h->mp;
    if (h->bag_layout == ROBE_BAGS_TABLE_MAJOR && batch > 0) {  // bag k belongs to table k / batch
        pb.mp.B = (uint32_t)batch;  // (below 2^32: checked with the other sizes)
        pb.mp.bmagic = 0xFFFFFFFFFFFFFFFFull / (uint64_t)batch + 1;
    }
    pb.array = h->array;
    pb.dtype = h->dtype;
    pb.sign = h->sign;
    pb.indices = IdList{indices, h->index_type == ROBE_I32 ? 1 : 0};
    pb.offsets = offsets;
    pb.nbags = batch * (int64_t)h->T;
    pb.nnz = nnz;
    pb.status = (h->validate && h->status_word) ? h->status_word : nullptr;
    pb.l2_keep = 0;  // (the backward calls set it)
    return pb;
}

// The deterministic backward runs its two apply kernels side by side: the one that walks often
// repeated ids (few CTAs, long) in a stream of higher priority, forked from and joined to the
// caller's stream by events.  Made once per handle; if that fails the kernels run one after the
// other in the caller's stream.
void lend_side_stream(robe_ctx* h, Problem& pb) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return;
    }
    if (!h->side_tried) {
        h->side_tried = true;
        h->side_device = dev;
        int least = 0, greatest = 0;
        cudaStream_t s = nullptr;
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        if (cudaDeviceGetStreamPriorityRange(&least, &greatest) == cudaSuccess &&
            cudaStreamCreateWithPriority(&s, cudaStreamNonBlocking, greatest) == cudaSuccess &&
            cudaEventCreateWithFlags(&e0, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) == cudaSuccess) {
            h->side = s;
            h->fork_event = e0;
            h->join_event = e1;
        } else {
            if (e0 != nullptr) cudaEventDestroy(e0);
            if (s != nullptr) cudaStreamDestroy(s);
            (void)cudaGetLastError();
        }
    }
    // a stream belongs to the device it was made on: a call made with another device current
    // runs everything in the caller's stream
    if (dev != h->side_device) return;
    pb.side = h->side;
    pb.fork_event = h->fork_event;
    pb.join_event = h->join_event;
}

// Size limits of the sort-based backward variants (binned, deterministic, Adam): block numbers,
// bag numbers and positions in grad_out are 32-bit, and the binned adds run one thread per
// (block, offset) on a one-dimensional grid.
bool sorted_path_fits(const robe_ctx* h, const Problem& pb) {
    const uint64_t nb = (uint64_t)pb.nnz * h->mp.C;
    uint32_t zp = 1;
    while (zp < h->mp.Z) zp <<= 1;
    if (nb >= (1ull << 32) || (uint64_t)pb.nbags >= (1ull << 32)) return false;
    if (nb * zp / 256 >= (1ull << 31)) return false;
    return (uint64_t)pb.nbags * h->mp.d <= (1ull << 32);
}

}  // namespace robe_api_detail
using namespace robe_api_detail;

namespace robe {
cudaError_t launch_validate(const Problem& pb, cudaStream_t st) {
    if (pb.status == nullptr) return cudaSuccess;
    const int64_t n = (pb.nnz > pb.nbags + 1 ? pb.nnz : pb.nbags + 1);
    validate_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(pb.indices, pb.offsets, pb.nbags,
                                                                 pb.nnz, pb.status);
    return cudaGetLastError();
}
}  // namespace robe

extern "C" {

int robe_create(robe_handle_t* out, uint64_t M, uint32_t Z, uint32_t d, uint32_t num_tables,
                uint64_t hash_seed) {
    if (out == nullptr) return ROBE_ERR_INVALID_ARG;
    *out = nullptr;
    if (M == 0 || Z == 0 || d == 0 || num_tables == 0) return ROBE_ERR_INVALID_ARG;
    if ((uint64_t)d > M) return ROBE_ERR_INVALID_ARG;
    if (Z > d && (Z % d != 0 || (uint64_t)Z > M)) return ROBE_ERR_INVALID_ARG;
    if (d > 32768u) return ROBE_ERR_INVALID_ARG;
    if (M + (uint64_t)d > (1ull << 32)) return ROBE_ERR_INVALID_ARG;
    robe_ctx* h = new (std::nothrow) robe_ctx();
    if (h == nullptr) return ROBE_ERR_INVALID_ARG;
    h->M = M;
    h->Z = Z;
    h->d = d;
    h->T = num_tables;
    draw_constants(hash_seed, h->consts);
    MapParams& mp = h->mp;
    mp.h = HashConsts{h->consts[1], h->consts[2], h->consts[3], h->consts[4]};
    mp.g = HashConsts{h->consts[5], h->consts[6], h->consts[7], h->consts[8]};
    mp.m = (uint32_t)M;
    mp.mu = (M == 1) ? ~0ull : (uint64_t)((((unsigned __int128)1) << 64) / M);
    mp.T = num_tables;
    mp.d = d;
    // Z > d: Z/d rows share one block; every kernel then sees one block of d elements per id
    const uint32_t Zb = Z > d ? d : Z;
    mp.Z = Zb;
    mp.R = Z > d ? Z / d : 1;
    mp.C = (d + Zb - 1) / Zb;
    mp.log2Z = 0xFFFFFFFFu;
    if ((Zb & (Zb - 1)) == 0) {
        uint32_t l = 0;
        while ((1u << l) < Zb) ++l;
        mp.log2Z = l;
    }
    mp.tmagic = 0xFFFFFFFFFFFFFFFFull / num_tables + 1;
    mp.bmagic = 0;
    mp.B = 0;
    h->array = nullptr;
    h->dtype = ROBE_F32;
    h->sign = 0;
    h->bwd_mode = ROBE_BWD_ATOMIC;
    h->validate = 0;
    h->fwd_variant = 0;
    h->bwd_variant = 0;
    h->status_word = nullptr;
    h->index_type = ROBE_I64;
    h->bag_layout = ROBE_BAGS_SAMPLE_MAJOR;
    h->l2_keep = 0;
    h->side_tried = false;
    h->side_device = -1;
    h->side = nullptr;
    h->fork_event = h->join_event = nullptr;
    *out = h;
    return ROBE_OK;
}

int robe_destroy(robe_handle_t h) {
    if (h == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->side != nullptr) {
        cudaStreamSynchronize(h->side);
        cudaStreamDestroy(h->side);
        cudaEventDestroy(h->fork_event);
        cudaEventDestroy(h->join_event);
    }
    delete h;
    return ROBE_OK;
}

int robe_set_option(robe_handle_t h, int key, int64_t value) {
    if (h == nullptr) return ROBE_ERR_INVALID_ARG;
    switch (key) {
        case ROBE_OPT_SIGN:
            if (value != 0 && value != 1) return ROBE_ERR_INVALID_ARG;
            h->sign = (int)value;
            return ROBE_OK;
        case ROBE_OPT_BWD_MODE:
            if (value != ROBE_BWD_ATOMIC && value != ROBE_BWD_DETERMINISTIC && value != ROBE_BWD_BINNED)
                return ROBE_ERR_INVALID_ARG;
            h->bwd_mode = (int)value;
            return ROBE_OK;
        case ROBE_OPT_VALIDATE:
            if (value != 0 && value != 1) return ROBE_ERR_INVALID_ARG;
            h->validate = (int)value;
            return ROBE_OK;
        case ROBE_OPT_FWD_KERNEL:
            if (value < 0 || value > 4) return ROBE_ERR_INVALID_ARG;
            h->fwd_variant = (int)value;
            return ROBE_OK;
        case ROBE_OPT_INDEX_TYPE:
            if (value != ROBE_I64 && value != ROBE_I32) return ROBE_ERR_INVALID_ARG;
            h->index_type = (int)value;
            return ROBE_OK;
        case ROBE_OPT_BAG_LAYOUT:
            if (value != ROBE_BAGS_SAMPLE_MAJOR && value != ROBE_BAGS_TABLE_MAJOR) return ROBE_ERR_INVALID_ARG;
            h->bag_layout = (int)value;
            return ROBE_OK;
        case ROBE_OPT_ARRAY_L2_KEEP:
            if (value != 0 && value != 1) return ROBE_ERR_INVALID_ARG;
            h->l2_keep = (int)value;
            return ROBE_OK;
        case ROBE_OPT_BWD_KERNEL:
            if (value < 0 || value > 6) return ROBE_ERR_INVALID_ARG;
            h->bwd_variant = (int)value;
            return ROBE_OK;
        default:
            return ROBE_ERR_INVALID_ARG;
    }
}

int robe_attach_array(robe_handle_t h, void* dev_array, int dtype) {
    if (h == nullptr || dev_array == nullptr) return ROBE_ERR_INVALID_ARG;
    if (dtype != ROBE_F32 && dtype != ROBE_BF16) return ROBE_ERR_INVALID_ARG;
    if (((uintptr_t)dev_array & 15u) != 0) return ROBE_ERR_INVALID_ARG;
    h->array = dev_array;
    h->dtype = dtype;
    return ROBE_OK;
}

int robe_get_hash_constants(robe_handle_t h, uint64_t out[9]) {
    if (h == nullptr || out == nullptr) return ROBE_ERR_INVALID_ARG;
    for (int k = 0; k < 9; ++k) out[k] = h->consts[k];
    return ROBE_OK;
}

int robe_set_status_word(robe_handle_t h, int32_t* dev_word) {
    if (h == nullptr) return ROBE_ERR_INVALID_ARG;
    h->status_word = dev_word;
    return ROBE_OK;
}

int robe_last_device_status(robe_handle_t h, void* stream) {
    if (h == nullptr || h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    int32_t v = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&v, h->status_word, sizeof v, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ROBE_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ROBE_ERR_CUDA;
    return (int)v;
}

int robe_forward(robe_handle_t h, const void* indices, const int64_t* offsets, int64_t batch,
                 int64_t nnz, float* out, void* stream) {
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    const Problem pb = make_problem(h, indices, offsets, batch, nnz);
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    return launch_status(launch_forward(pb, out, h->fwd_variant, st));
}

int robe_forward_keep(robe_handle_t h, const void* indices, const int64_t* offsets, int64_t batch,
                      int64_t nnz, float* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (h != nullptr && h->bwd_mode == ROBE_BWD_ATOMIC)  // that backward sorts nothing
        return robe_forward(h, indices, offsets, batch, nnz, out, stream);
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    const Problem pb = make_problem(h, indices, offsets, batch, nnz);
    if (!sorted_path_fits(h, pb)) return ROBE_ERR_UNSUPPORTED;
    const size_t need = det_workspace_bytes(h->mp, pb.nbags, nnz, offsets != nullptr);
    if (nnz > 0 && (workspace == nullptr || workspace_bytes < need)) return ROBE_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return ROBE_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    uint32_t *keys = nullptr, *vals = nullptr;
    if (nnz > 0 && batch > 0) block_key_buffers(pb, workspace, &keys, &vals);
    bool kept = false;
    const int frc = launch_status(launch_forward(pb, out, h->fwd_variant, st, keys, vals, &kept));
    if (frc != ROBE_OK) return frc;
    // a forward kernel that keeps nothing (rows longer than 128): the backward's own key kernels
    if (!kept && launch_block_keys(pb, workspace, workspace_bytes, st) != cudaSuccess) return ROBE_ERR_CUDA;
    return ROBE_OK;
}

size_t robe_backward_workspace_bytes(robe_handle_t h, int64_t batch, int64_t nnz) {
    if (h == nullptr || batch < 0 || nnz < 0) return 0;
    if (h->bwd_mode == ROBE_BWD_ATOMIC) return 0;
    // the pooled layout is the larger of the two; a caller may size once for both
    return det_workspace_bytes(h->mp, batch * (int64_t)h->T, nnz, true);
}

static int backward_any(robe_handle_t h, const float* grad_out, const void* indices,
                        const int64_t* offsets, int64_t batch, int64_t nnz, float* grad_array, float lr,
                        void* workspace, size_t workspace_bytes, void* stream, bool keys_kept) {
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && grad_out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    const bool sgd = grad_array == nullptr;
    if (sgd) {
        if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
        if (h->dtype != ROBE_F32) return ROBE_ERR_INVALID_ARG;
    }
    float* target = sgd ? (float*)h->array : grad_array;
    Problem pb = make_problem(h, indices, offsets, batch, nnz);
    pb.l2_keep = h->l2_keep == 0 ? 1 : 0;  // the reductions of the atomic and the binned backward
    cudaStream_t st = (cudaStream_t)stream;
    if (h->bwd_mode == ROBE_BWD_ATOMIC) {
        if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
        return launch_status(launch_backward_atomic(pb, grad_out, target, sgd ? -lr : 1.0f, h->bwd_variant, st));
    }
    // the sort-based variants (binned, deterministic)
    if (!sorted_path_fits(h, pb)) return ROBE_ERR_UNSUPPORTED;
    const size_t need = det_workspace_bytes(h->mp, pb.nbags, nnz, offsets != nullptr);
    if (nnz > 0 && (workspace == nullptr || workspace_bytes < need)) return ROBE_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return ROBE_ERR_WORKSPACE;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    const bool binned = h->bwd_mode == ROBE_BWD_BINNED;
    if (!binned) lend_side_stream(h, pb);
    if (launch_backward_det(pb, grad_out, target, binned ? 3 : (sgd ? 1 : 0),
                            binned ? (sgd ? -lr : 1.0f) : lr, nullptr, workspace, workspace_bytes,
                            st, keys_kept) != cudaSuccess)
        return ROBE_ERR_CUDA;
    return ROBE_OK;
}

int robe_backward(robe_handle_t h, const float* grad_out, const void* indices,
                  const int64_t* offsets, int64_t batch, int64_t nnz, float* grad_array, float lr,
                  void* workspace, size_t workspace_bytes, void* stream) {
    return backward_any(h, grad_out, indices, offsets, batch, nnz, grad_array, lr, workspace,
                        workspace_bytes, stream, false);
}

int robe_backward_kept(robe_handle_t h, const float* grad_out, const void* indices,
                       const int64_t* offsets, int64_t batch, int64_t nnz, float* grad_array, float lr,
                       void* workspace, size_t workspace_bytes, void* stream) {
    return backward_any(h, grad_out, indices, offsets, batch, nnz, grad_array, lr, workspace,
                        workspace_bytes, stream, true);
}

// Device address of robe_static_scratch on the current device, looked up once per device.
static int static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* addr[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return ROBE_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ROBE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, robe_static_scratch) != cudaSuccess || p == nullptr)
            return ROBE_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return ROBE_OK;
}

int robe_backward_deterministic_static(robe_handle_t h, const float* grad_out,
                                       const void* indices, const int64_t* offsets,
                                       int64_t batch, int64_t nnz, float* grad_array, float lr,
                                       void* stream) {
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && grad_out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    const bool sgd = grad_array == nullptr;
    if (sgd) {
        if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
        if (h->dtype != ROBE_F32) return ROBE_ERR_INVALID_ARG;
    }
    float* target = sgd ? (float*)h->array : grad_array;
    Problem pb = make_problem(h, indices, offsets, batch, nnz);
    if (!sorted_path_fits(h, pb)) return ROBE_ERR_UNSUPPORTED;
    // the fixed array is the whole workspace: a call that needs more is refused up front (by
    // the same figure robe_backward_workspace_bytes reports, which covers pooled input too)
    const size_t need = det_workspace_bytes(h->mp, pb.nbags, nnz, true);
    if (need > (size_t)ROBE_STATIC_SCRATCH_BYTES) return ROBE_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != ROBE_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    // Stale contents are harmless: keys, values and digit counters are fully rewritten before
    // they are read, and the one buffer that must start from zero (the bag number of each id,
    // pooled input only) is cleared by the launch itself on the same stream.
    if (launch_backward_det(pb, grad_out, target, sgd ? 1 : 0, lr, nullptr, scratch,
                            (size_t)ROBE_STATIC_SCRATCH_BYTES, st) != cudaSuccess)
        return ROBE_ERR_CUDA;
    return ROBE_OK;
}

int robe_backward_adam(robe_handle_t h, const float* grad_out, const void* indices,
                       const int64_t* offsets, int64_t batch, int64_t nnz, float* m1, float* m2,
                       float lr, float beta1, float beta2, float eps, int64_t step, void* workspace,
                       size_t workspace_bytes, void* stream) {
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && grad_out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (m1 == nullptr || m2 == nullptr || step < 1) return ROBE_ERR_INVALID_ARG;
    if (!(beta1 >= 0.0f && beta1 < 1.0f && beta2 >= 0.0f && beta2 < 1.0f && eps >= 0.0f))
        return ROBE_ERR_INVALID_ARG;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
    if (h->dtype != ROBE_F32) return ROBE_ERR_INVALID_ARG;
    Problem pb = make_problem(h, indices, offsets, batch, nnz);
    if (!sorted_path_fits(h, pb)) return ROBE_ERR_UNSUPPORTED;
    const size_t need = det_workspace_bytes(h->mp, pb.nbags, nnz, offsets != nullptr);
    if (nnz > 0 && (workspace == nullptr || workspace_bytes < need)) return ROBE_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return ROBE_ERR_WORKSPACE;
    lend_side_stream(h, pb);
    AdamState ad;
    ad.m1 = m1;
    ad.m2 = m2;
    ad.beta1 = beta1;
    ad.beta2 = beta2;
    ad.eps = eps;
    ad.bias1 = (float)(1.0 - pow((double)beta1, (double)step));
    ad.bias2 = (float)(1.0 - pow((double)beta2, (double)step));
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    if (launch_backward_det(pb, grad_out, (float*)h->array, 2, lr, &ad, workspace, workspace_bytes,
                            st) != cudaSuccess)
        return ROBE_ERR_CUDA;
    return ROBE_OK;
}

int robe_backward_adagrad(robe_handle_t h, const float* grad_out, const void* indices,
                          const int64_t* offsets, int64_t batch, int64_t nnz, float* sum_sq, float lr,
                          float eps, void* workspace, size_t workspace_bytes, void* stream) {
    if (!check_sizes(h, indices, offsets, batch, nnz)) return ROBE_ERR_INVALID_ARG;
    if (batch > 0 && grad_out == nullptr) return ROBE_ERR_INVALID_ARG;
    if (sum_sq == nullptr || !(eps >= 0.0f)) return ROBE_ERR_INVALID_ARG;
    if (h->validate && h->status_word == nullptr) return ROBE_ERR_INVALID_ARG;
    if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
    if (h->dtype != ROBE_F32) return ROBE_ERR_INVALID_ARG;
    Problem pb = make_problem(h, indices, offsets, batch, nnz);
    if (!sorted_path_fits(h, pb)) return ROBE_ERR_UNSUPPORTED;
    const size_t need = det_workspace_bytes(h->mp, pb.nbags, nnz, offsets != nullptr);
    if (nnz > 0 && (workspace == nullptr || workspace_bytes < need)) return ROBE_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return ROBE_ERR_WORKSPACE;
    lend_side_stream(h, pb);
    AdamState ad{};
    ad.m2 = sum_sq;
    ad.eps = eps;
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_validate(pb, st) != cudaSuccess) return ROBE_ERR_CUDA;
    if (launch_backward_det(pb, grad_out, (float*)h->array, 4, lr, &ad, workspace, workspace_bytes, st) !=
        cudaSuccess)
        return ROBE_ERR_CUDA;
    return ROBE_OK;
}

int robe_apply_sgd(robe_handle_t h, float* grad_array, float lr, int zero_grad, void* stream) {
    if (h == nullptr || grad_array == nullptr) return ROBE_ERR_INVALID_ARG;
    if (zero_grad != 0 && zero_grad != 1) return ROBE_ERR_INVALID_ARG;
    if (h->array == nullptr) return ROBE_ERR_NO_ARRAY;
    if (h->dtype != ROBE_F32) return ROBE_ERR_INVALID_ARG;
    if (((uintptr_t)grad_array & 15u) != 0) return ROBE_ERR_INVALID_ARG;
    if (launch_dense_sgd_apply((float*)h->array, grad_array, h->M, lr, zero_grad != 0,
                               (cudaStream_t)stream) != cudaSuccess)
        return ROBE_ERR_CUDA;
    return ROBE_OK;
}

#ifdef ROBE_DEBUG
namespace robe_api_detail {
__global__ void debug_selftest_kernel() { (void)ROBE_CHK(threadIdx.x > 31u, ROBE_DBG_SELFTEST); }
}  // namespace robe_api_detail
#endif

int robe_debug_status(void* stream) {
#ifdef ROBE_DEBUG
    cudaStream_t st = (cudaStream_t)stream;
    int32_t code = 0;
    const int32_t zero = 0;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ROBE_ERR_CUDA;
    if (cudaMemcpyFromSymbol(&code, g_robe_debug_code, sizeof code) != cudaSuccess) return ROBE_ERR_CUDA;
    if (cudaMemcpyToSymbol(g_robe_debug_code, &zero, sizeof zero) != cudaSuccess) return ROBE_ERR_CUDA;
    return (int)code;
#else
    (void)stream;
    return ROBE_ERR_UNSUPPORTED;
#endif
}

int robe_debug_selftest(void* stream) {
#ifdef ROBE_DEBUG
    debug_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>();
    return cudaGetLastError() == cudaSuccess ? ROBE_OK : ROBE_ERR_CUDA;
#else
    (void)stream;
    return ROBE_ERR_UNSUPPORTED;
#endif
}

const char* robe_status_string(int status) {
    switch (status) {
        case ROBE_OK: return "ok";
        case ROBE_ERR_INVALID_ARG: return "invalid argument";
        case ROBE_ERR_NO_ARRAY: return "no array attached";
        case ROBE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case ROBE_ERR_CUDA: return "CUDA runtime error at launch";
        case ROBE_ERR_UNSUPPORTED: return "size not supported by this build";
        default: return "unknown status";
    }
}

}  // extern "C"
