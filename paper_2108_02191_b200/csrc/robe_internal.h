// Host-side declarations shared by the translation units of librobe.so.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "robe_device.cuh"

namespace robe {

struct Problem {
    MapParams mp;
    const void* array;       // device, M elements
    int dtype;               // 0 fp32, 1 bf16
    int sign;                // 0 / 1
    IdList indices;          // device [nnz], int64 or int32
    const int64_t* offsets;  // device [nbags+1] or nullptr (one-hot)
    int64_t nbags;           // batch * T
    int64_t nnz;
    int32_t* status;         // device status word or nullptr (validation off)
    int l2_keep = 0;         // 1: array reads (forward) and reductions (atomic backward) carry the L2 "keep" policy
    // deterministic backward: a second stream of higher priority with the two events that fork
    // it from and join it to the caller's stream, or all nullptr (everything in the caller's)
    cudaStream_t side = nullptr;
    cudaEvent_t fork_event = nullptr;
    cudaEvent_t join_event = nullptr;
};

// forward: out [nbags, d].  With keep_keys/keep_vals (device, one word per block each) the staged
// kernel also stores every block's start and payload as the sort-based backward wants them;
// *kept says whether the kernel that ran did so.
cudaError_t launch_forward(const Problem& pb, float* out, int variant, cudaStream_t st,
                           uint32_t* keep_keys = nullptr, uint32_t* keep_vals = nullptr,
                           bool* kept = nullptr);

// atomic backward: adds scale * g * grad_out into target (fp32 [M])
cudaError_t launch_backward_atomic(const Problem& pb, const float* grad_out, float* target,
                                   float scale, int variant, cudaStream_t st);

// deterministic backward
size_t det_workspace_bytes(const MapParams& mp, int64_t nbags, int64_t nnz, bool bags);
// Adam moments and constants of the deterministic backward's update mode 2
struct AdamState {
    float* m1;     // device [M], first moment
    float* m2;     // device [M], second moment
    float beta1, beta2, eps;
    float bias1;   // 1 - beta1^t
    float bias2;   // 1 - beta2^t
};

// mode 0: target[j] += delta; 1: target = attached array, target[j] = fma(-lr, delta, target[j]);
// 2: Adam step on the attached array with the moments in *adam; 4: Adagrad step on the attached
// array with the accumulators in adam->m2 and adam->eps; 3: binned atomic adds of
// lr * delta terms into target (one sort pass on the top key bits, then red.global in bin order)
// keys_kept: the workspace already holds the block starts and payloads of these ids (left by
// launch_forward or launch_block_keys), so they are not computed again.
cudaError_t launch_backward_det(const Problem& pb, const float* grad_out, float* target, int mode,
                                float lr, const AdamState* adam, void* workspace,
                                size_t workspace_bytes, cudaStream_t st, bool keys_kept = false);
// where in a workspace of the sort-based backward the block starts and payloads go
void block_key_buffers(const Problem& pb, void* workspace, uint32_t** keys, uint32_t** vals);
// block starts and payloads of pb's ids into the workspace (what the backward does first)
cudaError_t launch_block_keys(const Problem& pb, void* workspace, size_t workspace_bytes,
                              cudaStream_t st);

// dense SGD apply of the data-parallel step: array[j] = fma(-lr, grad[j], array[j]) for j < m,
// grad zeroed afterwards when zero_grad
cudaError_t launch_dense_sgd_apply(float* array, float* grad, uint64_t m, float lr, bool zero_grad,
                                   cudaStream_t st);

// id / offset range check into the status word
cudaError_t launch_validate(const Problem& pb, cudaStream_t st);

}  // namespace robe
