// Dense SGD apply of the data-parallel training step (Section 1 of the paper: the compressed
// model fits every GPU, so the step is plain data-parallel and what the ranks exchange is one
// gradient the size of the array).  Every rank scatter-adds its shard's output gradients into a
// dense fp32 gradient (robe_backward), the ranks sum those gradients, and this kernel applies the
// sum:  M[j] <- fma(-lr, g[j], M[j])  for every slot j, optionally leaving g zeroed for the next
// step.  One streaming pass: 8 bytes read and 4 (8 with the zeroing) written per slot.
#include "robe_internal.h"

namespace robe {

namespace {

constexpr int kApplyThreads = 256;
constexpr int kApplyVecPerThread = 4;  // float4 pairs in flight per thread

template <bool ZERO>
__global__ void __launch_bounds__(kApplyThreads)
dense_sgd_apply_kernel(float* __restrict__ array, float* __restrict__ grad, uint64_t m, float lr) {
    const uint64_t nvec = m >> 2;
    float4* a4 = reinterpret_cast<float4*>(array);
    float4* g4 = reinterpret_cast<float4*>(grad);
    const uint64_t stride = (uint64_t)gridDim.x * kApplyThreads;
    uint64_t v = (uint64_t)blockIdx.x * kApplyThreads + threadIdx.x;
    const float nlr = -lr;
    // kApplyVecPerThread independent 16-byte loads of each stream before the first store
    for (; v + (kApplyVecPerThread - 1) * stride < nvec; v += kApplyVecPerThread * stride) {
        float4 a[kApplyVecPerThread], g[kApplyVecPerThread];
#pragma unroll
        for (int t = 0; t < kApplyVecPerThread; ++t) {
            a[t] = a4[v + t * stride];
            g[t] = __ldcs(g4 + v + t * stride);
        }
#pragma unroll
        for (int t = 0; t < kApplyVecPerThread; ++t) {
            a[t].x = __fmaf_rn(nlr, g[t].x, a[t].x);
            a[t].y = __fmaf_rn(nlr, g[t].y, a[t].y);
            a[t].z = __fmaf_rn(nlr, g[t].z, a[t].z);
            a[t].w = __fmaf_rn(nlr, g[t].w, a[t].w);
            a4[v + t * stride] = a[t];
            if (ZERO) __stcs(g4 + v + t * stride, make_float4(0.0f, 0.0f, 0.0f, 0.0f));
        }
    }
    for (; v < nvec; v += stride) {
        float4 a = a4[v];
        const float4 g = __ldcs(g4 + v);
        a.x = __fmaf_rn(nlr, g.x, a.x);
        a.y = __fmaf_rn(nlr, g.y, a.y);
        a.z = __fmaf_rn(nlr, g.z, a.z);
        a.w = __fmaf_rn(nlr, g.w, a.w);
        a4[v] = a;
        if (ZERO) __stcs(g4 + v, make_float4(0.0f, 0.0f, 0.0f, 0.0f));
    }
    // the last m mod 4 slots
    const uint64_t t = (uint64_t)blockIdx.x * kApplyThreads + threadIdx.x;
    const uint64_t j = (nvec << 2) + t;
    if (t < 4 && j < m) {
        array[j] = __fmaf_rn(nlr, grad[j], array[j]);
        if (ZERO) grad[j] = 0.0f;
    }
}

}  // namespace

cudaError_t launch_dense_sgd_apply(float* array, float* grad, uint64_t m, float lr, bool zero_grad,
                                   cudaStream_t st) {
    if (m == 0) return cudaSuccess;
    // a few waves of CTAs over the SMs of the current device; the loop strides over the rest
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess)
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    (void)cudaGetLastError();
    const uint64_t nvec = m >> 2;
    uint64_t want = (nvec + (uint64_t)kApplyThreads * kApplyVecPerThread - 1) /
                    ((uint64_t)kApplyThreads * kApplyVecPerThread);
    const uint64_t cap = (uint64_t)sms * 8;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (zero_grad)
        dense_sgd_apply_kernel<true><<<(unsigned)want, kApplyThreads, 0, st>>>(array, grad, m, lr);
    else
        dense_sgd_apply_kernel<false><<<(unsigned)want, kApplyThreads, 0, st>>>(array, grad, m, lr);
    return cudaGetLastError();
}

}  // namespace robe
