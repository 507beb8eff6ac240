// Optimiser-side kernels of the update: fused Adam step (fp32 master weights and moments, optional
// bf16 copy written straight into a policy's padded weight matrix), global-norm gradient scale and
// the KL-adaptive learning rate.  Learning rate and gradient scale are device scalars, so a whole
// update (loss -> gradients -> scale -> Adam -> new learning rate) runs without the host reading
// anything back (the paper's Section 4.2 rule applied to the update phase).
//
//   g = grad * grad_scale;  m = b1 m + (1 - b1) g;  v = b2 v + (1 - b2) g^2
//   param -= lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)
//
// Streams 28 (+2) bytes per parameter; four parameters per thread with 16-byte accesses when the
// tensors allow it.
#include <cmath>
#include <cuda_bf16.h>

#include "im_internal.h"

namespace im {

namespace {

struct AdamParams {
    float *param, *m, *v;
    const float *grad;
    const float *lr, *grad_scale;          // device scalars (grad_scale may be null: 1)
    long long n;
    float b1, b2, eps, inv_c1, inv_c2;     // inv_c = 1 / (1 - b^t)
    __nv_bfloat16 *bf16_out;               // optional copy: element (r, c) of the [rows][cols] tensor at r * ld_bf16 + c
    int cols, ld_bf16;
};

__device__ __forceinline__ float adam_one(const AdamParams &P, float lr, float gs, float p, float g, float &m, float &v)
{
    g *= gs;
    m = fmaf(P.b1, m, (1.0f - P.b1) * g);
    v = fmaf(P.b2, v, (1.0f - P.b2) * g * g);
    return p - lr * (m * P.inv_c1) / (sqrtf(v * P.inv_c2) + P.eps);
}

__device__ __forceinline__ void store_bf16(const AdamParams &P, long long i, float x)
{
    if (!P.bf16_out) return;
    const long long r = i / P.cols, c = i - r * P.cols;
    P.bf16_out[r * P.ld_bf16 + c] = __float2bfloat16_rn(x);
}

template <bool VEC4>
__global__ void __launch_bounds__(256) adam_kernel(const AdamParams P)
{
    const float lr = __ldg(P.lr), gs = P.grad_scale ? __ldg(P.grad_scale) : 1.0f;
    const long long stride = (long long)gridDim.x * blockDim.x;
    if (VEC4) {
        const long long n4 = P.n >> 2;
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
            const float4 p = reinterpret_cast<const float4 *>(P.param)[i], g = __ldg(reinterpret_cast<const float4 *>(P.grad) + i);
            float4 m = reinterpret_cast<const float4 *>(P.m)[i], v = reinterpret_cast<const float4 *>(P.v)[i];
            float4 q;
            q.x = adam_one(P, lr, gs, p.x, g.x, m.x, v.x);
            q.y = adam_one(P, lr, gs, p.y, g.y, m.y, v.y);
            q.z = adam_one(P, lr, gs, p.z, g.z, m.z, v.z);
            q.w = adam_one(P, lr, gs, p.w, g.w, m.w, v.w);
            reinterpret_cast<float4 *>(P.param)[i] = q;
            reinterpret_cast<float4 *>(P.m)[i] = m;
            reinterpret_cast<float4 *>(P.v)[i] = v;
            store_bf16(P, 4 * i, q.x); store_bf16(P, 4 * i + 1, q.y); store_bf16(P, 4 * i + 2, q.z); store_bf16(P, 4 * i + 3, q.w);
        }
    } else {
        for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < P.n; i += stride) {
            float m = P.m[i], v = P.v[i];
            const float q = adam_one(P, lr, gs, P.param[i], __ldg(P.grad + i), m, v);
            P.param[i] = q; P.m[i] = m; P.v[i] = v;
            store_bf16(P, i, q);
        }
    }
}

// ---- global gradient norm -> scale
constexpr int kSqThreads = 256;
constexpr int kSqMaxGrid = 64;             // partial sums per tensor

// Sum of squares of up to kSqMaxTensors tensors in one launch.  Tensor k owns blocks [first[k], first[k+1]) of the
// grid and as many partial sums; a block adds its grid-strided share of the tensor in double precision.
constexpr int kSqMaxTensors = 64;
struct SumSqArgs {
    const float *x[kSqMaxTensors];
    long long n[kSqMaxTensors];
    int first[kSqMaxTensors + 1];
    int n_tensors;
};

__global__ void __launch_bounds__(kSqThreads) sumsq_kernel(const __grid_constant__ SumSqArgs a, double *__restrict__ partial)
{
    __shared__ double s[kSqThreads];
    int k = 0;
    while (k + 1 < a.n_tensors && (int)blockIdx.x >= a.first[k + 1]) ++k;
    const float *__restrict__ x = a.x[k];
    const long long n = a.n[k];
    const int blocks = a.first[k + 1] - a.first[k], blk = (int)blockIdx.x - a.first[k];
    double q = 0.0;
    for (long long i = (long long)blk * kSqThreads + threadIdx.x; i < n; i += (long long)blocks * kSqThreads) {
        const double v = (double)__ldg(x + i);
        q = fma(v, v, q);
    }
    s[threadIdx.x] = q;
    __syncthreads();
    for (int o = kSqThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) partial[blockIdx.x] = s[0];
}

// One warp: lane l adds partials l, l + 32, ... in order, then a fixed butterfly.
__global__ void __launch_bounds__(32) grad_scale_finish_kernel(const double *__restrict__ partial, int count, float max_norm,
                                                               float *__restrict__ scale_out)
{
    double q = 0.0;
    for (int i = threadIdx.x; i < count; i += 32) q += partial[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    if (threadIdx.x == 0) {
        const double s = (double)max_norm / (sqrt(q) + 1e-6);
        scale_out[0] = (float)(s < 1.0 ? s : 1.0);
        scale_out[1] = (float)sqrt(q);
    }
}

__global__ void adaptive_lr_kernel(float *lr, const float *kl, float kl_target, float lr_min, float lr_max)
{
    const float k = *kl;
    float x = *lr;
    if (k > 2.0f * kl_target) x = fmaxf(x / 1.5f, lr_min);
    else if (k > 0.0f && k < 0.5f * kl_target) x = fminf(x * 1.5f, lr_max);
    *lr = x;
}

}  // namespace

}  // namespace im

extern "C" {

im_status im_adam_step(const im_adam_config *cfg, int32_t t, int64_t n, float *param, const float *grad, float *m,
                       float *v, const float *lr, const float *grad_scale, uint16_t *bf16_out, int32_t cols,
                       int32_t ld_bf16, void *cuda_stream)
{
    using namespace im;
    if (!cfg || !param || !grad || !m || !v || !lr || n < 1 || t < 1) return IM_ERR_INVALID_ARG;
    if (!(cfg->beta1 >= 0.0f && cfg->beta1 < 1.0f) || !(cfg->beta2 >= 0.0f && cfg->beta2 < 1.0f) || !(cfg->eps > 0.0f))
        return IM_ERR_INVALID_ARG;
    if (bf16_out && (cols < 1 || ld_bf16 < cols || n % cols != 0)) return IM_ERR_INVALID_ARG;
    AdamParams p;
    p.param = param; p.m = m; p.v = v; p.grad = grad; p.lr = lr; p.grad_scale = grad_scale; p.n = n;
    p.b1 = cfg->beta1; p.b2 = cfg->beta2; p.eps = cfg->eps;
    p.inv_c1 = (float)(1.0 / (1.0 - std::pow((double)cfg->beta1, (double)t)));
    p.inv_c2 = (float)(1.0 / (1.0 - std::pow((double)cfg->beta2, (double)t)));
    p.bf16_out = reinterpret_cast<__nv_bfloat16 *>(bf16_out);
    p.cols = bf16_out ? cols : 1; p.ld_bf16 = ld_bf16;
    const auto al16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
    const bool vec = (n % 4 == 0) && al16(param) && al16(grad) && al16(m) && al16(v);
    const long long work = vec ? n / 4 : n;
    long long g = (work + 255) / 256;
    const int grid = (int)(g > 148 * 8 ? 148 * 8 : g);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (vec) adam_kernel<true><<<grid, 256, 0, st>>>(p);
    else adam_kernel<false><<<grid, 256, 0, st>>>(p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_grad_scale(int32_t n_tensors, const float *const *grads, const int64_t *sizes, float max_norm,
                        float *scale_out, void *workspace, void *cuda_stream)
{
    using namespace im;
    if (n_tensors < 1 || n_tensors > 64 || !grads || !sizes || !scale_out || !workspace || !(max_norm > 0.0f))
        return IM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 7u) return IM_ERR_INVALID_ARG;
    double *partial = static_cast<double *>(workspace);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    SumSqArgs a;
    a.n_tensors = n_tensors;
    int count = 0;
    for (int k = 0; k < n_tensors; ++k) {
        if (!grads[k] || sizes[k] < 1) return IM_ERR_INVALID_ARG;
        long long g = (sizes[k] + kSqThreads * 8 - 1) / (kSqThreads * 8);
        const int grid = (int)(g < 1 ? 1 : (g > kSqMaxGrid ? kSqMaxGrid : g));
        a.x[k] = grads[k];
        a.n[k] = sizes[k];
        a.first[k] = count;
        count += grid;
    }
    for (int k = n_tensors; k <= kSqMaxTensors; ++k) a.first[k] = count;
    for (int k = n_tensors; k < kSqMaxTensors; ++k) { a.x[k] = nullptr; a.n[k] = 0; }
    sumsq_kernel<<<count, kSqThreads, 0, st>>>(a, partial);
    grad_scale_finish_kernel<<<1, 32, 0, st>>>(partial, count, max_norm, scale_out);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_adaptive_lr(float *lr, const float *kl, float kl_target, float lr_min, float lr_max, void *cuda_stream)
{
    using namespace im;
    if (!lr || !kl || !(kl_target > 0.0f) || !(lr_min > 0.0f) || !(lr_max >= lr_min)) return IM_ERR_INVALID_ARG;
    adaptive_lr_kernel<<<1, 1, 0, (cudaStream_t)cuda_stream>>>(lr, kl, kl_target, lr_min, lr_max);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // extern "C"
