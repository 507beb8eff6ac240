// PPO minibatch loss with its gradients at the network outputs, and the advantage moments.
//
// Everything the update needs between the forward and the backward GEMMs, in two launches
// (clipped surrogate of Schulman et al. 2017 with the coefficients of the paper's hyper-parameter
// table: ratio clip, value-loss and entropy coefficients; the mean KL is the quantity its "KL
// threshold" is compared with).  For sample i, action dimension k, sigma_k = exp(log_std_k):
//
//   logp_i = -1/2 sum_k z_ik^2 - sum_k log_std_k - A/2 ln 2 pi,   z_ik = (a_ik - mu_ik) / sigma_k
//   r_i = exp(logp_i - logp_old_i),  Ahat_i = (adv_i - adv_mean) adv_rstd
//   surr_i = -min(r_i Ahat_i, clip(r_i, 1 - eps, 1 + eps) Ahat_i)
//   vl_i = (V_i - R_i)^2  [or max with the clipped-value variant]
//   L = mean surr + c_v mean vl - c_e sum_k (log_std_k + 1/2 ln 2 pi e)
//
// The kernel is a stream over the minibatch (3 A + 5 floats in, A + 1 out per sample): one warp
// per sample row, lanes over the action dimensions, so rows are read and written as contiguous
// runs; the per-row sums are warp shuffles; the per-dimension and scalar sums over the batch are
// kept per lane, folded per CTA in a fixed order and finished by a second one-CTA launch, so the
// result does not depend on scheduling.  No value is read on the host.
#include <cmath>

#include "im_internal.h"

namespace im {

namespace {

constexpr int kWarps = 8;                 // per CTA
constexpr int kMaxGrid = 1024;
constexpr int kMaxA = 128;
constexpr int kScalars = 4;               // surrogate, value loss, kl, clip count
constexpr int kPartial = kMaxA + kScalars;

struct PpoParams {
    im_ppo_config cfg;
    im_ppo_batch b;
    long long M;
    int A;
    float *d_mean, *d_log_std, *d_value, *summary;
    float *partial;                        // [grid][kPartial]
};

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int NI>
__global__ void __launch_bounds__(32 * kWarps) ppo_loss_kernel(const PpoParams P)
{
    __shared__ float s_acc[kWarps][kPartial];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int A = P.A;
    const float eps = P.cfg.clip, cv = P.cfg.value_coef;
    const float inv_M = 1.0f / (float)P.M;
    float ls[NI], inv_sg[NI], so2[NI], dls[NI], acc_ls[NI];
    float sum_log = 0.0f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int k = lane + 32 * i;
        const bool ok = k < A;
        ls[i] = ok ? __ldg(P.b.log_std + k) : 0.0f;
        const float lo = ok ? __ldg(P.b.log_std_old + k) : 0.0f;
        inv_sg[i] = expf(-ls[i]);
        so2[i] = expf(2.0f * lo);
        dls[i] = ls[i] - lo;
        acc_ls[i] = 0.0f;
        sum_log += ls[i];
    }
    sum_log = warp_sum(sum_log);
    const float logp_const = -sum_log - 0.5f * (float)A * 1.8378770664093453f;
    float adv_mean = 0.0f, adv_rstd = 1.0f;
    if (P.b.adv_moments) { adv_mean = __ldg(P.b.adv_moments); adv_rstd = __ldg(P.b.adv_moments + 1); }
    float s_surr = 0.0f, s_vl = 0.0f, s_kl = 0.0f, s_clip = 0.0f;

    const long long stride = (long long)gridDim.x * kWarps;
    for (long long row = (long long)blockIdx.x * kWarps + warp; row < P.M; row += stride) {
        const size_t base = (size_t)row * (size_t)A;
        float z[NI], zz = 0.0f, kl = 0.0f;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int k = lane + 32 * i;
            z[i] = 0.0f;
            if (k < A) {
                const float mu = __ldg(P.b.mean + base + k);
                const float dm = __ldg(P.b.mean_old + base + k) - mu;
                z[i] = (__ldg(P.b.action + base + k) - mu) * inv_sg[i];
                zz = fmaf(z[i], z[i], zz);
                kl += dls[i] + 0.5f * (so2[i] + dm * dm) * inv_sg[i] * inv_sg[i] - 0.5f;
            }
        }
        zz = warp_sum(zz);
        kl = warp_sum(kl);
        const float r = expf(fmaf(-0.5f, zz, logp_const) - __ldg(P.b.logp_old + row));
        const float ah = (__ldg(P.b.advantage + row) - adv_mean) * adv_rstd;
        const float rc = fminf(fmaxf(r, 1.0f - eps), 1.0f + eps);
        const float s1 = r * ah, s2 = rc * ah;
        const bool live = s1 <= s2;                        // the unclipped branch is the minimum
        const float coef = live ? -ah * r * inv_M : 0.0f;  // dL/dlogp_i
        s_surr -= live ? s1 : s2;
        s_clip += fabsf(r - 1.0f) > eps ? 1.0f : 0.0f;
        s_kl += kl;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int k = lane + 32 * i;
            if (k < A) {
                P.d_mean[base + k] = coef * z[i] * inv_sg[i];
                acc_ls[i] = fmaf(coef, fmaf(z[i], z[i], -1.0f), acc_ls[i]);
            }
        }
        const float v = __ldg(P.b.value + row), R = __ldg(P.b.returns + row);
        const float e1 = v - R;
        float vl = e1 * e1, gv = 2.0f * e1;
        if (P.cfg.clip_value_loss) {
            const float vo = __ldg(P.b.value_old + row);
            const float d = v - vo, dc = fminf(fmaxf(d, -eps), eps);
            const float e2 = vo + dc - R;
            if (e2 * e2 > vl) { vl = e2 * e2; gv = d == dc ? 2.0f * e2 : 0.0f; }
        }
        s_vl += vl;
        if (lane == 0) P.d_value[row] = cv * gv * inv_M;
    }
    // per-CTA fold, warps in order
#pragma unroll
    for (int i = 0; i < NI; ++i) s_acc[warp][lane + 32 * i] = acc_ls[i];
    if (lane == 0) {
        s_acc[warp][kMaxA + 0] = s_surr; s_acc[warp][kMaxA + 1] = s_vl;
        s_acc[warp][kMaxA + 2] = s_kl;   s_acc[warp][kMaxA + 3] = s_clip;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < kPartial; j += blockDim.x) {
        const bool used = j < 32 * NI || j >= kMaxA;
        float t = 0.0f;
        if (used)
            for (int w = 0; w < kWarps; ++w) t += s_acc[w][j];
        P.partial[(size_t)blockIdx.x * kPartial + j] = t;
    }
}

// Sums the CTAs' partial rows in order (fp64) and writes d_log_std and the summary.
__global__ void __launch_bounds__(kPartial) ppo_finish_kernel(const PpoParams P, int grid)
{
    __shared__ double s_tot[kPartial];
    const int j = threadIdx.x;
    double t = 0.0;
    for (int g = 0; g < grid; ++g) t += (double)P.partial[(size_t)g * kPartial + j];
    s_tot[j] = t;
    __syncthreads();
    const double M = (double)P.M;
    if (j < P.A) P.d_log_std[j] = (float)(t - (double)P.cfg.entropy_coef);   // the row terms already carry 1/M
    if (j == 0) {
        double H = 0.0;
        for (int k = 0; k < P.A; ++k) H += (double)P.b.log_std[k] + 0.5 * 2.8378770664093453;   // 1/2 ln(2 pi e)
        const double surr = s_tot[kMaxA + 0] / M, vl = s_tot[kMaxA + 1] / M;
        P.summary[0] = (float)(surr + (double)P.cfg.value_coef * vl - (double)P.cfg.entropy_coef * H);
        P.summary[1] = (float)surr;
        P.summary[2] = (float)vl;
        P.summary[3] = (float)H;
        P.summary[4] = (float)(s_tot[kMaxA + 2] / M);
        P.summary[5] = (float)(s_tot[kMaxA + 3] / M);
    }
}

// ---- moments: mean and 1 / (std + 1e-8), n - 1 divisor
constexpr int kMomThreads = 256;

__global__ void __launch_bounds__(kMomThreads) moments_partial_kernel(const float *__restrict__ x, long long n,
                                                                      double *__restrict__ partial)
{
    __shared__ double s_sum[kMomThreads], s_sq[kMomThreads];
    double s = 0.0, q = 0.0;
    for (long long i = (long long)blockIdx.x * kMomThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kMomThreads) {
        const double v = (double)__ldg(x + i);
        s += v;
        q = fma(v, v, q);
    }
    s_sum[threadIdx.x] = s;
    s_sq[threadIdx.x] = q;
    __syncthreads();
    for (int o = kMomThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) { s_sum[threadIdx.x] += s_sum[threadIdx.x + o]; s_sq[threadIdx.x] += s_sq[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { partial[2 * blockIdx.x] = s_sum[0]; partial[2 * blockIdx.x + 1] = s_sq[0]; }
}

__global__ void moments_finish_kernel(const double *__restrict__ partial, int grid, long long n, float *__restrict__ out)
{
    double s = 0.0, q = 0.0;
    for (int g = 0; g < grid; ++g) { s += partial[2 * g]; q += partial[2 * g + 1]; }
    const double mean = s / (double)n;
    double var = n > 1 ? (q - s * mean) / (double)(n - 1) : 0.0;
    var = var > 0.0 ? var : 0.0;
    out[0] = (float)mean;
    out[1] = (float)(1.0 / (sqrt(var) + 1e-8));
}

}  // namespace

}  // namespace im

extern "C" {

size_t im_ppo_workspace_bytes(void) { return (size_t)im::kMaxGrid * im::kPartial * sizeof(float); }

im_status im_moments(const float *x, int64_t n, float *out2, void *workspace, void *cuda_stream)
{
    using namespace im;
    if (!x || !out2 || !workspace || n < 1) return IM_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 7u) return IM_ERR_INVALID_ARG;
    long long g = (n + kMomThreads * 8 - 1) / (kMomThreads * 8);
    const int grid = (int)(g < 1 ? 1 : (g > kMaxGrid ? kMaxGrid : g));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    moments_partial_kernel<<<grid, kMomThreads, 0, st>>>(x, n, static_cast<double *>(workspace));
    moments_finish_kernel<<<1, 1, 0, st>>>(static_cast<const double *>(workspace), grid, n, out2);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_ppo_loss(const im_ppo_config *cfg, int64_t M, int32_t A, const im_ppo_batch *batch, float *d_mean,
                      float *d_log_std, float *d_value, float *summary, void *workspace, void *cuda_stream)
{
    using namespace im;
    if (!cfg || !batch || !d_mean || !d_log_std || !d_value || !summary || !workspace) return IM_ERR_INVALID_ARG;
    if (M < 1 || A < 1 || A > kMaxA) return IM_ERR_INVALID_ARG;
    if (!batch->mean || !batch->log_std || !batch->action || !batch->logp_old || !batch->mean_old ||
        !batch->log_std_old || !batch->advantage || !batch->value || !batch->returns)
        return IM_ERR_INVALID_ARG;
    if (cfg->clip_value_loss && !batch->value_old) return IM_ERR_INVALID_ARG;
    if (!(cfg->clip >= 0.0f) || !std::isfinite(cfg->clip) || !std::isfinite(cfg->value_coef) ||
        !std::isfinite(cfg->entropy_coef))
        return IM_ERR_INVALID_ARG;
    PpoParams p;
    p.cfg = *cfg; p.b = *batch; p.M = M; p.A = A;
    p.d_mean = d_mean; p.d_log_std = d_log_std; p.d_value = d_value; p.summary = summary;
    p.partial = static_cast<float *>(workspace);
    long long g = (M + kWarps * 4 - 1) / (kWarps * 4);           // at least four rows per warp
    const int grid = (int)(g < 1 ? 1 : (g > kMaxGrid ? kMaxGrid : g));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    switch ((A + 31) / 32) {
    case 1: ppo_loss_kernel<1><<<grid, 32 * kWarps, 0, st>>>(p); break;
    case 2: ppo_loss_kernel<2><<<grid, 32 * kWarps, 0, st>>>(p); break;
    case 3: ppo_loss_kernel<3><<<grid, 32 * kWarps, 0, st>>>(p); break;
    default: ppo_loss_kernel<4><<<grid, 32 * kWarps, 0, st>>>(p); break;
    }
    ppo_finish_kernel<<<1, kPartial, 0, st>>>(p, grid);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // extern "C"
