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

constexpr int kWarps = 4;                 // per CTA
constexpr int kMaxGrid = 888;              // six CTAs per SM: bounds the partial rows the finishing launch walks
constexpr int kFinishGroups = 4;
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

// A row is handled by a group of LPR lanes (8, 16 or 32, chosen so that the row's A floats fill the
// group's NI rounds well); a warp works on 32 / LPR consecutive rows at once, which divides the
// per-row instruction count accordingly.  Each group streams its rows through a private ring of
// kDepth shared-memory slots (three rows of LPR x NI floats -- mean, mean_old, action -- plus five
// scalars) filled with asynchronous 4-byte copies: kDepth - 1 rows of memory requests are in flight
// per group while one row is worked on, at no cost in registers.
template <int LPR, int NI>
struct Ring {
    static constexpr int kGroups = 32 / LPR;
    static constexpr int kRow = LPR * NI;
    static constexpr int kSlotFloats = 3 * kRow + 8;
    // as deep as fits 40 KB of static shared memory per CTA, at most 4
    static constexpr int kFit = (40 * 1024) / (kWarps * kGroups * kSlotFloats * 4);
    static constexpr int kDepth = kFit >= 4 ? 4 : (kFit >= 3 ? 3 : 2);
};

__device__ __forceinline__ void cp_async4(uint32_t dst_smem, const float *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Sum over the LPR lanes of a group (xor butterfly: every lane of the group ends with the same value).
template <int LPR>
__device__ __forceinline__ float group_sum(float v)
{
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int LPR, int NI>
__global__ void __launch_bounds__(32 * kWarps) ppo_loss_kernel(const PpoParams P)
{
    using R = Ring<LPR, NI>;
    constexpr int kGroups = R::kGroups, kDepth = R::kDepth, kRow = R::kRow, kSlotFloats = R::kSlotFloats;
    __shared__ float s_acc[kWarps][kPartial];
    __shared__ __align__(16) float s_ring[kWarps][kGroups][kDepth][kSlotFloats];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane / LPR, sl = lane % LPR;          // group within the warp, lane within the group
    const int A = P.A;
    const float eps = P.cfg.clip, cv = P.cfg.value_coef;
    const float inv_M = 1.0f / (float)P.M;
    float inv_sg[NI], so2[NI], dls[NI], acc_ls[NI];
    float sum_log = 0.0f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int k = sl + LPR * i;
        const bool ok = k < A;
        const float ls = ok ? __ldg(P.b.log_std + k) : 0.0f;
        const float lo = ok ? __ldg(P.b.log_std_old + k) : 0.0f;
        inv_sg[i] = expf(-ls);
        so2[i] = expf(2.0f * lo);
        dls[i] = ls - lo;
        acc_ls[i] = 0.0f;
        sum_log += ls;
    }
    sum_log = group_sum<LPR>(sum_log);
    const float logp_const = -sum_log - 0.5f * (float)A * 1.8378770664093453f;
    float adv_mean = 0.0f, adv_rstd = 1.0f;
    if (P.b.adv_moments) { adv_mean = __ldg(P.b.adv_moments); adv_rstd = __ldg(P.b.adv_moments + 1); }
    float s_surr = 0.0f, s_vl = 0.0f, s_kl = 0.0f, s_clip = 0.0f;

    // A lane reads back only what it copied itself (element k of the three arrays); the five per-row
    // scalars are copied by the group's lanes 0..4 and read by all of its lanes after a __syncwarp.
    float *ring = s_ring[warp][grp][0];
    const long long stride = (long long)gridDim.x * kWarps * kGroups;
    const long long first = ((long long)blockIdx.x * kWarps + warp) * kGroups + grp;
    auto issue = [&](long long row, int slot) {
        if (row < P.M) {
            const size_t base = (size_t)row * (size_t)A;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(ring + slot * kSlotFloats);
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int k = sl + LPR * i;
                if (k < A) {
                    cp_async4(dst + 4u * (uint32_t)k, P.b.mean + base + k);
                    cp_async4(dst + 4u * (uint32_t)(kRow + k), P.b.mean_old + base + k);
                    cp_async4(dst + 4u * (uint32_t)(2 * kRow + k), P.b.action + base + k);
                }
            }
            const float *sc = sl == 0 ? P.b.logp_old : sl == 1 ? P.b.advantage : sl == 2 ? P.b.value
                            : sl == 3 ? P.b.returns : (sl == 4 && P.cfg.clip_value_loss) ? P.b.value_old : nullptr;
            if (sc) cp_async4(dst + 4u * (uint32_t)(3 * kRow + sl), sc + row);
        }
        cp_async_commit();                                  // an empty group past the end keeps the count in step
    };
#pragma unroll
    for (int d = 0; d < kDepth - 1; ++d) issue(first + d * stride, d);
    int slot = 0;
    // the warp's groups run in lock step; a group whose rows have run out idles through the trip
    const long long warp_first = ((long long)blockIdx.x * kWarps + warp) * kGroups;
    for (long long row0 = warp_first; row0 < P.M; row0 += stride) {
        const long long row = row0 + grp;
        const bool in = row < P.M;
        issue(row + (kDepth - 1) * stride, (slot + kDepth - 1) % kDepth);
        cp_async_wait<kDepth - 1>();
        __syncwarp();
        const float *cur = ring + slot * kSlotFloats;
        const size_t base = (size_t)row * (size_t)A;
        float z[NI], zz = 0.0f, kl = 0.0f;
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const int k = sl + LPR * i;
            z[i] = 0.0f;
            if (in && k < A) {
                const float mu = cur[k];
                const float dm = cur[kRow + k] - mu;
                z[i] = (cur[2 * kRow + k] - mu) * inv_sg[i];
                zz = fmaf(z[i], z[i], zz);
                kl += dls[i] + 0.5f * (so2[i] + dm * dm) * inv_sg[i] * inv_sg[i] - 0.5f;
            }
        }
        zz = group_sum<LPR>(zz);
        kl = group_sum<LPR>(kl);
        if (in) {
            const float r = expf(fmaf(-0.5f, zz, logp_const) - cur[3 * kRow + 0]);
            const float ah = (cur[3 * kRow + 1] - adv_mean) * adv_rstd;
            const float rc = fminf(fmaxf(r, 1.0f - eps), 1.0f + eps);
            const float s1 = r * ah, s2 = rc * ah;
            const bool live = s1 <= s2;                        // the unclipped branch is the minimum
            const float coef = live ? -ah * r * inv_M : 0.0f;  // dL/dlogp_i
            s_surr -= live ? s1 : s2;
            s_clip += fabsf(r - 1.0f) > eps ? 1.0f : 0.0f;
            s_kl += kl;
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int k = sl + LPR * i;
                if (k < A) {
                    P.d_mean[base + k] = coef * z[i] * inv_sg[i];
                    acc_ls[i] = fmaf(coef, fmaf(z[i], z[i], -1.0f), acc_ls[i]);
                }
            }
            const float v = cur[3 * kRow + 2], Rt = cur[3 * kRow + 3];
            const float e1 = v - Rt;
            float vl = e1 * e1, gv = 2.0f * e1;
            if (P.cfg.clip_value_loss) {
                const float vo = cur[3 * kRow + 4];
                const float d = v - vo, dc = fminf(fmaxf(d, -eps), eps);
                const float e2 = vo + dc - Rt;
                if (e2 * e2 > vl) { vl = e2 * e2; gv = d == dc ? 2.0f * e2 : 0.0f; }
            }
            s_vl += vl;
            if (sl == 0) P.d_value[row] = cv * gv * inv_M;
        }
        __syncwarp();                                      // every lane is done with the slot before it is refilled
        slot = slot + 1 == kDepth ? 0 : slot + 1;
    }
    cp_async_wait<0>();
    // fold the warp's groups (the same k sits in lane sl of every group), then the CTA's warps in order
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int i = 0; i < NI; ++i) acc_ls[i] += __shfl_xor_sync(0xffffffffu, acc_ls[i], o);
        s_surr += __shfl_xor_sync(0xffffffffu, s_surr, o);
        s_vl += __shfl_xor_sync(0xffffffffu, s_vl, o);
        s_kl += __shfl_xor_sync(0xffffffffu, s_kl, o);
        s_clip += __shfl_xor_sync(0xffffffffu, s_clip, o);
    }
    for (int j = lane; j < kPartial; j += 32) s_acc[warp][j] = 0.0f;
    __syncwarp();
    if (grp == 0) {
#pragma unroll
        for (int i = 0; i < NI; ++i)
            if (sl + LPR * i < kMaxA) s_acc[warp][sl + LPR * i] = acc_ls[i];
    }
    if (lane == 0) {
        s_acc[warp][kMaxA + 0] = s_surr; s_acc[warp][kMaxA + 1] = s_vl;
        s_acc[warp][kMaxA + 2] = s_kl;   s_acc[warp][kMaxA + 3] = s_clip;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < kPartial; j += blockDim.x) {
        float t = 0.0f;
        for (int w = 0; w < kWarps; ++w) t += s_acc[w][j];
        P.partial[(size_t)blockIdx.x * kPartial + j] = t;
    }
}

// Sums the CTAs' partial rows (fp64, four interleaved groups, each in order, then the groups in order)
// and writes d_log_std and the summary.
__global__ void __launch_bounds__(kFinishGroups * kPartial) ppo_finish_kernel(const PpoParams P, int grid)
{
    __shared__ double s_grp[kFinishGroups][kPartial];
    __shared__ double s_tot[kPartial];
    const int j = threadIdx.x % kPartial, q = threadIdx.x / kPartial;
    double t = 0.0;
    for (int g = q; g < grid; g += kFinishGroups) t += (double)P.partial[(size_t)g * kPartial + j];
    s_grp[q][j] = t;
    __syncthreads();
    if (q == 0) {
        t = 0.0;
        for (int k = 0; k < kFinishGroups; ++k) t += s_grp[k][j];
        s_tot[j] = t;
        if (j < P.A) P.d_log_std[j] = (float)(t - (double)P.cfg.entropy_coef);   // the row terms already carry 1/M
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const double M = (double)P.M;
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

// One warp: lane l adds partials l, l + 32, ... in order, then a butterfly in a fixed order.
__global__ void __launch_bounds__(32) moments_finish_kernel(const double *__restrict__ partial, int grid, long long n,
                                                            float *__restrict__ out)
{
    double s = 0.0, q = 0.0;
    for (int g = threadIdx.x; g < grid; g += 32) { s += partial[2 * g]; q += partial[2 * g + 1]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (threadIdx.x != 0) return;
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
    moments_finish_kernel<<<1, 32, 0, st>>>(static_cast<const double *>(workspace), grid, n, out2);
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
    long long g = (M + kWarps * 16 - 1) / (kWarps * 16);         // at least a few trips per warp
    const int grid = (int)(g < 1 ? 1 : (g > kMaxGrid ? kMaxGrid : g));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // lanes per row and rounds: rows up to 32 floats on 8 lanes, up to 80 on 16, wider ones on a whole warp
#define IM_PPO_LAUNCH(LPR, NI) ppo_loss_kernel<LPR, NI><<<grid, 32 * kWarps, 0, st>>>(p)
    if (A <= 32) {
        switch ((A + 7) / 8) {
        case 1: IM_PPO_LAUNCH(8, 1); break;
        case 2: IM_PPO_LAUNCH(8, 2); break;
        case 3: IM_PPO_LAUNCH(8, 3); break;
        default: IM_PPO_LAUNCH(8, 4); break;
        }
    } else if (A <= 80) {
        switch ((A + 15) / 16) {
        case 3: IM_PPO_LAUNCH(16, 3); break;
        case 4: IM_PPO_LAUNCH(16, 4); break;
        default: IM_PPO_LAUNCH(16, 5); break;
        }
    } else if (A <= 96) {
        IM_PPO_LAUNCH(32, 3);
    } else {
        IM_PPO_LAUNCH(32, 4);
    }
#undef IM_PPO_LAUNCH
    ppo_finish_kernel<<<1, kFinishGroups * kPartial, 0, st>>>(p, grid);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // extern "C"
