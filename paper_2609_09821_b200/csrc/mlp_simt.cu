// fp32 SIMT policy layers and the Gaussian sampling kernel.
//
// linear_simt: C[m][n] = act(sum_k A[m][k] W[n][k] + b[n]) with fp32
// accumulation; W is float or bf16.  Used for fp32 policies (the tiny
// configuration) and as a cross-check of the tensor-core path.
#include <cuda_bf16.h>

#include "im_internal.h"
#include "im_device.cuh"
#include "mlp.h"

namespace im {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename TW, bool RELU>
__global__ void __launch_bounds__(256) linear_simt_kernel(const float *__restrict__ A, int lda,
                                                          const TW *__restrict__ W, const float *__restrict__ bias,
                                                          float *__restrict__ C, int ldc, int M, int N, int K)
{
    __shared__ float As[BK][BM + 1];
    __shared__ float Ws[BK][BN + 1];
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        for (int i = threadIdx.x; i < BM * BK; i += 256) {
            const int r = i / BK, c = i % BK;
            const int m = m0 + r, k = k0 + c;
            As[c][r] = (m < M && k < K) ? A[(size_t)m * lda + k] : 0.0f;
            const int n = n0 + r;
            Ws[c][r] = (n < N && k < K) ? to_f32(W[(size_t)n * K + k]) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int jn = 0; jn < 4; ++jn) acc[i][jn] = fmaf(a[i], w[jn], acc[i][jn]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) {
            const int n = n0 + tx * 4 + jn;
            if (n >= N) continue;
            float v = acc[i][jn] + bias[n];
            if (RELU) v = fmaxf(v, 0.0f);
            C[(size_t)m * ldc + n] = v;
        }
    }
}

// action = mean + sigma z, z from Philox counter (env id, step, 1, block) and
// Box-Muller; logp = -0.5 sum z^2 - A ln sigma - (A/2) ln 2 pi.  One thread per env.
__global__ void sample_kernel(const float *__restrict__ mean, float *__restrict__ action, float *__restrict__ logp,
                              int n, int A, float sigma, const float *__restrict__ log_std, uint32_t seed_lo,
                              uint32_t seed_hi, uint32_t step, uint32_t env_id_base)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    float zz = 0.0f, sum_log = (float)A * logf(sigma);
    if (log_std) {
        sum_log = 0.0f;
        for (int i = 0; i < A; ++i) sum_log += __ldg(log_std + i);
    }
    for (int blk = 0; 4 * blk < A; ++blk) {
        const uint4 x = philox4x32_10(make_uint4(env_id_base + (uint32_t)e, step, IM_STREAM_ACTION, (uint32_t)blk),
                                      make_uint2(seed_lo, seed_hi));
        float z[4];
        box_muller(x.x, x.y, z[0], z[1]);
        box_muller(x.z, x.w, z[2], z[3]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int o = 4 * blk + i;
            if (o < A) {
                const float sg = log_std ? expf(__ldg(log_std + o)) : sigma;
                action[(size_t)e * A + o] = mean[(size_t)e * A + o] + sg * z[i];
                zz += z[i] * z[i];
            }
        }
    }
    if (logp) logp[e] = -0.5f * zz - sum_log - 0.5f * (float)A * 1.8378770664093453f;
}

}  // namespace

cudaError_t launch_linear_simt(const float *A, int lda, const void *W, bool w_bf16, const float *bias, float *C,
                               int ldc, int M, int N, int K, bool relu, cudaStream_t stream)
{
    const dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM), block(256);
    if (w_bf16) {
        const __nv_bfloat16 *Wb = static_cast<const __nv_bfloat16 *>(W);
        if (relu) linear_simt_kernel<__nv_bfloat16, true><<<grid, block, 0, stream>>>(A, lda, Wb, bias, C, ldc, M, N, K);
        else linear_simt_kernel<__nv_bfloat16, false><<<grid, block, 0, stream>>>(A, lda, Wb, bias, C, ldc, M, N, K);
    } else {
        const float *Wf = static_cast<const float *>(W);
        if (relu) linear_simt_kernel<float, true><<<grid, block, 0, stream>>>(A, lda, Wf, bias, C, ldc, M, N, K);
        else linear_simt_kernel<float, false><<<grid, block, 0, stream>>>(A, lda, Wf, bias, C, ldc, M, N, K);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

cudaError_t launch_sample(const float *mean, float *action, float *logp, int n, int A, float sigma, const float *log_std,
                          uint64_t seed, uint32_t step, uint32_t env_id_base, cudaStream_t stream)
{
    sample_kernel<<<(n + 127) / 128, 128, 0, stream>>>(mean, action, logp, n, A, sigma, log_std, (uint32_t)seed,
                                                       (uint32_t)(seed >> 32), step, env_id_base);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace im
