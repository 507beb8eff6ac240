// Policy-side declarations shared by the MLP translation units and the API glue.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/im.h"

struct im_policy {
    im_policy_config cfg;
    cudaStream_t stream;
    int nl;
    bool tensor_path;                 // bf16 tcgen05 chain (else fp32 SIMT layers)
    void *d_W[IM_MAX_LAYERS];         // SIMT path: weights as given ([out][in], float or bf16)
    float *d_b[IM_MAX_LAYERS];
    float *d_act[2];                  // SIMT path: fp32 activations, [max_batch][max hidden]
    int act_ld;
    uint32_t *d_status;
    float *d_log_std;                 // [A] per-dimension ln(sigma) once im_policy_set_log_std has been called, else null
    struct im_policy_tc *tc;          // tensor path state (weights padded for the GEMM tiles, bf16 activations, tensor maps)
};

namespace im {
cudaError_t launch_linear_simt(const float *A, int lda, const void *W, bool w_bf16, const float *bias, float *C,
                               int ldc, int M, int N, int K, bool relu, cudaStream_t stream);
cudaError_t launch_sample(const float *mean, float *action, float *logp, int n, int A, float sigma, const float *log_std,
                          uint64_t seed, uint32_t step, uint32_t env_id_base, cudaStream_t stream);

// Tensor-core path (mlp_tc.cu).
im_status tc_policy_create(im_policy *p, const void *const *W, const float *const *b);
void tc_policy_destroy(im_policy *p);
void tc_policy_layer(im_policy *p, int layer, void **W, int32_t *ld, float **bias);
void *tc_policy_input(im_policy *p, int32_t *ld);     // bf16 [max_batch][ld] staging buffer of the first layer
im_status tc_policy_forward(im_policy *p, uint32_t step, int32_t n, const float *obs, int32_t ld_obs,
                            float *mean_out, float *action_out, float *logp_out, im_policy *src = nullptr);
im_status tc_gemm(const void *A, int64_t lda, const void *B, int64_t ldb, void *C, int64_t ldc, int M, int N, int K,
                  const float *bias, bool relu, uint32_t *status, cudaStream_t stream, int batches = 1,
                  const void *mask = nullptr, int64_t ld_mask = 0, float *colsum_partial = nullptr, int ld_partial = 0);
im_status tc_gemm_tn(const void *A, int64_t lda, const void *B, int64_t ldb, void *C, int64_t ldc, int R, int Mo, int No,
                     int slices, int c_pitch, uint32_t *status, cudaStream_t stream);
im_status tc_gemm_head(const void *A, int64_t lda, const void *B, int64_t ldb, int M, int N, int K, const float *bias,
                       float *mean_out, uint32_t *status, cudaStream_t stream);
// bounded-wait diagnostics of the tensor-core GEMM kernels and of the bulk-copy PPO loss kernel (current device)
cudaError_t tc_set_wait_debug(unsigned long long limit_ns, int skip_loads);
cudaError_t ppo_set_wait_debug(unsigned long long limit_ns, int skip_loads);
}  // namespace im
