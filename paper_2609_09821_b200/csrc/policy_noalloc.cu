// Allocation-free policy forward for callers that must not allocate device memory.
//
// Some users of this library run inside code that is not allowed to call cudaMalloc once it is
// up: a control loop with a hard latency budget (an allocation can block for milliseconds and
// synchronises the device), a process whose memory pool was sized and handed out at start-up, a
// plug-in that lives inside somebody else's allocator.  For them the fp32 policy chain is offered
// once more with its activation scratch taken from a fixed array that is part of the library
// image instead of from cudaMalloc: the caller passes every input and output (weights included,
// as device pointers it owns); the library adds nothing but the two ping-pong activation buffers
// below.
//
// The array is file-scope device memory: every GPU that loads the library holds
// IM_NOALLOC_SCRATCH_BYTES of it until the process exits.  Its name is only a stand-in in host
// code, so the address the kernels get is looked up with cudaGetSymbolAddress, once per device,
// with that device current.
#include <cuda_runtime.h>

#include "im_internal.h"
#include "mlp.h"

namespace {

constexpr size_t kScratchFloats = 2ull * IM_NOALLOC_MAX_BATCH * IM_NOALLOC_MAX_WIDTH;

static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats];

std::atomic<float *> g_scratch_ptr[im::kMaxDevices];      // per device; threads racing on the first call store the same value

// Device address of the scratch array on the current device (set-up on first use per device).
im_status scratch_for_current_device(float **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= im::kMaxDevices) return IM_ERR_CUDA;
    float *ptr = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return IM_ERR_CUDA;
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return IM_OK;
}

}  // namespace

extern "C" im_status im_policy_forward_noalloc(int32_t n_layers, const int32_t *dims, const float *const *W,
                                               const float *const *b, float sigma, uint64_t seed,
                                               uint32_t env_id_base, uint32_t step, int32_t n, const float *obs,
                                               int32_t ld_obs, float *mean_out, float *action_out, float *logp_out,
                                               void *cuda_stream)
{
    if (!dims || !W || !b || !obs || !mean_out || !action_out) return IM_ERR_INVALID_ARG;
    if (n_layers < 1 || n_layers > IM_MAX_LAYERS) return IM_ERR_INVALID_ARG;
    if (n < 1 || n > IM_NOALLOC_MAX_BATCH) return IM_ERR_UNSUPPORTED;        // more rows than the scratch holds
    if (!(sigma > 0.0f)) return IM_ERR_INVALID_ARG;
    for (int l = 0; l <= n_layers; ++l)
        if (dims[l] < 1) return IM_ERR_INVALID_ARG;
    for (int l = 1; l < n_layers; ++l)
        if (dims[l] > IM_NOALLOC_MAX_WIDTH) return IM_ERR_UNSUPPORTED;       // hidden layer wider than the scratch
    for (int l = 0; l < n_layers; ++l)
        if (!W[l] || !b[l]) return IM_ERR_INVALID_ARG;
    if (ld_obs < dims[0]) return IM_ERR_INVALID_ARG;

    float *scratch = nullptr;
    const im_status st = scratch_for_current_device(&scratch);
    if (st != IM_OK) return st;
    // Nothing in the scratch has to start at zero: every layer writes all n x dims[l+1] values
    // that the next layer reads, so what an earlier call left behind is never looked at.
    float *act[2] = {scratch, scratch + (size_t)IM_NOALLOC_MAX_BATCH * IM_NOALLOC_MAX_WIDTH};
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const float *in = obs;
    int ld_in = ld_obs;
    const int A = dims[n_layers];
    for (int l = 0; l < n_layers; ++l) {
        const bool last = l == n_layers - 1;
        float *outp = last ? mean_out : act[l & 1];
        const int ldc = last ? A : IM_NOALLOC_MAX_WIDTH;
        if (im::launch_linear_simt(in, ld_in, W[l], false, b[l], outp, ldc, n, dims[l + 1], dims[l], !last, stream) !=
            cudaSuccess)
            return IM_ERR_CUDA;
        in = outp;
        ld_in = ldc;
    }
    if (im::launch_sample(mean_out, action_out, logp_out, n, A, sigma, nullptr, seed, step, env_id_base, stream) != cudaSuccess)
        return IM_ERR_CUDA;
    return IM_OK;
}
