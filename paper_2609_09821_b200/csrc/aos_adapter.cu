// Adapter between a simulator's native body-state arrays and the layout the env kernel streams.
//
// Physics engines keep per-env records (array of structures): element (env e, body j, component c)
// of an array sits at base[e * env_stride + j * body_stride + c] -- e.g. positions [N][nbody][3]
// with a leading world body, or spatial velocities [N][nbody][6] holding angular and linear parts
// side by side.  The env kernel wants component rows with the env index fastest (one full line per
// warp load).  gather_kernel transposes one 32-env tile through shared memory: the reads walk each
// env's record front to back (contiguous runs of a body's components), the writes are whole
// 128-byte lines.  scatter_reset_kernel is the way back for envs the step has reset (masked by the
// flag bytes), so the simulator continues from the reference state.  Both touch device memory only.
#include "im_internal.h"

namespace im {

namespace {

constexpr int kTile = 32;

struct AosView {
    const float *base[4];        // pos, quat, linvel, angvel
    long long env_stride[4];
    int body_stride[4];
};

// Row r of the [13 J] component rows -> (array, body, component).
__device__ __forceinline__ void row_to_elem(int r, int J, int &a, int &j, int &c)
{
    if (r < 3 * J) { a = 0; j = r / 3; c = r - 3 * j; return; }
    r -= 3 * J;
    if (r < 4 * J) { a = 1; j = r >> 2; c = r & 3; return; }
    r -= 4 * J;
    if (r < 3 * J) { a = 2; j = r / 3; c = r - 3 * j; return; }
    r -= 3 * J;
    a = 3; j = r / 3; c = r - 3 * j;
}

constexpr int kMaxRows = 13 * IM_MAX_BODIES;

// Per CTA: where row r lives inside an env's records (array index and offset from the env's start).
__device__ __forceinline__ void build_row_table(const AosView &V, int J, uint8_t *arr, int *off)
{
    for (int r = threadIdx.x; r < 13 * J; r += blockDim.x) {
        int a, j, c;
        row_to_elem(r, J, a, j, c);
        arr[r] = (uint8_t)a;
        off[r] = j * V.body_stride[a] + c;
    }
}

__global__ void __launch_bounds__(256) gather_kernel(const __grid_constant__ AosView V, int J, int N,
                                                     float *__restrict__ soa, long long stride)
{
    extern __shared__ float tile[];                    // [32][R | 1]
    __shared__ int off[kMaxRows];
    __shared__ uint8_t arr[kMaxRows];
    const int R = 13 * J, ldt = R | 1;                 // odd row stride: conflict-free column reads
    const int env0 = blockIdx.x * kTile;
    const int n_env = min(kTile, N - env0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    build_row_table(V, J, arr, off);
    __syncthreads();
    // a warp reads one env's records front to back (runs of consecutive addresses)
    for (int e = warp; e < n_env; e += n_warps) {
        const float *b0 = V.base[0] + (long long)(env0 + e) * V.env_stride[0];
        const float *b1 = V.base[1] + (long long)(env0 + e) * V.env_stride[1];
        const float *b2 = V.base[2] + (long long)(env0 + e) * V.env_stride[2];
        const float *b3 = V.base[3] + (long long)(env0 + e) * V.env_stride[3];
        // all of the env's loads are issued before the first value is stored
        float v[kMaxRows / 32];
#pragma unroll
        for (int i = 0; i < kMaxRows / 32; ++i) {
            const int r = lane + 32 * i;
            if (r < R) {
                const int a = arr[r];
                const float *b = a == 0 ? b0 : (a == 1 ? b1 : (a == 2 ? b2 : b3));
                v[i] = __ldg(b + off[r]);
            }
        }
#pragma unroll
        for (int i = 0; i < kMaxRows / 32; ++i) {
            const int r = lane + 32 * i;
            if (r < R) tile[e * ldt + r] = v[i];
        }
    }
    __syncthreads();
    if (lane < n_env) {
#pragma unroll 8
        for (int r = warp; r < R; r += n_warps) soa[(long long)r * stride + env0 + lane] = tile[lane * ldt + r];
    }
}

__global__ void __launch_bounds__(256) scatter_reset_kernel(const __grid_constant__ AosView V, int J, int N,
                                                            const float *__restrict__ soa, long long stride,
                                                            const uint8_t *__restrict__ flags)
{
    extern __shared__ float tile[];
    __shared__ int off[kMaxRows];
    __shared__ uint8_t arr[kMaxRows];
    __shared__ int any_reset;
    const int R = 13 * J, ldt = R | 1;
    const int env0 = blockIdx.x * kTile;
    const int n_env = min(kTile, N - env0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    if (threadIdx.x == 0) any_reset = 0;
    __syncthreads();
    const bool mine = lane < n_env && flags[env0 + lane] != 0;
    if (warp == 0 && __any_sync(0xffffffffu, mine) && lane == 0) any_reset = 1;
    __syncthreads();
    if (!any_reset) return;                             // uniform: read after the barrier
    build_row_table(V, J, arr, off);
    if (mine)
        for (int r = warp; r < R; r += n_warps) tile[lane * ldt + r] = soa[(long long)r * stride + env0 + lane];
    __syncthreads();
    for (int e = warp; e < n_env; e += n_warps) {
        if (flags[env0 + e] == 0) continue;
        for (int r = lane; r < R; r += 32) {
            const int a = arr[r];
            const_cast<float *>(V.base[a])[(long long)(env0 + e) * V.env_stride[a] + off[r]] = tile[e * ldt + r];
        }
    }
}

AosView make_view(const im_body_state_aos &s)
{
    AosView v;
    const im_aos_array *arr[4] = {&s.pos, &s.quat, &s.linvel, &s.angvel};
    for (int i = 0; i < 4; ++i) {
        v.base[i] = arr[i]->base;
        v.env_stride[i] = arr[i]->env_stride;
        v.body_stride[i] = arr[i]->body_stride;
    }
    return v;
}

size_t tile_bytes(int J) { return (size_t)kTile * (13 * J + 1) * sizeof(float); }

}  // namespace

cudaError_t launch_aos_gather(const im_body_state_aos &sim, int J, int N, float *soa, long long stride, cudaStream_t stream)
{
    gather_kernel<<<(N + kTile - 1) / kTile, 256, tile_bytes(J), stream>>>(make_view(sim), J, N, soa, stride);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

cudaError_t launch_aos_scatter_reset(const im_body_state_aos &sim, int J, int N, const float *soa, long long stride,
                                     const uint8_t *flags, cudaStream_t stream)
{
    scatter_reset_kernel<<<(N + kTile - 1) / kTile, 256, tile_bytes(J), stream>>>(make_view(sim), J, N, soa, stride, flags);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

cudaError_t aos_adapter_prepare()
{
    static DeviceOnce once;
    return once.run([] {
        const int bytes = (int)tile_bytes(IM_MAX_BODIES);      // 53 KB at 32 bodies: above the 48 KB default
        cudaError_t e = cudaFuncSetAttribute(gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(scatter_reset_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        return e;
    });
}

}  // namespace im
