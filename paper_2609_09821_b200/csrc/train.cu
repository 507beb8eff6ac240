// Building blocks of the backward pass of the policy / critic MLP (the paper's update phase):
// the generic bf16 GEMM entries on the tcgen05 kernels of the forward path, and the small
// HBM-bound kernels between them.  With activations H_l = relu(H_{l-1} W_l^T + b_l) and dZ_l the
// gradient at layer l's pre-activation:
//
//   dW_l = dZ_l^T H_{l-1}      as a GEMM over the batch dimension: (dZ_l^T)[N][M] x (H_{l-1}^T)[K][M]^T
//   db_l = column sums of dZ_l
//   dH_{l-1} = dZ_l W_l        as a GEMM over N: dZ_l[M][N] x (W_l^T)[K][N]^T
//   dZ_{l-1} = dH_{l-1} where H_{l-1} > 0, else 0
//
// Every GEMM is C[M][N] = A[M][K] B[N][K]^T with both operands contiguous along the contraction,
// the one form the tensor-core kernels implement; the transposed operands are made by
// transpose_bf16.  Sums over the batch are two-stage and ordered (bit-reproducible).
#include <cmath>
#include <cuda_bf16.h>

#include "im_internal.h"
#include "mlp.h"

namespace im {

namespace {

// A tensor-core product launched with programmatic stream serialization right after one of these kernels may set
// up (barriers, tensor memory) while this grid drains; it still waits for this grid to complete before it reads.
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }


// out[c][r] = in[r][c] for a [rows][cols] bf16 matrix, 64 x 64 tiles through shared memory.
// VEC: both matrices allow 16-byte accesses (pointers and row strides multiples of 8 elements): a tile is
// read and written as 8-element chunks, the transposition happens in the 2-byte shared-memory reads
// (the 8-element chunks of a tile row are XOR-swizzled by the row group, so a column walk spreads over the banks).
template <bool VEC>
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16 *__restrict__ in, long long ld_in, int rows,
                                                             int cols, __nv_bfloat16 *__restrict__ out, long long ld_out)
{
    __shared__ __align__(16) __nv_bfloat16 tile[64][72];
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    if (VEC) {
        // 64 rows x 8 chunks of 8 elements: two chunks per thread
        for (int q = threadIdx.x; q < 512; q += 256) {
            const int i = q >> 3, ch = (q & 7) << 3;
            const int r = r0 + i, c = c0 + ch;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (r < rows && c + 8 <= cols) {
                v = __ldg(reinterpret_cast<const uint4 *>(in + (long long)r * ld_in + c));
            } else if (r < rows) {
                __nv_bfloat16 e[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) e[k] = c + k < cols ? in[(long long)r * ld_in + c + k] : __float2bfloat16_rn(0.0f);
                v = *reinterpret_cast<const uint4 *>(e);
            }
            *reinterpret_cast<uint4 *>(&tile[i][ch ^ (((i >> 3) & 7) << 3)]) = v;        // chunk index swizzled by the row group
        }
        __syncthreads();
        for (int q = threadIdx.x; q < 512; q += 256) {
            const int j = q >> 3, ch = (q & 7) << 3;          // output row c0 + j, elements r0 + ch .. + 7
            const int c = c0 + j, r = r0 + ch;
            if (c >= cols || r >= rows) continue;
            __nv_bfloat16 e[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) e[k] = tile[ch + k][(((j >> 3) ^ (ch >> 3)) << 3) + (j & 7)];
            if (r + 8 <= rows) {
                *reinterpret_cast<uint4 *>(out + (long long)c * ld_out + r) = *reinterpret_cast<const uint4 *>(e);
            } else {
                for (int k = 0; k < 8 && r + k < rows; ++k) out[(long long)c * ld_out + r + k] = e[k];
            }
        }
    } else {
        const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;          // 64 x 4
        for (int i = ty; i < 64; i += 4) {
            const int r = r0 + i, c = c0 + tx;
            tile[i][tx] = (r < rows && c < cols) ? in[(long long)r * ld_in + c] : __float2bfloat16_rn(0.0f);
        }
        __syncthreads();
        for (int i = ty; i < 64; i += 4) {
            const int c = c0 + i, r = r0 + tx;
            if (c < cols && r < rows) out[(long long)c * ld_out + r] = tile[tx][i];
        }
    }
}

// out[r][c] = bf16(in[r][c]) for c < cols, 0 for cols <= c < ld_out.
__global__ void __launch_bounds__(256) to_bf16_padded_kernel(const float *__restrict__ in, long long ld_in, int rows, int cols,
                                                             __nv_bfloat16 *__restrict__ out, int ld_out)
{
    release_dependents();
    const long long total = (long long)rows * ld_out;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / ld_out;
        const int c = (int)(i - r * ld_out);
        out[i] = __float2bfloat16_rn(c < cols ? __ldg(in + r * ld_in + c) : 0.0f);
    }
}

// The same with 16-byte stores: a thread converts eight consecutive columns of one row (ld_out a multiple of 8,
// out 16-byte aligned); its eight loads are 32 consecutive bytes, a warp's one contiguous kilobyte of the row.
__global__ void __launch_bounds__(256) to_bf16_padded_vec_kernel(const float *__restrict__ in, long long ld_in, int rows, int cols,
                                                                 __nv_bfloat16 *__restrict__ out, int ld_out)
{
    release_dependents();
    const int gpr = ld_out >> 3;                                   // 8-column groups per row
    const long long total = (long long)rows * gpr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / gpr;
        const int c = (int)(i - r * gpr) << 3;
        const float *src = in + r * ld_in + c;
        float v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = c + j < cols ? __ldg(src + j) : 0.0f;
        uint4 o;
        __nv_bfloat162 h;
        h = __floats2bfloat162_rn(v[0], v[1]); o.x = *reinterpret_cast<const uint32_t *>(&h);
        h = __floats2bfloat162_rn(v[2], v[3]); o.y = *reinterpret_cast<const uint32_t *>(&h);
        h = __floats2bfloat162_rn(v[4], v[5]); o.z = *reinterpret_cast<const uint32_t *>(&h);
        h = __floats2bfloat162_rn(v[6], v[7]); o.w = *reinterpret_cast<const uint32_t *>(&h);
        *reinterpret_cast<uint4 *>(out + r * ld_out + c) = o;
    }
}

// out[r][c] (float, dense [rows][cols]) = sum over s of in[s][r][c] (bf16 slices `slice_stride` elements
// apart, row stride ld_in), slices added in order.
__global__ void __launch_bounds__(256) sum_slices_kernel(const __nv_bfloat16 *__restrict__ in, long long slice_stride,
                                                         long long ld_in, int slices, int rows, int cols, float *__restrict__ out)
{
    release_dependents();
    const long long total = (long long)rows * cols;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / cols;
        const int c = (int)(i - r * cols);
        float acc = 0.0f;
        for (int k = 0; k < slices; ++k) acc += __bfloat162float(in[k * slice_stride + r * ld_in + c]);
        out[i] = acc;
    }
}

// Row gather for shuffled minibatches: out[i][0..cols) = in[idx[i]][0..cols), written as float or, with
// zero padding up to ld_out, as bf16.  A warp copies one row (consecutive lanes, consecutive columns).
template <bool TO_BF16>
__global__ void __launch_bounds__(256) gather_rows_kernel(const float *__restrict__ in, long long ld_in,
                                                          const int32_t *__restrict__ idx, long long n_src, int rows, int cols,
                                                          void *__restrict__ out, int ld_out, uint32_t *__restrict__ status)
{
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < rows; i += warps) {
        long long src = idx[i];
        if (src < 0 || src >= n_src) {                       // a bad index is clamped and reported, never followed
            if (lane == 0) atomicOr(status, IM_DEV_BAD_STATE);
            src = src < 0 ? 0 : n_src - 1;
        }
        const float *row = in + src * ld_in;
        if (TO_BF16) {
            __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(out) + (long long)i * ld_out;
            for (int c = lane; c < ld_out; c += 32) o[c] = __float2bfloat16_rn(c < cols ? __ldg(row + c) : 0.0f);
        } else {
            float *o = static_cast<float *>(out) + (long long)i * ld_out;
            for (int c = lane; c < cols; c += 32) o[c] = __ldg(row + c);
        }
    }
}

// Column sums, stage 1: a CTA adds a slice of 256 rows for 64 columns; thread (column, row group g of 4)
// adds rows g, g + 4, ... in two independent chains, the four groups are then added in order.
constexpr int kColsumRowsPerCta = 256;
template <typename T>
__device__ __forceinline__ float ld_as_float(const T *p);
template <>
__device__ __forceinline__ float ld_as_float<float>(const float *p) { return __ldg(p); }

template <typename T>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const T *__restrict__ x, long long ld, long long rows, int cols,
                                                             float *__restrict__ partial)
{
    __shared__ float s_part[4][64];
    const int cx = threadIdx.x & 63, g = threadIdx.x >> 6;
    const int c = blockIdx.x * 64 + cx;
    const long long r0 = (long long)blockIdx.y * kColsumRowsPerCta;
    long long r1 = r0 + kColsumRowsPerCta;
    r1 = r1 < rows ? r1 : rows;
    float s0 = 0.0f, s1 = 0.0f;
    if (c < cols) {
        long long r = r0 + g;
        for (; r + 4 < r1; r += 8) {
            s0 += ld_as_float(x + r * ld + c);
            s1 += ld_as_float(x + (r + 4) * ld + c);
        }
        if (r < r1) s0 += ld_as_float(x + r * ld + c);
    }
    s_part[g][cx] = s0 + s1;
    __syncthreads();
    if (g == 0 && c < cols)
        partial[(long long)blockIdx.y * cols + c] = ((s_part[0][cx] + s_part[1][cx]) + s_part[2][cx]) + s_part[3][cx];
}

// The same for matrices that allow 16-byte row accesses: a thread owns 4 adjacent
// columns and adds every eighth row of the slice; a CTA covers 32 such column groups and 8 row groups.
template <typename T>
struct VecOf;
template <>
struct VecOf<float> {
    static constexpr int kN = 4;
    static __device__ __forceinline__ void load(const float *p, float (&v)[4])
    {
        const float4 x = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
    }
};

template <typename T>
__global__ void __launch_bounds__(256) colsum_partial_vec_kernel(const T *__restrict__ x, long long ld, long long rows, int cols,
                                                                 float *__restrict__ partial)
{
    constexpr int V = VecOf<T>::kN;
    __shared__ float s_part[8][32 * V];
    const int cg = threadIdx.x & 31, g = threadIdx.x >> 5;
    const int c = (blockIdx.x * 32 + cg) * V;                     // first of this thread's columns
    const long long r0 = (long long)blockIdx.y * kColsumRowsPerCta;
    long long r1 = r0 + kColsumRowsPerCta;
    r1 = r1 < rows ? r1 : rows;
    float acc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) acc[k] = 0.0f;
    if (c < cols) {                                               // cols is a multiple of V here
        for (long long r = r0 + g; r < r1; r += 8) {
            float v[V];
            VecOf<T>::load(x + r * ld + c, v);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] += v[k];
        }
    }
#pragma unroll
    for (int k = 0; k < V; ++k) s_part[g][cg * V + k] = acc[k];
    __syncthreads();
    for (int j = threadIdx.x; j < 32 * V; j += 256) {
        const int cc = blockIdx.x * 32 * V + j;
        if (cc >= cols) continue;
        float t = 0.0f;
#pragma unroll
        for (int gg = 0; gg < 8; ++gg) t += s_part[gg][j];
        partial[(long long)blockIdx.y * cols + cc] = t;
    }
}

// Stage 2: the slices in fp64 in a fixed order: sixteen threads per column each add every sixteenth slice,
// then the sixteen sums are added in order.
constexpr int kFinishParts = 16;
__global__ void __launch_bounds__(32 * kFinishParts) colsum_finish_kernel(const float *__restrict__ partial, int slices, int cols,
                                                                          float *__restrict__ out)
{
    release_dependents();
    __shared__ double part[kFinishParts][33];
    const int c = blockIdx.x * 32 + threadIdx.x;
    double s = 0.0;
    if (c < cols)
        for (int g = threadIdx.y; g < slices; g += kFinishParts) s += (double)partial[(long long)g * cols + c];
    part[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && c < cols) {
        double t = 0.0;
#pragma unroll
        for (int p = 0; p < kFinishParts; ++p) t += part[p][threadIdx.x];
        out[c] = (float)t;
    }
}

bool al16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
im_status colsum(const T *x, int64_t ld, int64_t rows, int32_t cols, float *out, void *workspace, size_t workspace_bytes,
                 cudaStream_t st)
{
    if (!x || !out || !workspace || rows < 1 || cols < 1 || ld < cols) return IM_ERR_INVALID_ARG;
    const long long slices = (rows + kColsumRowsPerCta - 1) / kColsumRowsPerCta;
    if ((size_t)slices * (size_t)cols * sizeof(float) > workspace_bytes || slices > 65535) return IM_ERR_INVALID_ARG;
    constexpr int V = VecOf<T>::kN;
    if (cols % V == 0 && ld % V == 0 && al16(x)) {
        const dim3 grid((cols + 32 * V - 1) / (32 * V), (unsigned)slices);
        colsum_partial_vec_kernel<T><<<grid, 256, 0, st>>>(x, ld, rows, cols, static_cast<float *>(workspace));
    } else {
        const dim3 grid((cols + 63) / 64, (unsigned)slices);
        colsum_partial_kernel<T><<<grid, 256, 0, st>>>(x, ld, rows, cols, static_cast<float *>(workspace));
    }
    colsum_finish_kernel<<<(cols + 31) / 32, dim3(32, kFinishParts), 0, st>>>(static_cast<const float *>(workspace), (int)slices, cols, out);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // namespace

}  // namespace im

extern "C" {

im_status im_gemm_bf16(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, uint16_t *C, int64_t ldc,
                       int32_t M, int32_t N, int32_t K, const float *bias, int32_t relu, uint32_t *status,
                       void *cuda_stream)
{
    using namespace im;
    if (!A || !B || !C || !bias || !status || M < 1 || N < 64 || K < 64) return IM_ERR_INVALID_ARG;
    if ((N & 63) || (K & 63) || lda < K || ldb < K || ldc < N || (lda & 7) || (ldb & 7) || (ldc & 7)) return IM_ERR_INVALID_ARG;
    if (!al16(A) || !al16(B) || !al16(C) || !al16(bias)) return IM_ERR_INVALID_ARG;
    return tc_gemm(A, lda, B, ldb, C, ldc, M, N, K, bias, relu != 0, status, (cudaStream_t)cuda_stream);
}

im_status im_gemm_bf16_dgrad(const uint16_t *dZ, int64_t ld_dz, const uint16_t *Wt, int64_t ld_wt, uint16_t *dH, int64_t ld_dh,
                             int32_t M, int32_t N, int32_t K, const uint16_t *H, int64_t ld_h, float *colsum_partial,
                             int32_t ld_partial, uint32_t *status, void *cuda_stream)
{
    using namespace im;
    if (!dZ || !Wt || !dH || !status || M < 32 || (M & 31) || N < 64 || K < 64) return IM_ERR_INVALID_ARG;
    if ((N & 63) || (K & 63) || ld_dz < K || ld_wt < K || ld_dh < N || (ld_dz & 7) || (ld_wt & 7) || (ld_dh & 7)) return IM_ERR_INVALID_ARG;
    if (!al16(dZ) || !al16(Wt) || !al16(dH)) return IM_ERR_INVALID_ARG;
    if (H && (ld_h < N || (ld_h & 7) || !al16(H))) return IM_ERR_INVALID_ARG;
    if (colsum_partial && (ld_partial < N || (ld_partial & 1) || (reinterpret_cast<uintptr_t>(colsum_partial) & 7u))) return IM_ERR_INVALID_ARG;
    return tc_gemm(dZ, ld_dz, Wt, ld_wt, dH, ld_dh, M, N, K, nullptr, false, status, (cudaStream_t)cuda_stream, 1, H, ld_h,
                   colsum_partial, ld_partial);
}

im_status im_gemm_bf16_tn(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, uint16_t *C, int64_t ldc,
                          int32_t R, int32_t Mo, int32_t No, int32_t slices, int32_t c_pitch, uint32_t *status,
                          void *cuda_stream)
{
    using namespace im;
    if (!A || !B || !C || !status || R < 64 || Mo < 1 || No < 64 || slices < 1) return IM_ERR_INVALID_ARG;
    if ((No & 63) || R % (64 * slices) || lda < Mo || ldb < No || ldc < No || (lda & 7) || (ldb & 7) || (ldc & 7))
        return IM_ERR_INVALID_ARG;
    if (c_pitch < Mo || (c_pitch & 127)) return IM_ERR_INVALID_ARG;
    if (!al16(A) || !al16(B) || !al16(C)) return IM_ERR_INVALID_ARG;
    return tc_gemm_tn(A, lda, B, ldb, C, ldc, R, Mo, No, slices, c_pitch, status, (cudaStream_t)cuda_stream);
}

im_status im_sum_slices_bf16_to_f32(const uint16_t *in, int64_t slice_stride, int64_t ld_in, int32_t slices, int32_t rows,
                                    int32_t cols, float *out, void *cuda_stream)
{
    using namespace im;
    if (!in || !out || slices < 1 || rows < 1 || cols < 1 || ld_in < cols) return IM_ERR_INVALID_ARG;
    const long long total = (long long)rows * cols;
    long long g = (total + 255) / 256;
    const int grid = (int)(g > 148 * 16 ? 148 * 16 : g);
    sum_slices_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(reinterpret_cast<const __nv_bfloat16 *>(in), slice_stride, ld_in,
                                                                   slices, rows, cols, out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_gemm_bf16_f32out(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, float *C, int32_t M,
                              int32_t N, int32_t K, const float *bias, uint32_t *status, void *cuda_stream)
{
    using namespace im;
    if (!A || !B || !C || !bias || !status || M < 1 || N < 1 || N > 80 || K < 64) return IM_ERR_INVALID_ARG;
    if ((K & 63) || lda < K || ldb < K || (lda & 7) || (ldb & 7)) return IM_ERR_INVALID_ARG;
    if (!al16(A) || !al16(B) || !al16(C)) return IM_ERR_INVALID_ARG;
    return tc_gemm_head(A, lda, B, ldb, M, N, K, bias, C, status, (cudaStream_t)cuda_stream);
}

im_status im_transpose_bf16(const uint16_t *in, int64_t ld_in, int32_t rows, int32_t cols, uint16_t *out, int64_t ld_out,
                            void *cuda_stream)
{
    using namespace im;
    if (!in || !out || rows < 1 || cols < 1 || ld_in < cols || ld_out < rows) return IM_ERR_INVALID_ARG;
    const dim3 grid((cols + 63) / 64, (rows + 63) / 64);
    if (grid.y > 65535) return IM_ERR_INVALID_ARG;
    const bool vec = al16(in) && al16(out) && (ld_in & 7) == 0 && (ld_out & 7) == 0;
    const __nv_bfloat16 *pi = reinterpret_cast<const __nv_bfloat16 *>(in);
    __nv_bfloat16 *po = reinterpret_cast<__nv_bfloat16 *>(out);
    if (vec) transpose_bf16_kernel<true><<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(pi, ld_in, rows, cols, po, ld_out);
    else transpose_bf16_kernel<false><<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(pi, ld_in, rows, cols, po, ld_out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_f32_to_bf16_padded(const float *in, int64_t ld_in, int32_t rows, int32_t cols, uint16_t *out, int32_t ld_out,
                                void *cuda_stream)
{
    using namespace im;
    if (!in || !out || rows < 1 || cols < 1 || ld_in < cols || ld_out < cols) return IM_ERR_INVALID_ARG;
    const bool vec = (ld_out & 7) == 0 && al16(out);
    const long long total = vec ? (long long)rows * (ld_out >> 3) : (long long)rows * ld_out;
    long long g = (total + 255) / 256;
    const int grid = (int)(g > 148 * 16 ? 148 * 16 : g);
    if (vec)
        to_bf16_padded_vec_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(in, ld_in, rows, cols,
                                                                               reinterpret_cast<__nv_bfloat16 *>(out), ld_out);
    else
        to_bf16_padded_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(in, ld_in, rows, cols,
                                                                           reinterpret_cast<__nv_bfloat16 *>(out), ld_out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_gather_rows_f32(const float *in, int64_t ld_in, const int32_t *idx, int64_t n_src, int32_t rows, int32_t cols,
                             void *out, int32_t ld_out, int32_t to_bf16, uint32_t *status, void *cuda_stream)
{
    using namespace im;
    if (!in || !idx || !out || !status || n_src < 1 || rows < 1 || cols < 1 || ld_in < cols || ld_out < cols)
        return IM_ERR_INVALID_ARG;
    long long g = ((long long)rows * 32 + 255) / 256;
    const int grid = (int)(g > 148 * 16 ? 148 * 16 : g);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (to_bf16) gather_rows_kernel<true><<<grid, 256, 0, st>>>(in, ld_in, idx, n_src, rows, cols, out, ld_out, status);
    else gather_rows_kernel<false><<<grid, 256, 0, st>>>(in, ld_in, idx, n_src, rows, cols, out, ld_out, status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

im_status im_copy_f32(float *dst, const float *src, int64_t n, void *cuda_stream)
{
    if (!dst || !src || n < 1) return IM_ERR_INVALID_ARG;
    return cudaMemcpyAsync(dst, src, (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream) == cudaSuccess
               ? IM_OK : IM_ERR_CUDA;
}

im_status im_colsum_f32(const float *x, int64_t ld, int64_t rows, int32_t cols, float *out, void *workspace,
                        size_t workspace_bytes, void *cuda_stream)
{
    return im::colsum<float>(x, ld, rows, cols, out, workspace, workspace_bytes, (cudaStream_t)cuda_stream);
}

}  // extern "C"
