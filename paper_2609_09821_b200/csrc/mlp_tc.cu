// Tensor-core policy chain for sm_100a: one persistent, warp-specialised GEMM
// kernel per layer, C[M][N] = act(A[M][K] W[N][K]^T + b), bf16 operands, fp32
// accumulation in tensor memory.
//
//   warp 0      TMA producer: A and W tiles (128B-swizzled, K-major) into a ring of smem stages
//   warp 1      MMA issuer: tcgen05.mma 128 x BLOCK_N x 16 into one of two TMEM accumulators
//   warps 2..5  epilogue: tcgen05.ld the finished accumulator, add bias, then either ReLU + bf16
//               store (hidden layers) or the Gaussian head (last layer: mean, Philox/Box-Muller
//               noise, action, log-probability), while the MMA warp works on the next tile
//
// Hidden activations stay bf16 and L2-resident between layers.  Every wait on
// an mbarrier is bounded: when the limit runs out the kernel raises
// IM_DEV_WAIT_TIMEOUT in the status word, stops issuing work, and leaves
// through the common exit that frees its tensor memory.
#include <cmath>
#include <cstring>
#include <utility>
#include <cuda.h>
#include <cuda_bf16.h>

#include <new>
#include <vector>

#include "im_internal.h"
#include "im_device.cuh"
#include "mlp.h"

namespace im {

namespace {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;               // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
// Limit of every bounded wait below (2 s unless im_debug_set_wait changed it), and the diagnostic switch that makes the
// TMA producers issue nothing, so that a test can watch a wait run out with no copy or MMA in flight.
__device__ unsigned long long g_wait_limit_ns = 2000000000ull;
__device__ int g_skip_loads = 0;


// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (int spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 255) == 255) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > g_wait_limit_ns) { *abort_flag = 1; return false; }
        }
    }
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may start while its
// predecessor in the stream is still running; dep_wait() returns once that predecessor has completed and its
// writes are visible, dep_release() lets the successor's blocks be scheduled as SMs free up.  Both are no-ops
// for a plain launch.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], single-CTA, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 16 consecutive columns of fp32: thread i gets row (lane base + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 columns, issue only; pair with tmem_ld_wait() before the values are used.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, float *v)
{
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128B swizzle,
// 8-row groups 1024 bytes apart (the layout a SWIZZLE_128B tensor-map load produces).
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);          // start address, 16-byte units
    d |= (uint64_t)0 << 16;                                // leading byte offset: unused for swizzled K-major
    d |= (uint64_t)(1024u >> 4) << 32;                     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                                // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                                // SWIZZLE_128B
    return d;
}
// Operand stored with its M (or N) index contiguous: rows of the shared-memory tile are contraction
// (K) steps, each row holding 64 consecutive M/N elements (128 bytes, 128B-swizzled).  Eight K rows
// form a 1024-byte group (stride byte offset); the next block of 64 M/N elements starts
// `mn_block_bytes` further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_mn_major_sw128(uint32_t smem_addr, uint32_t mn_block_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((mn_block_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M x N tile.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// ... the same with both operands M/N-major (bits 15 and 16).
__host__ __device__ constexpr uint32_t instr_desc_bf16_mn(int M, int N) { return instr_desc_bf16(M, N) | (1u << 15) | (1u << 16); }

struct GemmParams {
    int M;             // rows in use (envs)
    int N;             // valid output columns
    int K_blocks;      // K / 64 (K is padded with zeros)
    int n_tiles_n;     // N tiles of BLOCK_N
    int stages;        // depth of the operand ring in shared memory
    const float *bias; // [n_tiles_n * BLOCK_N], zero padded
    float act_floor;   // hidden-layer epilogue: out = max(acc + bias, act_floor); 0 is ReLU, -inf no activation
    // Batched products on the single-CTA hidden kernel: batch b multiplies rows [b a_batch_rows, +M) of A
    // with rows [b b_batch_rows, +N) of B into rows [b a_batch_rows, +M) of C.  n_batches = 1: plain GEMM.
    int n_batches, a_batch_rows, b_batch_rows;
    int c_batch_rows;  // rows of C between two batches
    // Backward-pass epilogue (BWD instantiations): output (r, c) is zeroed where mask[r][c] <= 0 (the ReLU of the
    // forward pass), and the column sums of the masked fp32 values over each 32-row block r / 32 go to
    // colsum_partial[(r / 32) * ld_partial + c] (M a multiple of 32).  Either may be null.
    const __nv_bfloat16 *mask;
    long long ld_mask;
    float *colsum_partial;
    int ld_partial;
    // Gaussian head
    float *mean, *action, *logp;
    float sigma;
    const float *log_std;   // [N] per-column ln(sigma), or null: the scalar sigma for every column
    uint32_t seed_lo, seed_hi, step, env_id_base;
    uint32_t *status;
};

constexpr int kEpiSlabBytes = 32 * 128;    // one epilogue warp's 32 rows x 64 bf16 staging slab

constexpr size_t kSmemLimit = 232448;       // opt-in shared memory per block on this architecture (227 KB)

template <int BLOCK_N>
struct SmemPlan {
    static constexpr int kABytes = BLOCK_M * BLOCK_K * 2;
    static constexpr int kBBytes = BLOCK_N * BLOCK_K * 2;
    static constexpr int kBBytesPadded = (kBBytes + 1023) / 1024 * 1024;     // keep every tile 1024-byte aligned
    static constexpr int kStageBytes = kABytes + kBBytesPadded;
    static constexpr int kAccStride = BLOCK_N <= 128 ? 128 : 256;           // TMEM columns between the two accumulators
    static constexpr int kTmemCols = 2 * kAccStride;
    static constexpr int kBarBytes = 256;
    static constexpr int kMaxStages = 8;
    // hidden layers: two staging slabs per epilogue warp for the TMA stores
    // (backward epilogue: two more per warp for the ReLU mask boxes)
    static constexpr __host__ __device__ int hidden_epi_bytes(bool bwd = false) { return (bwd ? 2 : 1) * 4 * 2 * kEpiSlabBytes; }
    // head: [2 accumulators][mean, action][128 rows][A] floats laid out as in global memory,
    // partial sums of z^2 [2][4][128], band counters [2][4]
    // (+ bias and per-column sigma of the tile's columns, 2 x 128 floats)
    __host__ __device__ static constexpr int head_epi_bytes(int A)
    {
        return (2 * 2 * 128 * A * 4 + 2 * 4 * 128 * 4 + 64 + 2 * 128 * 4 + 1023) / 1024 * 1024;
    }
    __host__ __device__ static constexpr int stages_for(int epi_bytes)
    {
        const int room = (int)kSmemLimit - 1024 - kBarBytes - epi_bytes;
        const int s = room / kStageBytes;
        return s > kMaxStages ? kMaxStages : s;
    }
    __host__ __device__ static constexpr size_t bytes(int stages, int epi_bytes) { return 1024 + (size_t)stages * kStageBytes + epi_bytes + kBarBytes; }
};

struct Pipe {
    int stages;
    uint8_t *tiles;
    uint64_t *full, *empty, *acc_full, *acc_empty;
    uint32_t *tmem_slot;
    volatile int *abort_flag;
    uint64_t *mask_bar;      // [4 epilogue warps][2]
    uint8_t *epi;
};

template <class Plan>
__device__ __forceinline__ Pipe carve_pipe(uint8_t *smem_raw, int stages, int epi_bytes)
{
    Pipe p;
    p.stages = stages;
    p.tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    p.epi = p.tiles + (size_t)stages * Plan::kStageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(p.epi + epi_bytes);
    p.full = bars;
    p.empty = bars + Plan::kMaxStages;
    p.acc_full = bars + 2 * Plan::kMaxStages;
    p.acc_empty = bars + 2 * Plan::kMaxStages + 2;
    p.tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * Plan::kMaxStages + 4);
    p.abort_flag = reinterpret_cast<volatile int *>(p.tmem_slot + 1);
    p.mask_bar = bars + 2 * Plan::kMaxStages + 5;
    return p;
}

template <class Plan>
__device__ __forceinline__ void pipe_init(const Pipe &p, int epi_arrivals)
{
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&p.full[s], 1); mbar_init(&p.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&p.acc_full[a], 1); mbar_init(&p.acc_empty[a], epi_arrivals); }
        for (int i = 0; i < 2 * kEpiWarps; ++i) mbar_init(&p.mask_bar[i], 1);
        *p.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if ((threadIdx.x >> 5) == 1) tmem_alloc(p.tmem_slot, Plan::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
}

// Common exit: everyone meets, the allocating warp frees tensor memory.
template <class Plan>
__device__ __forceinline__ void pipe_exit(const Pipe &p, uint32_t tmem_base, uint32_t *status)
{
    if (*p.abort_flag && (threadIdx.x & 31) == 0) {
        // a wait ran out: give copies and MMAs that are still in flight time to land (bounded)
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *p.abort_flag) atomicOr(status, IM_DEV_WAIT_TIMEOUT);
    if ((threadIdx.x >> 5) == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, Plan::kTmemCols);
    }
}

// TMA producer (one thread): A and W tiles of every k-block of every tile of this CTA.
template <class Plan, int BLOCK_N, bool MN = false>
__device__ __forceinline__ void producer_role(const Pipe &p, const CUtensorMap *map_a, const CUtensorMap *map_b,
                                              const GemmParams &P, int n_tiles)
{
    int stage = 0;
    uint32_t phase = 0;
    const int tiles_per_batch = n_tiles / P.n_batches;
    if (g_skip_loads) return;                        // diagnostic: the consumers' first wait runs out
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int b = tile / tiles_per_batch, t = tile - b * tiles_per_batch;
        if (MN) {
            // operands are [contraction rows][M or N columns]: a K block is 64 rows, fetched as boxes of 64 columns;
            // batch b is the row range starting at b * a_batch_rows of both operands
            const int mm = (t / P.n_tiles_n) * BLOCK_M, nn = (t % P.n_tiles_n) * BLOCK_N, r0 = b * P.a_batch_rows;
            for (int kb = 0; kb < P.K_blocks; ++kb) {
                if (!mbar_wait(&p.empty[stage], phase ^ 1u, p.abort_flag)) return;
                uint8_t *sa = p.tiles + (size_t)stage * Plan::kStageBytes;
                mbar_arrive_expect_tx(&p.full[stage], Plan::kABytes + Plan::kBBytes);
#pragma unroll
                for (int i = 0; i < BLOCK_M / 64; ++i)
                    tma_load_2d(sa + i * 8192, map_a, &p.full[stage], mm + 64 * i, r0 + kb * BLOCK_K);
#pragma unroll
                for (int i = 0; i < BLOCK_N / 64; ++i)
                    tma_load_2d(sa + Plan::kABytes + i * 8192, map_b, &p.full[stage], nn + 64 * i, r0 + kb * BLOCK_K);
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
            }
            continue;
        }
        const int m0 = b * P.a_batch_rows + (t / P.n_tiles_n) * BLOCK_M, n0 = b * P.b_batch_rows + (t % P.n_tiles_n) * BLOCK_N;
        for (int kb = 0; kb < P.K_blocks; ++kb) {
            if (!mbar_wait(&p.empty[stage], phase ^ 1u, p.abort_flag)) return;
            uint8_t *sa = p.tiles + (size_t)stage * Plan::kStageBytes;
            mbar_arrive_expect_tx(&p.full[stage], Plan::kABytes + Plan::kBBytes);
            tma_load_2d(sa, map_a, &p.full[stage], kb * BLOCK_K, m0);
            tma_load_2d(sa + Plan::kABytes, map_b, &p.full[stage], kb * BLOCK_K, n0);
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
    }
}

// MMA issuer (one thread).
template <class Plan, int BLOCK_N, bool MN = false>
__device__ __forceinline__ void mma_role(const Pipe &p, uint32_t tmem_base, const GemmParams &P, int n_tiles)
{
    constexpr uint32_t idesc = MN ? instr_desc_bf16_mn(BLOCK_M, BLOCK_N) : instr_desc_bf16(BLOCK_M, BLOCK_N);
    int stage = 0, acc = 0;
    uint32_t phase = 0, acc_phase = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        if (!mbar_wait(&p.acc_empty[acc], acc_phase ^ 1u, p.abort_flag)) return;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * Plan::kAccStride);
        for (int kb = 0; kb < P.K_blocks; ++kb) {
            if (!mbar_wait(&p.full[stage], phase, p.abort_flag)) return;
            tc_fence_after();
            const uint32_t sa = smem_u32(p.tiles + (size_t)stage * Plan::kStageBytes);
            if (MN) {
                const uint64_t da = smem_desc_mn_major_sw128(sa, 8192u), db = smem_desc_mn_major_sw128(sa + Plan::kABytes, 8192u);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                    // advancing K by 16 rows = two 1024-byte groups: +128 in 16-byte units
                    umma_bf16(d_tmem, da + (uint64_t)(128 * k), db + (uint64_t)(128 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                }
            } else {
                const uint64_t da = smem_desc_k_major_sw128(sa), db = smem_desc_k_major_sw128(sa + Plan::kABytes);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                    // advancing K by 16 bf16 = 32 bytes inside the swizzled row: +2 in 16-byte units
                    umma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                }
            }
            umma_commit(&p.empty[stage]);            // smem stage is free once these MMAs have read it
            if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        umma_commit(&p.acc_full[acc]);               // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
}

// Warp reduce-scatter step: every lane holds 2 C values; afterwards C sums over the lane pair (lane, lane ^ offset),
// the lower lane keeping the first C columns and the upper lane the second C.
template <int C>
__device__ __forceinline__ void reduce_scatter_step(float *v, int lane, int offset)
{
    const bool up = (lane & offset) != 0;
#pragma unroll
    for (int i = 0; i < C; ++i) {
        const float keep = up ? v[i + C] : v[i], send = up ? v[i] : v[i + C];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, offset);
    }
}

// One epilogue chunk of the hidden-layer kernels: 64 accumulator columns of this thread's row -> bias, floor,
// (BWD: ReLU mask of the forward activations, column sums over the warp's 32 rows) -> 32 packed bf16 pairs.
// ReLU mask of the backward epilogue: each epilogue warp keeps two 32-row x 64-column boxes of the forward
// activations in shared memory (128B-swizzled, like the output slabs), fetched by TMA one chunk ahead.
__device__ __forceinline__ void mask_issue(const CUtensorMap *map_m, uint8_t *slab, uint64_t *bar, int col0, int row0)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the warp's earlier reads of this slab come first
    mbar_arrive_expect_tx(bar, kEpiSlabBytes);
    tma_load_2d(slab, map_m, bar, col0, row0);
}
__device__ __forceinline__ void mask_read(const uint8_t *slab, int lane, uint4 (&mk)[8])
{
    const uint32_t row = smem_u32(slab) + (uint32_t)lane * 128u;
#pragma unroll
    for (int c = 0; c < 8; ++c)
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(mk[c].x), "=r"(mk[c].y), "=r"(mk[c].z), "=r"(mk[c].w)
                     : "r"(row + (uint32_t)((c ^ (lane & 7)) << 4)) : "memory");
}
__device__ __forceinline__ void mask_all_positive(uint4 (&mk)[8])
{
#pragma unroll
    for (int c = 0; c < 8; ++c) mk[c] = make_uint4(0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u);
}

template <bool BWD>
__device__ __forceinline__ void hidden_chunk(const GemmParams &P, uint32_t t_addr, int row, int col0, int lane,
                                             const uint4 (&mk)[8], uint32_t (&pk)[32])
{
    float v[64];
    tmem_ld32_issue(t_addr, v);
    tmem_ld32_issue(t_addr + 32u, v + 32);
    tmem_ld_wait();
    const float fl = P.act_floor;          // 0: ReLU; -inf: linear output
    if (P.bias) {
        const float4 *b4 = reinterpret_cast<const float4 *>(P.bias + col0);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float4 b = __ldg(b4 + i);
            v[4 * i] = fmaxf(v[4 * i] + b.x, fl);
            v[4 * i + 1] = fmaxf(v[4 * i + 1] + b.y, fl);
            v[4 * i + 2] = fmaxf(v[4 * i + 2] + b.z, fl);
            v[4 * i + 3] = fmaxf(v[4 * i + 3] + b.w, fl);
        }
    } else if (fl > -INFINITY) {
#pragma unroll
        for (int i = 0; i < 64; ++i) v[i] = fmaxf(v[i], fl);
    }
    if (BWD) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t w[4] = {mk[c].x, mk[c].y, mk[c].z, mk[c].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // a bf16 is positive when its 16 bits read as a signed integer are
                if ((int)(short)(w[j] & 0xffffu) <= 0) v[8 * c + 2 * j] = 0.0f;
                if ((int)(short)(w[j] >> 16) <= 0) v[8 * c + 2 * j + 1] = 0.0f;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        pk[i] = *reinterpret_cast<const uint32_t *>(&h);
    }
    if (BWD) {
        if (P.colsum_partial) {
            reduce_scatter_step<32>(v, lane, 16);
            reduce_scatter_step<16>(v, lane, 8);
            reduce_scatter_step<8>(v, lane, 4);
            reduce_scatter_step<4>(v, lane, 2);
            reduce_scatter_step<2>(v, lane, 1);
            const int row0 = row - lane;                 // lane now holds columns 2 lane, 2 lane + 1 of the 64
            if (row0 < P.M)
                *reinterpret_cast<float2 *>(P.colsum_partial + (long long)(row0 >> 5) * P.ld_partial + col0 + 2 * lane) =
                    make_float2(v[0], v[1]);
        }
    }
}

// ------------------------------------------------------------------ hidden layers
// C = relu(A W^T + b) as bf16.  Each epilogue warp owns 32 rows of the tile: it
// reads 64 accumulator columns at a time, applies bias and ReLU, packs to bf16
// into a 128B-swizzled slab in shared memory and hands the slab to a TMA store.
template <int BLOCK_N, bool MN = false, bool BWD = false>
__global__ void __launch_bounds__(kThreads, 1) linear_tc_hidden_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                       const __grid_constant__ CUtensorMap map_b,
                                                                       const __grid_constant__ CUtensorMap map_c,
                                                                       const __grid_constant__ CUtensorMap map_m,
                                                                       const GemmParams P)
{
    using Plan = SmemPlan<BLOCK_N>;
    extern __shared__ uint8_t smem_raw[];
    const Pipe p = carve_pipe<Plan>(smem_raw, P.stages, Plan::hidden_epi_bytes(BWD));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_per_batch = ((P.M + BLOCK_M - 1) / BLOCK_M) * P.n_tiles_n;
    const int n_tiles = tiles_per_batch * P.n_batches;
    pipe_init<Plan>(p, kEpiWarps);
    const uint32_t tmem_base = *p.tmem_slot;
    dep_release();
    dep_wait();                       // nothing before this line touches global memory

    if (warp == 0) {
        if (lane == 0) producer_role<Plan, BLOCK_N, MN>(p, &map_a, &map_b, P, n_tiles);
    } else if (warp == 1) {
        if (lane == 0) mma_role<Plan, BLOCK_N, MN>(p, tmem_base, P, n_tiles);
    } else {
        const int quad = warp & 3;                    // TMEM lanes 32*quad .. 32*quad+31 belong to this warp
        uint8_t *slabs = p.epi + (size_t)(warp - 2) * 2 * kEpiSlabBytes;       // two slabs, used alternately
        int which = 0;
        int acc = 0;
        uint32_t acc_phase = 0;
        // BWD: the mask box of a chunk is fetched one chunk ahead (across tile boundaries), so its latency
        // hides behind the previous chunk and the wait for the accumulator
        const bool masked = BWD && P.mask != nullptr;
        uint8_t *mslabs = p.epi + (size_t)(4 + warp - 2) * 2 * kEpiSlabBytes;
        uint64_t *mbar = p.mask_bar + (warp - 2) * 2;
        uint32_t ci = 0;                               // chunks consumed by this warp
        bool bail = false;
        uint4 mk[8];
        if (masked && (int)blockIdx.x < n_tiles && lane == 0) {
            const int bt = (int)blockIdx.x / tiles_per_batch, tt = (int)blockIdx.x - bt * tiles_per_batch;
            mask_issue(&map_m, mslabs, &mbar[0], (tt % P.n_tiles_n) * BLOCK_N, bt * P.c_batch_rows + (tt / P.n_tiles_n) * BLOCK_M + quad * 32);
        }
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            const int bt = tile / tiles_per_batch, tt = tile - bt * tiles_per_batch;
            const int m0 = bt * P.c_batch_rows + (tt / P.n_tiles_n) * BLOCK_M, n0 = (tt % P.n_tiles_n) * BLOCK_N;
            bool ready = mbar_wait(&p.acc_full[acc], acc_phase, p.abort_flag);
            if (BWD) ready = __all_sync(0xffffffffu, ready);           // the column sums shuffle across the whole warp
            if (!ready) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * Plan::kAccStride);
#pragma unroll 1
            for (int c0 = 0; c0 < BLOCK_N; c0 += 64) {
                uint32_t pk[32];
                if (BWD) {
                    if (masked) {
                        if (lane == 0) {
                            uint8_t *nslab = mslabs + ((ci + 1u) & 1u) * kEpiSlabBytes;
                            if (c0 + 64 < BLOCK_N) mask_issue(&map_m, nslab, &mbar[(ci + 1u) & 1u], n0 + c0 + 64, m0 + quad * 32);
                            else if (tile + (int)gridDim.x < n_tiles) {
                                const int t2 = tile + (int)gridDim.x, bt2 = t2 / tiles_per_batch, tt2 = t2 - bt2 * tiles_per_batch;
                                mask_issue(&map_m, nslab, &mbar[(ci + 1u) & 1u], (tt2 % P.n_tiles_n) * BLOCK_N,
                                           bt2 * P.c_batch_rows + (tt2 / P.n_tiles_n) * BLOCK_M + quad * 32);
                            }
                        }
                        if (!__all_sync(0xffffffffu, mbar_wait(&mbar[ci & 1u], (ci >> 1) & 1u, p.abort_flag))) { bail = true; break; }
                        mask_read(mslabs + (ci & 1u) * kEpiSlabBytes, lane, mk);
                        ++ci;
                    } else mask_all_positive(mk);
                }
                hidden_chunk<BWD>(P, t_row + (uint32_t)c0, m0 + quad * 32 + lane, n0 + c0, lane, mk, pk);
                // the store issued two slabs ago (same buffer) must have finished reading shared memory
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
                uint8_t *slab = slabs + which * kEpiSlabBytes;
                const uint32_t slab_row = smem_u32(slab) + (uint32_t)lane * 128u;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t dst = slab_row + (uint32_t)((c ^ (lane & 7)) << 4);      // 128B swizzle
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                                 "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                 ::"l"(&map_c), "r"(smem_u32(slab)), "r"(n0 + c0), "r"(m0 + quad * 32) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                which ^= 1;
            }
            if (bail) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p.acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores complete before smem goes away
    }
    pipe_exit<Plan>(p, tmem_base, P.status);
}

// ------------------------------------------------------------------ hidden layers, CTA pairs
// The single-CTA kernel above is limited by shared-memory bandwidth: per 64-deep k-block the
// tensor core reads A (16 KB) and W (32 KB) while TMA writes as much.  Here two CTAs of a cluster
// (one TPC) compute a 256 x 256 tile together with tcgen05.mma.cta_group::2: each holds its own 128
// rows of A and HALF of the W tile (128 of the 256 output columns' rows), the tensor cores exchange
// the W halves between the two SMs, and each CTA accumulates its 128 rows x 256 columns in its own
// tensor memory.  Per SM that is 32 KB per k-block instead of 48 KB, and a six-deep ring.
//   rank 0 ("leader"): its MMA thread issues for the pair; its full[] barriers collect the
//     transaction bytes of BOTH CTAs' TMA loads; its acc_empty[] barriers collect both epilogues.
//   both ranks: own TMA producer (own A rows, own W half), own epilogue (own accumulator rows),
//     own empty[] / acc_full[] barriers, which the leader's commits reach by multicast.
// No load is multicast; the only multicast is the commit's mbarrier arrive.
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * BLOCK_M * BLOCK_K * 2;             // A 128x64 + W half 128x64, bf16
constexpr int kPairTmemCols = 512;                                     // two 256-column accumulators
// The backward instantiation (ReLU mask and column sums in the epilogue) runs eight epilogue warps, two per
// tensor-memory lane quadrant, each owning one half of the tile's columns; every warp cycles through a ring of
// three 4 KB slabs, each of which first receives a chunk's mask box and is then overwritten with the chunk's
// output for the TMA store.  The ring takes the room of two operand stages.
constexpr int kPairEpiWarpsBwd = 8;
constexpr int kPairRing = 3;
constexpr __host__ __device__ int pair_epi_warps(bool bwd) { return bwd ? kPairEpiWarpsBwd : kEpiWarps; }
constexpr __host__ __device__ int pair_threads(bool bwd) { return 64 + 32 * pair_epi_warps(bwd); }
constexpr __host__ __device__ int pair_stages(bool bwd) { return bwd ? kPairStages - 2 : kPairStages; }
constexpr __host__ __device__ int pair_epi_bytes(bool bwd)
{
    return bwd ? kPairEpiWarpsBwd * kPairRing * kEpiSlabBytes : kEpiWarps * 2 * kEpiSlabBytes;
}
constexpr size_t pair_smem_bytes(bool bwd) { return 1024 + (size_t)pair_stages(bwd) * kPairStageBytes + pair_epi_bytes(bwd) + 512; }
static_assert(pair_smem_bytes(true) <= kSmemLimit && pair_smem_bytes(false) <= kSmemLimit, "shared memory plan of the pair kernel");
static_assert((2 * kPairStages + 5 + kPairEpiWarpsBwd * kPairRing) * 8 <= 512, "barrier area of the pair kernel");

__device__ __forceinline__ uint32_t cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory whose completion is signalled on a barrier that may live
// in the peer CTA (cluster address).
// Tensor memory of a CTA pair: one warp of EACH CTA issues the allocation, both get the same base.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives, once the pair's MMAs so far have completed, on the barrier at this offset in both CTAs.
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(both) : "memory");
}

// MN: both operands are stored [contraction rows][M or N columns] (the transposed product of two row-major
// matrices, as in the single-CTA kernel's MN instantiation), possibly over several row slices ("batches").
template <bool BWD = false, bool MN = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair_threads(BWD), 1)
linear_tc_hidden_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                             const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_m,
                             const GemmParams P)
{
    constexpr int kStages = pair_stages(BWD);
    constexpr int kEpi = pair_epi_warps(BWD);
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *epi = tiles + (size_t)kStages * kPairStageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(epi + pair_epi_bytes(BWD));
    uint64_t *mask_bar = bars + 2 * kPairStages + 5;
    uint64_t *full = bars, *empty = bars + kPairStages, *acc_full = bars + 2 * kPairStages,
             *acc_empty = bars + 2 * kPairStages + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kPairStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int tiles_m = (P.M + 2 * BLOCK_M - 1) / (2 * BLOCK_M);
    const int tiles_per_batch = tiles_m * P.n_tiles_n;               // 256 x 256 tiles
    const int n_tiles = tiles_per_batch * (MN ? P.n_batches : 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        if (BWD)
            for (int i = 0; i < kPairEpiWarpsBwd * kPairRing; ++i) mbar_init(&mask_bar[i], 1);
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 2 * kEpi); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(tmem_slot, kPairTmemCols);         // one warp of each CTA, collectively
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                              // both CTAs' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    dep_release();
    dep_wait();                       // nothing before this line touches global memory
    if (threadIdx.x == 0 && rank == 1) {
        // the pair's MMAs address the accumulator at the same tensor-memory address in both CTAs
        uint32_t leader_base;
        asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(leader_base) : "r"(map_to_rank(smem_u32(tmem_slot), 0)) : "memory");
        if (leader_base != tmem_base) *abort_flag = 1;
    }
    __syncthreads();

    if (warp == 0) {
        // ---------------- TMA producer (both ranks): own A rows and own half of W, signalled to the leader
        if (lane == 0 && !*abort_flag) {
            int stage = 0;
            uint32_t phase = 0;
            for (int tile = pair; tile < n_tiles; tile += n_pairs) {
                const int bt = MN ? tile / tiles_per_batch : 0, tt = tile - bt * tiles_per_batch;
                const int m0 = (tt / P.n_tiles_n) * 2 * BLOCK_M + (int)rank * BLOCK_M;
                const int n0 = (tt % P.n_tiles_n) * 256 + (int)rank * 128;
                bool ok = true;
                for (int kb = 0; kb < P.K_blocks; ++kb) {
                    if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *sa = tiles + (size_t)stage * kPairStageBytes;
                    const uint32_t leader_full = map_to_rank(smem_u32(&full[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(&full[stage], 2 * kPairStageBytes);
                    if (MN) {
                        // a K block is 64 rows of the slice; this CTA's 128 M columns and its 128 N columns as 64-column boxes
                        const int r = bt * P.a_batch_rows + kb * BLOCK_K;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            tma_load_2d_pair(sa + i * 8192, &map_a, leader_full, m0 + 64 * i, r);
                            tma_load_2d_pair(sa + BLOCK_M * BLOCK_K * 2 + i * 8192, &map_b, leader_full, n0 + 64 * i, r);
                        }
                    } else {
                        tma_load_2d_pair(sa, &map_a, leader_full, kb * BLOCK_K, m0);
                        tma_load_2d_pair(sa + BLOCK_M * BLOCK_K * 2, &map_b, leader_full, kb * BLOCK_K, n0);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only)
        if (lane == 0 && rank == 0 && !*abort_flag) {
            constexpr uint32_t idesc = MN ? instr_desc_bf16_mn(2 * BLOCK_M, 256) : instr_desc_bf16(2 * BLOCK_M, 256);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
                if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 256);
                for (int kb = 0; kb < P.K_blocks; ++kb) {
                    if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(tiles + (size_t)stage * kPairStageBytes);
                    if (MN) {
                        const uint64_t da = smem_desc_mn_major_sw128(sa, 8192u), db = smem_desc_mn_major_sw128(sa + BLOCK_M * BLOCK_K * 2, 8192u);
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                            umma_bf16_pair(d_tmem, da + (uint64_t)(128 * k), db + (uint64_t)(128 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                    } else {
                        const uint64_t da = smem_desc_k_major_sw128(sa), db = smem_desc_k_major_sw128(sa + BLOCK_M * BLOCK_K * 2);
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                            umma_bf16_pair(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    umma_commit_pair(&empty[stage]);          // both CTAs' stages are free once these MMAs have read them
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair(&acc_full[acc]);             // both CTAs' accumulators complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue warps (both ranks): own 128 rows x 256 columns
        const int quad = warp & 3;                     // tensor-memory lanes 32 quad .. 32 quad + 31
        int acc = 0;
        uint32_t acc_phase = 0;
        if constexpr (!BWD) {
            uint8_t *slabs = epi + (size_t)(warp - 2) * 2 * kEpiSlabBytes;
            int which = 0;
            uint4 mk[8];                                // unused without the backward epilogue
            if (!*abort_flag)
            for (int tile = pair; tile < n_tiles; tile += n_pairs) {
                const int bt = MN ? tile / tiles_per_batch : 0, tt = tile - bt * tiles_per_batch;
                const int m0 = bt * P.c_batch_rows + (tt / P.n_tiles_n) * 2 * BLOCK_M + (int)rank * BLOCK_M;
                const int n0 = (tt % P.n_tiles_n) * 256;
                if (!mbar_wait(&acc_full[acc], acc_phase, abort_flag)) break;
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * 256);
#pragma unroll 1
                for (int c0 = 0; c0 < 256; c0 += 64) {
                    uint32_t pk[32];
                    hidden_chunk<false>(P, t_row + (uint32_t)c0, m0 + quad * 32 + lane, n0 + c0, lane, mk, pk);
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
                    uint8_t *slab = slabs + which * kEpiSlabBytes;
                    const uint32_t slab_row = smem_u32(slab) + (uint32_t)lane * 128u;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t dst = slab_row + (uint32_t)((c ^ (lane & 7)) << 4);      // 128B swizzle
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                                     "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                     ::"l"(&map_c), "r"(smem_u32(slab)), "r"(n0 + c0), "r"(m0 + quad * 32) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    which ^= 1;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&acc_empty[acc]), 0));   // the leader's barrier
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        } else {
            // warp 2 + e: quadrant (2 + e) & 3, column chunks 2 (e / 4) and 2 (e / 4) + 1 of every tile.  Chunk j of
            // the warp's sequence uses slab j % 3: mask box in (requested one chunk ahead), output out.
            const int ew = warp - 2, half = ew >> 2;
            uint8_t *ring = epi + (size_t)ew * kPairRing * kEpiSlabBytes;
            uint64_t *mbar = mask_bar + ew * kPairRing;
            const bool masked = P.mask != nullptr;
            uint32_t ci = 0;
            bool bail = false;
            uint4 mk[8];
            auto issue_mask = [&](uint32_t j) {
                const int t2 = pair + (int)(j >> 1) * n_pairs;
                if (t2 >= n_tiles) return;
                mask_issue(&map_m, ring + (j % kPairRing) * kEpiSlabBytes, &mbar[j % kPairRing],
                           (t2 % P.n_tiles_n) * 256 + (2 * half + (int)(j & 1u)) * 64,
                           (t2 / P.n_tiles_n) * 2 * BLOCK_M + (int)rank * BLOCK_M + quad * 32);
            };
            if (masked && lane == 0 && !*abort_flag) issue_mask(0u);
            if (!*abort_flag)
            for (int tile = pair; tile < n_tiles; tile += n_pairs) {
                const int m0 = (tile / P.n_tiles_n) * 2 * BLOCK_M + (int)rank * BLOCK_M;
                const int n0 = (tile % P.n_tiles_n) * 256;
                // (the column sums shuffle across the whole warp: every lane takes the same decision)
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_full[acc], acc_phase, abort_flag))) break;
                tc_fence_after();
                const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * 256);
#pragma unroll 1
                for (int j = 0; j < 2; ++j) {
                    const int c0 = (2 * half + j) * 64;
                    if (lane == 0) {
                        // slab (ci + 1) % 3 last held chunk ci - 2: its store must have read it before the next box lands
                        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        if (masked) issue_mask(ci + 1u);
                    }
                    __syncwarp();
                    uint8_t *slab = ring + (ci % kPairRing) * kEpiSlabBytes;
                    if (masked) {
                        if (!__all_sync(0xffffffffu, mbar_wait(&mbar[ci % kPairRing], (ci / kPairRing) & 1u, abort_flag))) { bail = true; break; }
                        mask_read(slab, lane, mk);
                    } else mask_all_positive(mk);
                    uint32_t pk[32];
                    hidden_chunk<true>(P, t_row + (uint32_t)c0, m0 + quad * 32 + lane, n0 + c0, lane, mk, pk);
                    // each lane overwrites the 128 bytes it read its own mask words from
                    const uint32_t slab_row = smem_u32(slab) + (uint32_t)lane * 128u;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint32_t dst = slab_row + (uint32_t)((c ^ (lane & 7)) << 4);      // 128B swizzle
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * c]), "r"(pk[4 * c + 1]),
                                     "r"(pk[4 * c + 2]), "r"(pk[4 * c + 3]) : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                                     ::"l"(&map_c), "r"(smem_u32(slab)), "r"(n0 + c0), "r"(m0 + quad * 32) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    ++ci;
                }
                if (bail) break;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&acc_empty[acc]), 0));   // the leader's barrier
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------- common exit: both CTAs meet (the peer's shared memory and barriers stay alive
    // until the leader is done with them), then each frees its tensor memory
    if (*abort_flag && lane == 0) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(P.status, IM_DEV_WAIT_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kPairTmemCols);
    }
}

// ------------------------------------------------------------------ Gaussian head (last layer)
// mean = A W^T + b; action = mean + sigma z with z from Philox counter (env, step, 1, block)
// and Box-Muller; logp = -0.5 sum z^2 - A ln sigma - (A/2) ln 2 pi.  The GEMM is tiny, the
// noise is not: sixteen epilogue warps share the tile, four per group of 16 columns.
constexpr int kHeadEpiWarps = 16;
constexpr int kHeadThreads = 64 + 32 * kHeadEpiWarps;

template <int BLOCK_N>
__global__ void __launch_bounds__(kHeadThreads, 1) linear_tc_head_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                         const __grid_constant__ CUtensorMap map_b,
                                                                         const GemmParams P)
{
    using Plan = SmemPlan<BLOCK_N>;
    extern __shared__ uint8_t smem_raw[];
    const int A = P.N;
    const Pipe p = carve_pipe<Plan>(smem_raw, P.stages, Plan::head_epi_bytes(A));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = (P.M + BLOCK_M - 1) / BLOCK_M;             // one N tile holds the whole action row
    const int out_floats = 128 * A;
    // staging: per accumulator buffer the tile's mean and action rows laid out exactly as in global
    // memory ([128][A], dense), so a 32-row band leaves as one contiguous copy
    float *out_tiles = reinterpret_cast<float *>(p.epi);                            // [2][2][128 * A]
    float *zz_part = out_tiles + 2 * 2 * out_floats;                                // [2][4][128]
    int *band_count = reinterpret_cast<int *>(zz_part + 2 * 4 * 128);               // [2][4]
    float *s_bias = reinterpret_cast<float *>(band_count + 16);                     // [128]: bias of the tile's columns
    float *s_sigma = s_bias + 128;                                                  // [128]: standard deviation per column
    if (threadIdx.x < 8) band_count[threadIdx.x] = 0;
    pipe_init<Plan>(p, kHeadEpiWarps);
    const uint32_t tmem_base = *p.tmem_slot;
    dep_release();
    dep_wait();                       // nothing before this line touches global memory
    // the epilogue reads bias and sigma from shared memory as 16-byte words instead of one global load per output
    if (threadIdx.x < BLOCK_N) {
        const int cidx = threadIdx.x;
        s_bias[cidx] = __ldg(P.bias + cidx);
        s_sigma[cidx] = cidx < A ? (P.log_std ? expf(__ldg(P.log_std + cidx)) : P.sigma) : 0.0f;
    }
    __syncthreads();

    if (warp == 0) {
        if (lane == 0) producer_role<Plan, BLOCK_N>(p, &map_a, &map_b, P, n_tiles);
    } else if (warp == 1) {
        if (lane == 0) mma_role<Plan, BLOCK_N>(p, tmem_base, P, n_tiles);
    } else {
        const int quad = warp & 3;                                  // 32-row band of the tile (TMEM lane quadrant)
        const int group = (warp - 2) >> 2;                          // 16-column groups group, group+4, ...
        const int row_in_tile = quad * 32 + lane;
        constexpr int kGroups = (BLOCK_N / 16) < 4 ? (BLOCK_N / 16) : 4;
        const bool sample = P.action != nullptr;                     // a value head reads only the mean
        float logp_const = 0.0f;
        if (sample) {
            float sum_log = (float)A * logf(P.sigma);
            if (P.log_std) {                                         // same order in every thread
                sum_log = 0.0f;
                for (int i = 0; i < A; ++i) sum_log += __ldg(P.log_std + i);
            }
            logp_const = -sum_log - 0.5f * (float)A * 1.8378770664093453f;
        }
        int acc = 0;
        uint32_t acc_phase = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            const int m0 = tile * BLOCK_M;
            if (!mbar_wait(&p.acc_full[acc], acc_phase, p.abort_flag)) break;
            tc_fence_after();
            const int row = m0 + row_in_tile;
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * Plan::kAccStride);
            float *s_mean = out_tiles + (size_t)acc * 2 * out_floats;
            float *s_act = s_mean + out_floats;
            float zz = 0.0f;
            if (group < kGroups) {
#pragma unroll 1
                for (int c0 = 16 * group; c0 < BLOCK_N; c0 += 64) {
                    float v[16];
                    tmem_ld16(t_row + (uint32_t)c0, v);
                    if (c0 < A) {
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const int col = c0 + 4 * g;
                            if (col >= A) break;
                            float z[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                            if (sample) {
                                const uint4 x = philox4x32_10(make_uint4(P.env_id_base + (uint32_t)row, P.step,
                                                                         IM_STREAM_ACTION, (uint32_t)(col >> 2)),
                                                              make_uint2(P.seed_lo, P.seed_hi));
                                box_muller(x.x, x.y, z[0], z[1]);
                                box_muller(x.z, x.w, z[2], z[3]);
                            }
                            const float4 b4 = *reinterpret_cast<const float4 *>(s_bias + col);
                            const float4 s4 = *reinterpret_cast<const float4 *>(s_sigma + col);
                            const float bb[4] = {b4.x, b4.y, b4.z, b4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (col + i < A) {
                                    const float mu = v[4 * g + i] + bb[i];
                                    s_mean[row_in_tile * A + col + i] = mu;
                                    if (sample) s_act[row_in_tile * A + col + i] = mu + ss[i] * z[i];
                                    zz += z[i] * z[i];
                                }
                            }
                        }
                    }
                }
                zz_part[(acc * 4 + group) * 128 + row_in_tile] = zz;
            }
            tc_fence_before();
            // The last of the column-group warps to finish a 32-row band sums that band's partial z^2
            // in group order (so the result does not depend on which warp that is) and copies the
            // band's mean and action rows out as contiguous 16-byte stores.  The accumulator buffer,
            // and with it this staging buffer, is released only afterwards.
            if (group < kGroups) {
                __threadfence_block();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(&band_count[acc * 4 + quad], 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev == kGroups - 1) {
                    __threadfence_block();
                    if (lane == 0) band_count[acc * 4 + quad] = 0;
                    const int band_row0 = m0 + quad * 32;
                    int rows_valid = P.M - band_row0;
                    rows_valid = rows_valid > 32 ? 32 : rows_valid;
                    if (rows_valid > 0) {
                        if (P.logp && lane < rows_valid) {
                            float sum = 0.0f;
#pragma unroll
                            for (int g = 0; g < kGroups; ++g) sum += zz_part[(acc * 4 + g) * 128 + row_in_tile];
                            P.logp[row] = -0.5f * sum + logp_const;
                        }
                        const int count = rows_valid * A;                       // floats, contiguous in global
                        const float *src_m = s_mean + quad * 32 * A, *src_a = s_act + quad * 32 * A;
                        float *dst_m = P.mean + (size_t)band_row0 * A;
                        float *dst_a = sample ? P.action + (size_t)band_row0 * A : nullptr;
                        // both sides start on a 16-byte boundary: band offsets are multiples of 32 rows
                        const int n4 = count >> 2;
                        for (int i = lane; i < n4; i += 32) {
                            reinterpret_cast<float4 *>(dst_m)[i] = reinterpret_cast<const float4 *>(src_m)[i];
                            if (sample) reinterpret_cast<float4 *>(dst_a)[i] = reinterpret_cast<const float4 *>(src_a)[i];
                        }
                        for (int i = 4 * n4 + lane; i < count; i += 32) {
                            dst_m[i] = src_m[i];
                            if (sample) dst_a[i] = src_a[i];
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&p.acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }
    pipe_exit<Plan>(p, tmem_base, P.status);
}

// fp32 observations -> bf16 rows of a padded buffer; columns beyond `cols` are written as zero.
__global__ void obs_to_bf16_kernel(const float *__restrict__ obs, int ld_obs, int cols, __nv_bfloat16 *__restrict__ out,
                                   int ld_out, int n)
{
    const int chunks = ld_out / 8;
    const long long total = (long long)n * chunks;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(i / chunks), c = (int)(i % chunks) * 8;
        float v[8];
        if (c + 8 <= cols) {
            const float4 a = *reinterpret_cast<const float4 *>(obs + (size_t)r * ld_obs + c);
            const float4 b = *reinterpret_cast<const float4 *>(obs + (size_t)r * ld_obs + c + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = (c + k < cols) ? obs[(size_t)r * ld_obs + c + k] : 0.0f;
        }
        uint32_t pk[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
            pk[k] = *reinterpret_cast<const uint32_t *>(&h);
        }
        *reinterpret_cast<uint4 *>(out + (size_t)r * ld_out + c) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor map over a row-major [rows][ld] array; box = 64 columns x box_rows, 128B swizzle.
bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {BLOCK_K, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pick_block_n(int N, bool last)
{
    if (last) return (N + 15) / 16 * 16;            // one tile holds the whole action row
    if (N % 256 == 0) return 256;
    if (N % 128 == 0) return 128;
    return 64;
}

}  // namespace

struct TcLayer {
    int N, K, Kpad, block_n, n_tiles_n;
    __nv_bfloat16 *d_W;      // [n_tiles_n * block_n][Kpad], zero padded
    float *d_bias;           // [n_tiles_n * block_n]
    CUtensorMap map_a, map_b, map_c;    // map_c: the hidden-activation buffer this layer stores to
    CUtensorMap map_b2;                 // W in 128-row boxes: one CTA's half of a 256-column tile
    CUtensorMap map_m;                  // backward epilogue: the forward activations behind the ReLU mask (boxes like map_c)
};

}  // namespace im

struct im_policy_tc {
    std::vector<im::TcLayer> layers;
    __nv_bfloat16 *d_in;          // [max_batch][Kpad0] bf16 observations
    __nv_bfloat16 *d_hidden[2];   // [max_batch][max hidden]
    int ld_in, ld_hidden;
    int n_sm;
    const __nv_bfloat16 *ext_in;  // another policy's input buffer the first layer last read from (or null)
    CUtensorMap map_a_ext;        // first-layer operand map over ext_in
};

namespace im {

namespace {

// Launch with programmatic stream serialization (see dep_wait): the kernel's prologue overlaps the tail of the
// kernel before it in the stream.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <int BLOCK_N, bool BWD = false>
cudaError_t launch_hidden(const TcLayer &L, const GemmParams &gp_in, int n_sm, cudaStream_t stream)
{
    using Plan = SmemPlan<BLOCK_N>;
    static DeviceOnce once;                      // the attribute is per device
    {
        const cudaError_t e = once.run([] { return cudaFuncSetAttribute(linear_tc_hidden_kernel<BLOCK_N, false, BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit); });
        if (e != cudaSuccess) return e;
    }
    GemmParams gp = gp_in;
    gp.stages = Plan::stages_for(Plan::hidden_epi_bytes(BWD));
    const size_t smem = Plan::bytes(gp.stages, Plan::hidden_epi_bytes(BWD));
    const int tiles = ((gp.M + BLOCK_M - 1) / BLOCK_M) * gp.n_tiles_n * gp.n_batches;
    const int grid = tiles < n_sm ? tiles : n_sm;
    const cudaError_t le = launch_pdl(linear_tc_hidden_kernel<BLOCK_N, false, BWD>, dim3(grid), dim3(kThreads), smem, stream,
                                      L.map_a, L.map_b, L.map_c, L.map_m, gp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return le != cudaSuccess ? le : cudaGetLastError();
}

// 256-wide layers with enough rows to fill the machine run on CTA pairs.
// The same kernel with both operands stored [contraction rows][M or N columns].
template <int BLOCK_N>
cudaError_t launch_hidden_mn(const TcLayer &L, const GemmParams &gp_in, int n_sm, cudaStream_t stream)
{
    using Plan = SmemPlan<BLOCK_N>;
    static DeviceOnce once;                      // the attribute is per device
    {
        const cudaError_t e = once.run([] { return cudaFuncSetAttribute(linear_tc_hidden_kernel<BLOCK_N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit); });
        if (e != cudaSuccess) return e;
    }
    GemmParams gp = gp_in;
    gp.stages = Plan::stages_for(Plan::hidden_epi_bytes());
    const size_t smem = Plan::bytes(gp.stages, Plan::hidden_epi_bytes());
    const int tiles = ((gp.M + BLOCK_M - 1) / BLOCK_M) * gp.n_tiles_n * gp.n_batches;
    const int grid = tiles < n_sm ? tiles : n_sm;
    const cudaError_t le = launch_pdl(linear_tc_hidden_kernel<BLOCK_N, true>, dim3(grid), dim3(kThreads), smem, stream,
                                      L.map_a, L.map_b, L.map_c, L.map_c, gp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <bool BWD, bool MN = false>
cudaError_t launch_hidden_pair(const TcLayer &L, const GemmParams &gp, int n_sm, cudaStream_t stream)
{
    static DeviceOnce once;                      // the attribute is per device
    {
        const cudaError_t e = once.run([] { return cudaFuncSetAttribute(linear_tc_hidden_pair_kernel<BWD, MN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)pair_smem_bytes(BWD)); });
        if (e != cudaSuccess) return e;
    }
    const int tiles = ((gp.M + 2 * BLOCK_M - 1) / (2 * BLOCK_M)) * gp.n_tiles_n * (MN ? gp.n_batches : 1);
    const int pairs = tiles < n_sm / 2 ? tiles : n_sm / 2;
    const cudaError_t le = launch_pdl(linear_tc_hidden_pair_kernel<BWD, MN>, dim3(2 * pairs), dim3(pair_threads(BWD)), pair_smem_bytes(BWD), stream,
                                      L.map_a, MN ? L.map_b : L.map_b2, L.map_c, L.map_m, gp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <int BLOCK_N>
cudaError_t launch_head(const TcLayer &L, const GemmParams &gp_in, int n_sm, cudaStream_t stream)
{
    using Plan = SmemPlan<BLOCK_N>;
    static DeviceOnce once;                      // the attribute is per device
    {
        const cudaError_t e = once.run([] { return cudaFuncSetAttribute(linear_tc_head_kernel<BLOCK_N>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kSmemLimit); });
        if (e != cudaSuccess) return e;
    }
    GemmParams gp = gp_in;
    const int epi = Plan::head_epi_bytes(gp.N);
    gp.stages = Plan::stages_for(epi);
    if (gp.stages < 2) return cudaErrorInvalidValue;
    const size_t smem = Plan::bytes(gp.stages, epi);
    const int tiles = (gp.M + BLOCK_M - 1) / BLOCK_M;
    const int grid = tiles < n_sm ? tiles : n_sm;
    const cudaError_t le = launch_pdl(linear_tc_head_kernel<BLOCK_N>, dim3(grid), dim3(kHeadThreads), smem, stream, L.map_a, L.map_b, gp);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t dispatch_tc(const TcLayer &L, const GemmParams &gp, bool last, int n_sm, bool force_pairs, cudaStream_t stream)
{
    if (!last) {
        // CTA pairs pay off when the main loop is long enough to amortise the cluster set-up and there
        // are at least two waves of 256 x 256 tiles; otherwise the single-CTA kernel's finer tiles
        // balance the machine better (measured: 16384 x 1024 x 384 is 8 % faster single, 16384 x 1024 x 2048
        // 7 % faster paired)
        const int pair_tiles = ((gp.M + 2 * BLOCK_M - 1) / (2 * BLOCK_M)) * gp.n_tiles_n;
        const bool bwd = gp.mask || gp.colsum_partial;
        // (the backward epilogue is the longer part of a tile when K is short, and the pair kernel runs it on
        // eight warps: it takes those products whenever its tiles fill the machine)
        if (L.block_n == 256 && gp.n_batches == 1 &&
            (force_pairs || (pair_tiles >= n_sm && gp.K_blocks >= 8) || (bwd && pair_tiles >= n_sm / 2)))
            return bwd ? launch_hidden_pair<true>(L, gp, n_sm, stream) : launch_hidden_pair<false>(L, gp, n_sm, stream);
        switch (L.block_n) {
        case 256: return bwd ? launch_hidden<256, true>(L, gp, n_sm, stream) : launch_hidden<256>(L, gp, n_sm, stream);
        case 128: return bwd ? launch_hidden<128, true>(L, gp, n_sm, stream) : launch_hidden<128>(L, gp, n_sm, stream);
        default: return bwd ? launch_hidden<64, true>(L, gp, n_sm, stream) : launch_hidden<64>(L, gp, n_sm, stream);
        }
    }
    switch (L.block_n) {
    case 16: return launch_head<16>(L, gp, n_sm, stream);
    case 32: return launch_head<32>(L, gp, n_sm, stream);
    case 48: return launch_head<48>(L, gp, n_sm, stream);
    case 64: return launch_head<64>(L, gp, n_sm, stream);
    case 80: return launch_head<80>(L, gp, n_sm, stream);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace

im_status tc_policy_create(im_policy *p, const void *const *W, const float *const *b)
{
    const im_policy_config &cfg = p->cfg;
    const int nl = p->nl;
    if (nl < 2) return IM_ERR_UNSUPPORTED;
    for (int l = 1; l < nl; ++l)
        if (cfg.dims[l] % 64) return IM_ERR_UNSUPPORTED;
    if (cfg.dims[nl] > 80) return IM_ERR_UNSUPPORTED;      // staging of the head's output tiles is sized for this
    int dev = 0, cc_major = 0, n_sm = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (cc_major != 10 || !encode_tiled_fn()) return IM_ERR_UNSUPPORTED;

    im_policy_tc *tc = new (std::nothrow) im_policy_tc();
    if (!tc) return IM_ERR_ALLOC;
    p->tc = tc;
    tc->n_sm = n_sm;
    tc->d_in = nullptr;
    tc->ext_in = nullptr;
    tc->d_hidden[0] = tc->d_hidden[1] = nullptr;
    tc->layers.resize(nl);
    for (auto &L : tc->layers) { L.d_W = nullptr; L.d_bias = nullptr; }
    const size_t mb = (size_t)cfg.max_batch;
    int max_hidden = 64;
    for (int l = 1; l < nl; ++l) max_hidden = cfg.dims[l] > max_hidden ? cfg.dims[l] : max_hidden;
    tc->ld_in = (cfg.dims[0] + BLOCK_K - 1) / BLOCK_K * BLOCK_K;
    tc->ld_hidden = max_hidden;
    if (cudaMalloc(&tc->d_in, mb * tc->ld_in * 2) != cudaSuccess ||
        cudaMalloc(&tc->d_hidden[0], mb * max_hidden * 2) != cudaSuccess ||
        cudaMalloc(&tc->d_hidden[1], mb * max_hidden * 2) != cudaSuccess)
        return IM_ERR_ALLOC;

    for (int l = 0; l < nl; ++l) {
        TcLayer &L = tc->layers[l];
        const bool last = l == nl - 1;
        L.N = cfg.dims[l + 1];
        L.K = cfg.dims[l];
        L.Kpad = (L.K + BLOCK_K - 1) / BLOCK_K * BLOCK_K;
        L.block_n = pick_block_n(L.N, last);
        L.n_tiles_n = (L.N + L.block_n - 1) / L.block_n;
        const size_t rows = (size_t)L.n_tiles_n * L.block_n;
        std::vector<uint16_t> hw(rows * L.Kpad, 0);
        std::vector<float> hb(rows, 0.0f);
        const uint16_t *src = static_cast<const uint16_t *>(W[l]);
        for (int n = 0; n < L.N; ++n) {
            for (int k = 0; k < L.K; ++k) hw[(size_t)n * L.Kpad + k] = src[(size_t)n * L.K + k];
            hb[n] = b[l][n];
        }
        if (cudaMalloc(&L.d_W, hw.size() * 2) != cudaSuccess || cudaMalloc(&L.d_bias, hb.size() * 4) != cudaSuccess)
            return IM_ERR_ALLOC;
        if (cudaMemcpy(L.d_W, hw.data(), hw.size() * 2, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(L.d_bias, hb.data(), hb.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)
            return IM_ERR_CUDA;
        const __nv_bfloat16 *a_base = l == 0 ? tc->d_in : tc->d_hidden[(l - 1) & 1];
        const int a_ld = l == 0 ? tc->ld_in : tc->ld_hidden;
        if (!make_map(&L.map_a, a_base, mb, (uint64_t)L.Kpad, (uint64_t)a_ld, BLOCK_M) ||
            !make_map(&L.map_b, L.d_W, rows, (uint64_t)L.Kpad, (uint64_t)L.Kpad, (uint32_t)L.block_n))
            return IM_ERR_CUDA;
        if (!last && L.block_n == 256 && !make_map(&L.map_b2, L.d_W, rows, (uint64_t)L.Kpad, (uint64_t)L.Kpad, 128))
            return IM_ERR_CUDA;
        // hidden layers store 32-row x 64-column slabs of their output buffer
        if (!last && !make_map(&L.map_c, tc->d_hidden[l & 1], mb, rows, (uint64_t)tc->ld_hidden, 32))
            return IM_ERR_CUDA;
        L.map_m = L.map_c;               // the forward pass has no mask: a valid placeholder
    }
    return IM_OK;
}

void tc_policy_destroy(im_policy *p)
{
    im_policy_tc *tc = p->tc;
    if (!tc) return;
    for (auto &L : tc->layers) { cudaFree(L.d_W); cudaFree(L.d_bias); }
    cudaFree(tc->d_in); cudaFree(tc->d_hidden[0]); cudaFree(tc->d_hidden[1]);
    delete tc;
    p->tc = nullptr;
}

void tc_policy_layer(im_policy *p, int layer, void **W, int32_t *ld, float **bias)
{
    TcLayer &L = p->tc->layers[layer];
    *W = L.d_W;
    *ld = L.Kpad;
    *bias = L.d_bias;
}

void *tc_policy_input(im_policy *p, int32_t *ld)
{
    *ld = p->tc->ld_in;
    return p->tc->d_in;
}

// obs == nullptr: the bf16 input buffer has already been filled (by an attached environment); it is
// this policy's own buffer, or that of `src` (same input width), whose rows the first layer then reads
// through a tensor map built on first use.  action_out == nullptr: no sampling, only the mean is written.
im_status tc_policy_forward(im_policy *p, uint32_t step, int32_t n, const float *obs, int32_t ld_obs,
                            float *mean_out, float *action_out, float *logp_out, im_policy *src)
{
    im_policy_tc *tc = p->tc;
    const im_policy_config &cfg = p->cfg;
    const bool external = !obs && src && src != p;
    if (external) {
        im_policy_tc *st = src->tc;
        if (!st || st->ld_in != tc->ld_in || src->cfg.dims[0] != cfg.dims[0] || src->cfg.max_batch < n)
            return IM_ERR_INVALID_ARG;
        if (tc->ext_in != st->d_in) {
            const TcLayer &L0 = tc->layers[0];
            if (!make_map(&tc->map_a_ext, st->d_in, (uint64_t)src->cfg.max_batch, (uint64_t)L0.Kpad, (uint64_t)st->ld_in,
                          BLOCK_M))
                return IM_ERR_CUDA;
            tc->ext_in = st->d_in;
        }
    }
    if (obs) {
        const long long chunks = (long long)n * (tc->ld_in / 8);
        const int block = 256;
        long long grid = (chunks + block - 1) / block;
        if (grid > 148 * 16) grid = 148 * 16;
        obs_to_bf16_kernel<<<(int)grid, block, 0, p->stream>>>(obs, ld_obs, cfg.dims[0], tc->d_in, tc->ld_in, n);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return IM_ERR_CUDA;
    }
    for (int l = 0; l < p->nl; ++l) {
        TcLayer L = tc->layers[l];
        if (l == 0 && external) L.map_a = tc->map_a_ext;
        const bool last = l == p->nl - 1;
        GemmParams gp;
        std::memset(&gp, 0, sizeof(gp));
        gp.M = n; gp.N = L.N; gp.K_blocks = L.Kpad / BLOCK_K; gp.n_tiles_n = L.n_tiles_n; gp.bias = L.d_bias;
        gp.act_floor = 0.0f;
        gp.n_batches = 1; gp.a_batch_rows = 0; gp.b_batch_rows = 0; gp.c_batch_rows = 0;
        gp.mean = mean_out; gp.action = action_out; gp.logp = logp_out;
        gp.sigma = cfg.sigma; gp.log_std = p->d_log_std; gp.seed_lo = (uint32_t)cfg.seed; gp.seed_hi = (uint32_t)(cfg.seed >> 32);
        gp.step = step; gp.env_id_base = cfg.env_id_base; gp.status = p->d_status;
        if (dispatch_tc(L, gp, last, tc->n_sm, cfg.impl == 2, p->stream) != cudaSuccess) return IM_ERR_CUDA;
    }
    return IM_OK;
}


cudaError_t tc_set_wait_debug(unsigned long long limit_ns, int skip_loads)
{
    cudaError_t e = cudaMemcpyToSymbol(g_wait_limit_ns, &limit_ns, sizeof(limit_ns));
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_skip_loads, &skip_loads, sizeof(skip_loads));
    return e;
}

// C[M][N] = act(A[M][K] B[N][K]^T + bias) on the hidden-layer kernels, operands anywhere in device
// memory: the three tensor maps are encoded for this call and travel as kernel parameters.
im_status tc_gemm(const void *A, int64_t lda, const void *B, int64_t ldb, void *C, int64_t ldc, int M, int N, int K,
                  const float *bias, bool relu, uint32_t *status, cudaStream_t stream, int batches, const void *mask,
                  int64_t ld_mask, float *colsum_partial, int ld_partial)
{
    const int n_sm = device_sm_count();          // 0 unless the current device is an sm_100 part
    if (n_sm <= 0 || !encode_tiled_fn()) return IM_ERR_UNSUPPORTED;
    TcLayer L;
    L.N = N; L.K = K; L.Kpad = K;
    L.block_n = pick_block_n(N, false);
    L.n_tiles_n = N / L.block_n;
    L.d_W = nullptr; L.d_bias = nullptr;
    const uint64_t nb = (uint64_t)batches;
    if (!make_map(&L.map_a, A, nb * (uint64_t)M, (uint64_t)K, (uint64_t)lda, BLOCK_M) ||
        !make_map(&L.map_b, B, nb * (uint64_t)N, (uint64_t)K, (uint64_t)ldb, (uint32_t)L.block_n) ||
        !make_map(&L.map_c, C, nb * (uint64_t)M, (uint64_t)N, (uint64_t)ldc, 32))
        return IM_ERR_CUDA;
    if (L.block_n == 256 && !make_map(&L.map_b2, B, nb * (uint64_t)N, (uint64_t)K, (uint64_t)ldb, 128)) return IM_ERR_CUDA;
    L.map_m = L.map_c;
    if (mask && !make_map(&L.map_m, mask, (uint64_t)M, (uint64_t)N, (uint64_t)ld_mask, 32)) return IM_ERR_CUDA;
    GemmParams gp;
    std::memset(&gp, 0, sizeof(gp));
    gp.M = M; gp.N = N; gp.K_blocks = K / BLOCK_K; gp.n_tiles_n = L.n_tiles_n; gp.bias = bias;
    gp.act_floor = relu ? 0.0f : -INFINITY;
    gp.n_batches = batches; gp.a_batch_rows = M; gp.b_batch_rows = N; gp.c_batch_rows = M;
    if (mask || colsum_partial) gp.bias = nullptr;         // the backward product has no bias: its epilogue skips the add
    gp.mask = static_cast<const __nv_bfloat16 *>(mask); gp.ld_mask = ld_mask;
    gp.colsum_partial = colsum_partial; gp.ld_partial = ld_partial;
    gp.status = status;
    return dispatch_tc(L, gp, false, n_sm, false, stream) == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}


// C_s[Mo][No] = sum over the rows r of slice s of A[r][0..Mo) (x) B[r][0..No)  (bf16, fp32 accumulation):
// the transposed product A^T B of two row-major matrices over `slices` equal row ranges, the partial
// results stacked with a pitch of `c_pitch` rows.  Operands are read M/N-major, so no transposed copy
// of either matrix is needed.
im_status tc_gemm_tn(const void *A, int64_t lda, const void *B, int64_t ldb, void *C, int64_t ldc, int R, int Mo, int No,
                     int slices, int c_pitch, uint32_t *status, cudaStream_t stream)
{
    const int n_sm = device_sm_count();          // 0 unless the current device is an sm_100 part
    if (n_sm <= 0 || !encode_tiled_fn()) return IM_ERR_UNSUPPORTED;
    TcLayer L;
    L.N = No; L.K = R / slices; L.Kpad = L.K;
    // wide outputs take 256-column tiles even when that leaves a ragged last tile (640 columns: three tiles,
    // a sixth of the MMAs wasted, against five 128-column tiles at little more than half the tensor-pipe rate);
    // TMA fills the operand columns past No with zeros and clips the stores
    L.block_n = No > 256 ? 256 : pick_block_n(No, false);
    L.n_tiles_n = (No + L.block_n - 1) / L.block_n;
    L.d_W = nullptr; L.d_bias = nullptr;
    if (!make_map(&L.map_a, A, (uint64_t)R, (uint64_t)Mo, (uint64_t)lda, 64) ||
        !make_map(&L.map_b, B, (uint64_t)R, (uint64_t)No, (uint64_t)ldb, 64) ||
        !make_map(&L.map_c, C, (uint64_t)slices * (uint64_t)c_pitch, (uint64_t)No, (uint64_t)ldc, 32))
        return IM_ERR_CUDA;
    GemmParams gp;
    std::memset(&gp, 0, sizeof(gp));
    gp.M = Mo; gp.N = No; gp.K_blocks = (R / slices) / BLOCK_K; gp.n_tiles_n = L.n_tiles_n; gp.bias = nullptr;    // no bias in this product
    gp.act_floor = -INFINITY;
    gp.n_batches = slices; gp.a_batch_rows = R / slices; gp.b_batch_rows = 0; gp.c_batch_rows = c_pitch;
    gp.status = status;
    cudaError_t e;
    // CTA pairs (256 x 256 tiles, half of the N operand per SM) when the output splits into whole 256-row tiles,
    // the slices' pitch keeps those tiles apart and there are tiles for most pairs
    const int pair_tiles = ((Mo + 255) / 256) * L.n_tiles_n * slices;
    if (L.block_n == 256 && Mo % 256 == 0 && c_pitch % 256 == 0 && pair_tiles >= n_sm / 3 && gp.K_blocks >= 8) {
        L.map_m = L.map_c;
        return launch_hidden_pair<false, true>(L, gp, n_sm, stream) == cudaSuccess ? IM_OK : IM_ERR_CUDA;
    }
    switch (L.block_n) {
    case 256: e = launch_hidden_mn<256>(L, gp, n_sm, stream); break;
    case 128: e = launch_hidden_mn<128>(L, gp, n_sm, stream); break;
    default: e = launch_hidden_mn<64>(L, gp, n_sm, stream); break;
    }
    return e == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

// mean[M][N] (fp32, dense) = A[M][K] B[N][K]^T + bias on the Gaussian-head kernel without sampling.
// B must hold ceil(N / 16) * 16 rows (rows beyond N zero), bias as many floats.
im_status tc_gemm_head(const void *A, int64_t lda, const void *B, int64_t ldb, int M, int N, int K, const float *bias,
                       float *mean_out, uint32_t *status, cudaStream_t stream)
{
    const int n_sm = device_sm_count();          // 0 unless the current device is an sm_100 part
    if (n_sm <= 0 || !encode_tiled_fn()) return IM_ERR_UNSUPPORTED;
    TcLayer L;
    L.N = N; L.K = K; L.Kpad = K;
    L.block_n = pick_block_n(N, true);
    L.n_tiles_n = 1;
    L.d_W = nullptr; L.d_bias = nullptr;
    if (!make_map(&L.map_a, A, (uint64_t)M, (uint64_t)K, (uint64_t)lda, BLOCK_M) ||
        !make_map(&L.map_b, B, (uint64_t)L.block_n, (uint64_t)K, (uint64_t)ldb, (uint32_t)L.block_n))
        return IM_ERR_CUDA;
    GemmParams gp;
    std::memset(&gp, 0, sizeof(gp));
    gp.M = M; gp.N = N; gp.K_blocks = K / BLOCK_K; gp.n_tiles_n = 1; gp.bias = bias;
    gp.mean = mean_out; gp.sigma = 1.0f;
    gp.n_batches = 1;
    gp.status = status;
    return dispatch_tc(L, gp, true, n_sm, false, stream) == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // namespace im
