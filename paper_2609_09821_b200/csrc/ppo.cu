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
    float *partial;                        // [partial rows][kPartial]
    long long row_begin;                   // the generic kernel handles rows [row_begin, M) ...
    int partial_begin;                     // ... and writes its partial rows from this one on
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

// Per-lane constants of the action dimensions k = sl + LPR i a lane owns, and per-batch scalars.
template <int NI>
struct RowConsts {
    float inv_sg[NI], so2[NI], dls[NI];
    float logp_const, adv_mean, adv_rstd, eps, cv, inv_M;
    int clip_value;
};

// Per-lane running sums over the rows a lane has seen.
template <int NI>
struct Acc {
    float ls[NI];                          // dL/dlog_std_k without the entropy term
    float surr, vl, kl, clip;
};

template <int LPR, int NI>
__device__ __forceinline__ void setup_lane(const PpoParams &P, int sl, RowConsts<NI> &C, Acc<NI> &acc)
{
    float sum_log = 0.0f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int k = sl + LPR * i;
        const bool ok = k < P.A;
        const float ls = ok ? __ldg(P.b.log_std + k) : 0.0f;
        const float lo = ok ? __ldg(P.b.log_std_old + k) : 0.0f;
        C.inv_sg[i] = expf(-ls);
        C.so2[i] = expf(2.0f * lo);
        C.dls[i] = ls - lo;
        acc.ls[i] = 0.0f;
        sum_log += ls;
    }
    sum_log = group_sum<LPR>(sum_log);
    C.logp_const = -sum_log - 0.5f * (float)P.A * 1.8378770664093453f;
    C.adv_mean = 0.0f; C.adv_rstd = 1.0f;
    if (P.b.adv_moments) { C.adv_mean = __ldg(P.b.adv_moments); C.adv_rstd = __ldg(P.b.adv_moments + 1); }
    C.eps = P.cfg.clip; C.cv = P.cfg.value_coef; C.inv_M = 1.0f / (float)P.M;
    C.clip_value = P.cfg.clip_value_loss;
    acc.surr = acc.vl = acc.kl = acc.clip = 0.0f;
}

// One sample row, worked on by the LPR lanes of a group (all 32 lanes of the warp must call this:
// the reductions are warp shuffles).  mean / mean_old / action point at the row's A values, sc at its
// five scalars (logp_old, advantage, value, returns, value_old); d_mean_row receives dL/dmu.
// Returns dL/dV of the row.
template <int LPR, int NI>
__device__ __forceinline__ float process_row(const RowConsts<NI> &C, int A, int sl, bool in, const float *mean,
                                             const float *mean_old, const float *action, const float *sc,
                                             float *d_mean_row, Acc<NI> &acc)
{
    float z[NI], zz = 0.0f, kl = 0.0f;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int k = sl + LPR * i;
        z[i] = 0.0f;
        if (in && k < A) {
            const float mu = mean[k];
            const float dm = mean_old[k] - mu;
            z[i] = (action[k] - mu) * C.inv_sg[i];
            zz = fmaf(z[i], z[i], zz);
            kl += C.dls[i] + 0.5f * (C.so2[i] + dm * dm) * C.inv_sg[i] * C.inv_sg[i] - 0.5f;
        }
    }
    zz = group_sum<LPR>(zz);
    kl = group_sum<LPR>(kl);
    if (!in) return 0.0f;
    const float r = expf(fmaf(-0.5f, zz, C.logp_const) - sc[0]);
    const float ah = (sc[1] - C.adv_mean) * C.adv_rstd;
    const float rc = fminf(fmaxf(r, 1.0f - C.eps), 1.0f + C.eps);
    const float s1 = r * ah, s2 = rc * ah;
    const bool live = s1 <= s2;                            // the unclipped branch is the minimum
    const float coef = live ? -ah * r * C.inv_M : 0.0f;    // dL/dlogp_i
    acc.surr -= live ? s1 : s2;
    acc.clip += fabsf(r - 1.0f) > C.eps ? 1.0f : 0.0f;
    acc.kl += kl;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int k = sl + LPR * i;
        if (k < A) {
            d_mean_row[k] = coef * z[i] * C.inv_sg[i];
            acc.ls[i] = fmaf(coef, fmaf(z[i], z[i], -1.0f), acc.ls[i]);
        }
    }
    const float v = sc[2], Rt = sc[3];
    const float e1 = v - Rt;
    float vl = e1 * e1, gv = 2.0f * e1;
    if (C.clip_value) {
        const float vo = sc[4];
        const float d = v - vo, dc = fminf(fmaxf(d, -C.eps), C.eps);
        const float e2 = vo + dc - Rt;
        if (e2 * e2 > vl) { vl = e2 * e2; gv = d == dc ? 2.0f * e2 : 0.0f; }
    }
    acc.vl += vl;
    return C.cv * gv * C.inv_M;
}

// Folds the warp's groups (the same k sits in lane sl of every group), then the CTA's warps in
// order, and writes the CTA's partial row.
template <int LPR, int NI, int W>
__device__ __forceinline__ void fold_and_write(Acc<NI> &acc, float (*s_acc)[kPartial], float *partial_row)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane / LPR, sl = lane % LPR;
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int i = 0; i < NI; ++i) acc.ls[i] += __shfl_xor_sync(0xffffffffu, acc.ls[i], o);
        acc.surr += __shfl_xor_sync(0xffffffffu, acc.surr, o);
        acc.vl += __shfl_xor_sync(0xffffffffu, acc.vl, o);
        acc.kl += __shfl_xor_sync(0xffffffffu, acc.kl, o);
        acc.clip += __shfl_xor_sync(0xffffffffu, acc.clip, o);
    }
    for (int j = lane; j < kPartial; j += 32) s_acc[warp][j] = 0.0f;
    __syncwarp();
    if (grp == 0) {
#pragma unroll
        for (int i = 0; i < NI; ++i)
            if (sl + LPR * i < kMaxA) s_acc[warp][sl + LPR * i] = acc.ls[i];
    }
    if (lane == 0) {
        s_acc[warp][kMaxA + 0] = acc.surr; s_acc[warp][kMaxA + 1] = acc.vl;
        s_acc[warp][kMaxA + 2] = acc.kl;   s_acc[warp][kMaxA + 3] = acc.clip;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < kPartial; j += blockDim.x) {
        float t = 0.0f;
        for (int w = 0; w < W; ++w) t += s_acc[w][j];
        partial_row[j] = t;
    }
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
    RowConsts<NI> C;
    Acc<NI> acc;
    setup_lane<LPR, NI>(P, sl, C, acc);

    // A lane reads back only what it copied itself (element k of the three arrays); the five per-row
    // scalars are copied by the group's lanes 0..4 and read by all of its lanes after a __syncwarp.
    float *ring = s_ring[warp][grp][0];
    const long long stride = (long long)gridDim.x * kWarps * kGroups;
    const long long first = P.row_begin + ((long long)blockIdx.x * kWarps + warp) * kGroups + grp;
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
    const long long warp_first = P.row_begin + ((long long)blockIdx.x * kWarps + warp) * kGroups;
    for (long long row0 = warp_first; row0 < P.M; row0 += stride) {
        const long long row = row0 + grp;
        const bool in = row < P.M;
        issue(row + (kDepth - 1) * stride, (slot + kDepth - 1) % kDepth);
        cp_async_wait<kDepth - 1>();
        __syncwarp();
        const float *cur = ring + slot * kSlotFloats;
        const float dv = process_row<LPR, NI>(C, A, sl, in, cur, cur + kRow, cur + 2 * kRow, cur + 3 * kRow,
                                              P.d_mean + (size_t)row * (size_t)A, acc);
        if (in && sl == 0) P.d_value[row] = dv;
        __syncwarp();                                      // every lane is done with the slot before it is refilled
        slot = slot + 1 == kDepth ? 0 : slot + 1;
    }
    cp_async_wait<0>();
    fold_and_write<LPR, NI, kWarps>(acc, s_acc, P.partial + (size_t)(P.partial_begin + blockIdx.x) * kPartial);
}

// ------------------------------------------------------------------ bulk-copy path
// When the arrays are 16-byte aligned, whole tiles of kTileRows rows are moved by the copy engine:
// the rows of a tile are one contiguous run in each array (kTileRows A floats, a multiple of 16
// bytes because kTileRows is a multiple of 32), so one elected thread fetches a tile with eight bulk
// copies that signal an mbarrier, and sends the finished d_mean / d_value tile back with two bulk
// stores -- no per-element load, store or address instruction is left in the row loop.  Two stages:
// the next tile is in flight while the current one is worked on.  The CTAs stride over the full
// tiles; the rows after the last full tile go to the generic kernel.
// Warps per CTA: enough that a 32-row tile gives every warp two or more trips (8-lane groups: four
// rows per warp and trip, so 4 warps; wider groups: 8 warps).
__host__ __device__ constexpr int bulk_warps(int LPR) { return LPR == 8 ? 4 : 8; }
// Limit of the bounded waits below (2 s unless im_debug_set_wait changed it) and the diagnostic switch that makes
// the bulk-copy kernel fetch nothing, so that a test can watch a wait run out with no copy in flight.
__device__ unsigned long long g_wait_limit_ns = 2000000000ull;
__device__ int g_skip_loads = 0;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// Bounded wait: false when the limit ran out or another thread of the CTA already gave up.
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
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, const void *src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Floats of one stage: three input tiles and the output tile (kTileRows x A each), five input
// scalar columns and the d_value column (kTileRows each).  Every piece starts on a 16-byte boundary.
__host__ __device__ inline int stage_floats(int A, int T) { return T * (4 * A + 6); }
// 32 rows at every width: taller tiles for narrow rows cost more in occupancy (shared memory) than
// they save in per-tile barriers (measured at A = 28: 128-row tiles 87 us, 32-row tiles 70 us per 512 k rows).
__host__ inline int tile_rows_for(int) { return 32; }

template <int LPR, int NI>
__global__ void __launch_bounds__(32 * bulk_warps(LPR)) ppo_loss_bulk_kernel(const PpoParams P, long long n_tiles, int kTileRows)
{
    constexpr int kGroups = 32 / LPR, kBulkWarps = bulk_warps(LPR);
    extern __shared__ __align__(128) float s_stage[];      // [2][stage_floats]
    __shared__ float s_acc[kBulkWarps][kPartial];
    __shared__ __align__(8) uint64_t s_bar[2];
    __shared__ int s_abort;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = lane / LPR, sl = lane % LPR;
    const int A = P.A;
    const int TA = kTileRows * A, SF = stage_floats(A, kTileRows);
    RowConsts<NI> C;
    Acc<NI> acc;
    setup_lane<LPR, NI>(P, sl, C, acc);
    if (threadIdx.x == 0) {
        mbar_init(&s_bar[0], 1);
        mbar_init(&s_bar[1], 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const bool with_vold = P.cfg.clip_value_loss != 0;
    auto fetch = [&](long long tile, int s) {               // thread 0 only
        if (g_skip_loads) return;                           // diagnostic: the first wait runs out
        float *st = s_stage + (size_t)s * SF;
        const size_t r0 = (size_t)tile * kTileRows, e0 = r0 * (size_t)A;
        const uint32_t tile_bytes = (uint32_t)TA * 4u, col_bytes = (uint32_t)kTileRows * 4u;
        mbar_arrive_expect_tx(&s_bar[s], 3u * tile_bytes + (with_vold ? 5u : 4u) * col_bytes);
        bulk_load(st, P.b.mean + e0, tile_bytes, &s_bar[s]);
        bulk_load(st + TA, P.b.mean_old + e0, tile_bytes, &s_bar[s]);
        bulk_load(st + 2 * TA, P.b.action + e0, tile_bytes, &s_bar[s]);
        float *sc = st + 3 * TA;
        bulk_load(sc, P.b.logp_old + r0, col_bytes, &s_bar[s]);
        bulk_load(sc + kTileRows, P.b.advantage + r0, col_bytes, &s_bar[s]);
        bulk_load(sc + 2 * kTileRows, P.b.value + r0, col_bytes, &s_bar[s]);
        bulk_load(sc + 3 * kTileRows, P.b.returns + r0, col_bytes, &s_bar[s]);
        if (with_vold) bulk_load(sc + 4 * kTileRows, P.b.value_old + r0, col_bytes, &s_bar[s]);
    };

    uint32_t phases = 0u;                                   // bit s: parity stage s is waited on next
    if (threadIdx.x == 0 && (long long)blockIdx.x < n_tiles) fetch(blockIdx.x, 0);
    int s = 0;
    for (long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, s ^= 1) {
        // the other stage's inputs were last read before the barrier that ended the previous tile
        if (threadIdx.x == 0 && tile + gridDim.x < n_tiles) fetch(tile + gridDim.x, s ^ 1);
        const bool ok = mbar_wait(&s_bar[s], (phases >> s) & 1u, &s_abort);
        phases ^= 1u << s;
        if (__syncthreads_or(!ok)) break;                   // leave together if any thread's wait ran out
        float *st = s_stage + (size_t)s * SF;
        const float *sc = st + 3 * TA;
        float *out = st + 3 * TA + 5 * kTileRows;           // d_value column, then the d_mean tile
        float *out_mean = out + kTileRows;
#pragma unroll 1
        for (int r = warp * kGroups + grp; r < kTileRows; r += kBulkWarps * kGroups) {
            float scal[5] = {sc[r], sc[kTileRows + r], sc[2 * kTileRows + r], sc[3 * kTileRows + r],
                             with_vold ? sc[4 * kTileRows + r] : 0.0f};
            const float dv = process_row<LPR, NI>(C, A, sl, true, st + r * A, st + TA + r * A, st + 2 * TA + r * A, scal,
                                                  out_mean + r * A, acc);
            if (sl == 0) out[r] = dv;
        }
        fence_proxy_async();                                // the tile written above is read by the copy engine
        if (threadIdx.x == 0) bulk_wait_read_all();         // the previous tile's stores have left the other stage
        __syncthreads();
        if (threadIdx.x == 0) {
            const size_t r0 = (size_t)tile * kTileRows;
            bulk_store(P.d_value + r0, out, (uint32_t)kTileRows * 4u);
            bulk_store(P.d_mean + r0 * (size_t)A, out_mean, (uint32_t)TA * 4u);
            bulk_commit();
        }
    }
    if (threadIdx.x == 0) {
        bulk_wait_all();
        if (s_abort) {                                      // give copies still in flight a bounded chance to land
            volatile int ignore = 0;
            mbar_wait(&s_bar[0], phases & 1u, &ignore);
            mbar_wait(&s_bar[1], (phases >> 1) & 1u, &ignore);
        }
    }
    __syncthreads();
    if (s_abort) acc.surr = __int_as_float(0x7fc00000);     // a wait ran out: the summary turns NaN
    fold_and_write<LPR, NI, kBulkWarps>(acc, s_acc, P.partial + (size_t)(P.partial_begin + blockIdx.x) * kPartial);
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

cudaError_t ppo_set_wait_debug(unsigned long long limit_ns, int skip_loads)
{
    cudaError_t e = cudaMemcpyToSymbol(g_wait_limit_ns, &limit_ns, sizeof(limit_ns));
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_skip_loads, &skip_loads, sizeof(skip_loads));
    return e;
}

}  // namespace im

extern "C" {

size_t im_ppo_workspace_bytes(void) { return (size_t)(2 * im::kMaxGrid) * im::kPartial * sizeof(float); }

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
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // lanes per row and rounds: rows up to 32 floats on 8 lanes, up to 80 on 16, wider ones on a whole warp
#define IM_PPO_DISPATCH(CALL)                                   \
    if (A <= 32) {                                              \
        switch ((A + 7) / 8) {                                  \
        case 1: CALL(8, 1); break;                              \
        case 2: CALL(8, 2); break;                              \
        case 3: CALL(8, 3); break;                              \
        default: CALL(8, 4); break;                             \
        }                                                       \
    } else if (A <= 80) {                                       \
        switch ((A + 15) / 16) {                                \
        case 3: CALL(16, 3); break;                             \
        case 4: CALL(16, 4); break;                             \
        default: CALL(16, 5); break;                            \
        }                                                       \
    } else if (A <= 96) {                                       \
        CALL(32, 3);                                            \
    } else {                                                    \
        CALL(32, 4);                                            \
    }
    // full tiles through the bulk-copy kernel when every array allows 16-byte transfers
    const auto al16 = [](const void *q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; };
    const bool bulk_ok = al16(batch->mean) && al16(batch->mean_old) && al16(batch->action) && al16(batch->logp_old) &&
                         al16(batch->advantage) && al16(batch->value) && al16(batch->returns) &&
                         (!cfg->clip_value_loss || al16(batch->value_old)) && al16(d_mean) && al16(d_value);
    const int T = tile_rows_for(A);
    const long long n_tiles = bulk_ok ? M / T : 0;
    int grid_bulk = 0;
    if (n_tiles > 0) {
        int dev = 0, n_sm = 0, max_smem = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        const size_t smem = 2 * (size_t)stage_floats(A, T) * sizeof(float);
        p.row_begin = 0; p.partial_begin = 0;
#define IM_PPO_BULK(LPR, NI)                                                                                        \
        do {                                                                                                        \
            static DeviceOnce once;   /* the attribute is per device */                                           \
            if (once.run([&] {                                                                                      \
                    return cudaFuncSetAttribute(ppo_loss_bulk_kernel<LPR, NI>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                max_smem - 8192);   /* static part: 4.3 KB */                     \
                }) != cudaSuccess)                                                                                  \
                return IM_ERR_CUDA;                                                                                 \
            int per_sm = 1;   /* persistent grid: as many CTAs as are resident at once */                         \
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ppo_loss_bulk_kernel<LPR, NI>,                   \
                                                          32 * bulk_warps(LPR), smem);                              \
            per_sm = per_sm < 1 ? 1 : per_sm;                                                                       \
            const long long gb = (long long)n_sm * per_sm;                                                          \
            grid_bulk = (int)(gb > n_tiles ? n_tiles : gb);                                                         \
            if (grid_bulk > kMaxGrid) grid_bulk = kMaxGrid;                                                         \
            ppo_loss_bulk_kernel<LPR, NI><<<grid_bulk, 32 * bulk_warps(LPR), smem, st>>>(p, n_tiles, T);            \
        } while (0)
        IM_PPO_DISPATCH(IM_PPO_BULK)
#undef IM_PPO_BULK
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    // the rows after the last full tile (all rows without the bulk path) through the generic kernel
    const long long rest = M - n_tiles * T;
    int grid = 0;
    if (rest > 0) {
        long long g = (rest + kWarps * 16 - 1) / (kWarps * 16);  // a few trips per warp
        grid = (int)(g < 1 ? 1 : (g > kMaxGrid ? kMaxGrid : g));
        p.row_begin = n_tiles * T; p.partial_begin = grid_bulk;
#define IM_PPO_LAUNCH(LPR, NI) ppo_loss_kernel<LPR, NI><<<grid, 32 * kWarps, 0, st>>>(p)
        IM_PPO_DISPATCH(IM_PPO_LAUNCH)
#undef IM_PPO_LAUNCH
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
#undef IM_PPO_DISPATCH
    grid += grid_bulk;
    ppo_finish_kernel<<<1, kFinishGroups * kPartial, 0, st>>>(p, grid);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? IM_OK : IM_ERR_CUDA;
}

}  // extern "C"
