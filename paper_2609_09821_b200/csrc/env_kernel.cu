// Fused environment step: reference lookup + slerp + forward kinematics,
// error terms and reward, flags, masked Philox reset, heading-local
// observation (the post-physics phase of the paper's Figure 2 as one kernel).
//
// Mapping: one CTA handles 32 consecutive envs; warp j handles body j and lane
// e handles env e of the tile, so every global load of the structure-of-arrays
// body state is one fully used 128-byte line per warp.  Cross-body data (the
// kinematic chain, reward partial sums, root heading) goes through shared
// memory; the observation tile is transposed in shared memory so that rows of
// the row-major [N][ld_obs] output are written as whole lines.
#include "im_internal.h"
#include "im_device.cuh"

namespace im {

namespace {

constexpr int kTile = 32;          // envs per CTA
constexpr int kRefComps = 7;       // local quaternion + child-frame joint angular velocity
constexpr int kTgtComps = 4;       // local quaternion
constexpr int kSimComps = 7;       // world quaternion + world angular velocity (read by children)
constexpr int kPartials = 9;       // pose, vel, ee_pos, ee_rot, body_pos, body_vel, weighted com difference (3)

struct Smem {
    float *ref, *tgt, *rootp, *rootv, *tgt_rootp, *head;   // head: root x, root y, cos, sin
    int *cur_clip, *mask, *any;
    float *cur_t;
    float *simx, *part, *tile;                             // tile aliases simx + part
};

__host__ __device__ inline size_t smem_floats(int J)
{
    const int D = 24 * J + 1;
    const size_t fixed = (size_t)J * (kRefComps + kTgtComps) * kTile + 9 * kTile + 4 * kTile + 3 * kTile + kTile;
    const size_t a = (size_t)J * (kSimComps + kPartials) * kTile;
    const size_t b = (size_t)kTile * D;
    return fixed + (a > b ? a : b);
}

__device__ __forceinline__ Smem carve(float *base, int J)
{
    Smem s;
    float *p = base;
    s.ref = p;        p += J * kRefComps * kTile;
    s.tgt = p;        p += J * kTgtComps * kTile;
    s.rootp = p;      p += 3 * kTile;
    s.rootv = p;      p += 3 * kTile;
    s.tgt_rootp = p;  p += 3 * kTile;
    s.head = p;       p += 4 * kTile;
    s.cur_clip = reinterpret_cast<int *>(p);  p += kTile;
    s.mask = reinterpret_cast<int *>(p);      p += kTile;
    s.cur_t = p;      p += kTile;
    s.any = reinterpret_cast<int *>(p);       p += kTile;
    s.simx = p;
    s.part = p + J * kSimComps * kTile;
    s.tile = p;
    return s;
}

// Keyframe row and blend factor at `time` (step a1): f = fl32(time * fps),
// k = min(floor f, K - 2), alpha = f - k (exact in fp32).
__device__ __forceinline__ void lookup(const ClipMeta &m, float time, int &row, float &alpha)
{
    const float f = __fmul_rn(time, m.fps);
    int k = (int)floorf(f);
    k = min(k, m.K - 2);
    k = max(k, 0);
    alpha = fminf(fmaxf(f - (float)k, 0.0f), 1.0f);
    row = m.start + k;
}

__device__ __forceinline__ Quat ld_quat(const float4 *p)
{
    const float4 v = __ldg(p);
    return {v.x, v.y, v.z, v.w};
}

// Shortest-arc slerp of one joint plus, if asked, the joint's angular velocity
// in the child frame, 2 log(q0* q1) fps.  The vector part of q0* q1 is formed
// from q1 - q0, which avoids the cancellation of the direct product when the
// keyframes are close and keeps the velocity accurate to ~1e-6 rad/s.
template <bool VEL>
__device__ __forceinline__ void slerp_joint(Quat q0, Quat q1, float alpha, float fps, Quat &q, Vec3 &wl)
{
    float d = q0.w * q1.w + q0.x * q1.x + q0.y * q1.y + q0.z * q1.z;
    if (d < 0.0f) { d = -d; q1 = {-q1.w, -q1.x, -q1.y, -q1.z}; }
    const Quat diff = {q1.w - q0.w, q1.x - q0.x, q1.y - q0.y, q1.z - q0.z};
    const Quat c = qmul(qconj(q0), diff);
    const float n = sqrtf(c.x * c.x + c.y * c.y + c.z * c.z);
    const float theta = atan2f(n, d);
    float s0, s1;
    if (d > 1.0f - 1e-6f) { s0 = 1.0f - alpha; s1 = alpha; }
    else {
        const float inv = 1.0f / n;
        s0 = sinf((1.0f - alpha) * theta) * inv;
        s1 = sinf(alpha * theta) * inv;
    }
    Quat r = {s0 * q0.w + s1 * q1.w, s0 * q0.x + s1 * q1.x, s0 * q0.y + s1 * q1.y, s0 * q0.z + s1 * q1.z};
    const float rn = 1.0f / sqrtf(r.w * r.w + r.x * r.x + r.y * r.y + r.z * r.z);
    q = {r.w * rn, r.x * rn, r.y * rn, r.z * rn};
    if (VEL) {
        const float k = (n < 1e-12f) ? 0.0f : 2.0f * theta * fps / n;
        wl = {k * c.x, k * c.y, k * c.z};
    }
}

// Reference pose of body j's own joint at `time` into shared memory; warp 0
// also publishes the root position (lerp) and, if asked, the root velocity.
template <bool VEL, int NC>
__device__ __forceinline__ void stage_joint(const EnvKernelParams &P, const ClipMeta &cm, float time, int j,
                                            int lane, float *dst, float *rootp, float *rootv,
                                            Quat &ql, Vec3 &wl)
{
    int row;
    float alpha;
    lookup(cm, time, row, alpha);
    const int RS = P.sk.J + 1;
    const float4 *r0 = P.frames + (size_t)row * RS;
    const float4 *r1 = r0 + RS;
    slerp_joint<VEL>(ld_quat(r0 + 1 + j), ld_quat(r1 + 1 + j), alpha, cm.fps, ql, wl);
    float *o = dst + (j * NC) * kTile + lane;
    o[0 * kTile] = ql.w; o[1 * kTile] = ql.x; o[2 * kTile] = ql.y; o[3 * kTile] = ql.z;
    if (VEL) { o[4 * kTile] = wl.x; o[5 * kTile] = wl.y; o[6 * kTile] = wl.z; }
    if (j == 0) {
        const float4 a = __ldg(r0), b = __ldg(r1);
        rootp[0 * kTile + lane] = a.x + alpha * (b.x - a.x);
        rootp[1 * kTile + lane] = a.y + alpha * (b.y - a.y);
        rootp[2 * kTile + lane] = a.z + alpha * (b.z - a.z);
        if (VEL) {
            rootv[0 * kTile + lane] = (b.x - a.x) * cm.fps;
            rootv[1 * kTile + lane] = (b.y - a.y) * cm.fps;
            rootv[2 * kTile + lane] = (b.z - a.z) * cm.fps;
        }
    }
}

// Forward kinematics of body j by walking its ancestor chain root -> j
// (step a2), with velocity propagation when VEL.
template <bool VEL, int NC>
__device__ __forceinline__ void fk_walk(const SkelDev &sk, int j, int lane, const float *src,
                                        const float *rootp, const float *rootv,
                                        Quat &q, Vec3 &p, Vec3 &v, Vec3 &w)
{
    const float *r = src + lane;
    q = {r[0 * kTile], r[1 * kTile], r[2 * kTile], r[3 * kTile]};
    p = {rootp[0 * kTile + lane], rootp[1 * kTile + lane], rootp[2 * kTile + lane]};
    if (VEL) {
        v = {rootv[0 * kTile + lane], rootv[1 * kTile + lane], rootv[2 * kTile + lane]};
        w = qrot(q, Vec3{r[4 * kTile], r[5 * kTile], r[6 * kTile]});
    }
    const int depth = sk.depth[j];
    for (int d = 1; d <= depth; ++d) {
        const int b = sk.chain[j][d];
        const Vec3 arm = qrot(q, Vec3{sk.off[b][0], sk.off[b][1], sk.off[b][2]});
        if (VEL) v = v + cross(w, arm);
        p = p + arm;
        const float *c = src + (b * NC) * kTile + lane;
        q = qmul(q, Quat{c[0 * kTile], c[1 * kTile], c[2 * kTile], c[3 * kTile]});
        if (VEL) w = w + qrot(q, Vec3{c[4 * kTile], c[5 * kTile], c[6 * kTile]});
    }
}

template <bool RESET_ALL>
__global__ void __launch_bounds__(1024, 1) env_step_kernel(const __grid_constant__ EnvKernelParams P)
{
    extern __shared__ __align__(16) float smem_raw[];
    const SkelDev &sk = P.sk;
    const int J = sk.J;
    const int D = 24 * J + 1;
    const int lane = threadIdx.x & 31;
    const int j = threadIdx.x >> 5;
    const int env = blockIdx.x * kTile + lane;
    const bool valid = env < P.N;
    const int envc = valid ? env : P.N - 1;
    const Smem S = carve(smem_raw, J);

    int clip = 0;
    float t1 = 0.0f;
    ClipMeta cm = {2, 1.0f, 1.0f, 0};
    Quat ql_ref = {1, 0, 0, 0}, q_sim = {1, 0, 0, 0};
    Vec3 wl_ref = {0, 0, 0}, p_sim = {0, 0, 0}, v_sim = {0, 0, 0}, w_sim = {0, 0, 0};

    // ---- phase 1: advance time, stage the reference joint, load the simulated body
    if (!RESET_ALL) {
        clip = P.clip_id[envc];
        if (clip < 0 || clip >= P.C) {
            clip = min(max(clip, 0), P.C - 1);
            if (j == 0) atomicOr(P.status, IM_DEV_BAD_STATE);
        }
        t1 = __fadd_rn(P.t[envc], P.dt);
        cm = P.meta[clip];
        stage_joint<true, kRefComps>(P, cm, t1, j, lane, S.ref, S.rootp, S.rootv, ql_ref, wl_ref);

        const size_t st = (size_t)P.stride;
        p_sim = {P.pos[(3 * j + 0) * st + envc], P.pos[(3 * j + 1) * st + envc], P.pos[(3 * j + 2) * st + envc]};
        q_sim = {P.quat[(4 * j + 0) * st + envc], P.quat[(4 * j + 1) * st + envc],
                 P.quat[(4 * j + 2) * st + envc], P.quat[(4 * j + 3) * st + envc]};
        v_sim = {P.lin[(3 * j + 0) * st + envc], P.lin[(3 * j + 1) * st + envc], P.lin[(3 * j + 2) * st + envc]};
        w_sim = {P.ang[(3 * j + 0) * st + envc], P.ang[(3 * j + 1) * st + envc], P.ang[(3 * j + 2) * st + envc]};
        const float n2 = q_sim.w * q_sim.w + q_sim.x * q_sim.x + q_sim.y * q_sim.y + q_sim.z * q_sim.z;
        if (!(n2 > 1e-12f && n2 < 1e12f)) {
            q_sim = {1, 0, 0, 0};
            atomicOr(P.status, IM_DEV_BAD_SIM_QUAT);
        }
        float *o = S.simx + (j * kSimComps) * kTile + lane;
        o[0 * kTile] = q_sim.w; o[1 * kTile] = q_sim.x; o[2 * kTile] = q_sim.y; o[3 * kTile] = q_sim.z;
        o[4 * kTile] = w_sim.x; o[5 * kTile] = w_sim.y; o[6 * kTile] = w_sim.z;
    }
    __syncthreads();

    // ---- phase 2: reference FK, simulated joint-local quantities, per-body error partials
    if (!RESET_ALL) {
        Quat q_ref;
        Vec3 p_ref, v_ref, w_ref;
        fk_walk<true, kRefComps>(sk, j, lane, S.ref, S.rootp, S.rootv, q_ref, p_ref, v_ref, w_ref);

        Quat ql_sim = q_sim;
        Vec3 dw = w_sim;
        const int a = sk.parent[j];
        if (a >= 0) {
            const float *c = S.simx + (a * kSimComps) * kTile + lane;
            const Quat qa = {c[0 * kTile], c[1 * kTile], c[2 * kTile], c[3 * kTile]};
            ql_sim = qmul(qconj(qa), q_sim);
            dw = w_sim - Vec3{c[4 * kTile], c[5 * kTile], c[6 * kTile]};
        }
        const Vec3 wl_sim = qrot_inv(q_sim, dw);
        const float th = rel_angle(ql_ref, ql_sim);
        const Vec3 dwl = wl_sim - wl_ref;
        const Vec3 dp = p_sim - p_ref;
        const Vec3 dv = v_sim - v_ref;
        const float dp2 = dot(dp, dp);
        const bool is_ee = (sk.ee_mask >> j) & 1u;
        float ee_rot = 0.0f;
        if (is_ee) { const float th2 = rel_angle(q_ref, q_sim); ee_rot = th2 * th2; }
        const float mf = sk.mass_frac[j];
        float *o = S.part + j * kTile + lane;
        const int ps = J * kTile;
        o[0 * ps] = th * th;
        o[1 * ps] = dot(dwl, dwl);
        o[2 * ps] = is_ee ? dp2 : 0.0f;
        o[3 * ps] = ee_rot;
        o[4 * ps] = dp2;
        o[5 * ps] = dot(dv, dv);
        o[6 * ps] = mf * dp.x;
        o[7 * ps] = mf * dp.y;
        o[8 * ps] = mf * dp.z;
    }
    __syncthreads();

    // ---- phase 3 (warp 0): reduce over bodies, reward, flags, masked reset draw, state update
    if (j == 0) {
        int flags = 0;
        float t_cur = t1;
        int clip_cur = clip;
        if (!RESET_ALL) {
            float e[kPartials];
            const int ps = J * kTile;
#pragma unroll
            for (int k = 0; k < kPartials; ++k) {
                float acc = 0.0f;
                for (int b = 0; b < J; ++b) acc += S.part[k * ps + b * kTile + lane];
                e[k] = acc;
            }
            // term order of the configuration: pose, vel, ee_pos, ee_rot, com, body_pos, body_vel
            const float term[IM_N_TERMS] = {e[0], e[1], e[2], e[3], e[6] * e[6] + e[7] * e[7] + e[8] * e[8], e[4], e[5]};
            float r;
            if (P.reward.mode == 0) {
                float s = 0.0f;
#pragma unroll
                for (int k = 0; k < IM_N_TERMS; ++k) s += P.reward.w[k] * term[k];
                r = expf(-s);
            } else {
                r = 0.0f;
#pragma unroll
                for (int k = 0; k < IM_N_TERMS; ++k) r += P.reward.a[k] * expf(-P.reward.w[k] * term[k]);
            }
            const bool terminated = (p_sim.z < P.reward.h_min) || (r < P.reward.r_min);
            const bool truncated = __fadd_rn(t1, P.dt) > cm.dur;
            flags = (terminated ? 1 : 0) | (truncated ? 2 : 0);
            if (valid) {
                P.reward_out[env] = r;
                P.flags_out[env] = (uint8_t)flags;
                if (P.terms_out) {
#pragma unroll
                    for (int k = 0; k < IM_N_TERMS; ++k) P.terms_out[(size_t)k * P.N + env] = term[k];
                }
            }
        }
        const bool reset = RESET_ALL || flags != 0;
        if (reset) {
            const uint4 x = philox4x32_10(make_uint4(P.env_id_base + (uint32_t)envc, P.step, IM_STREAM_RESET, 0u),
                                          make_uint2(P.seed_lo, P.seed_hi));
            clip_cur = (int)__umulhi(x.x, (uint32_t)P.C);
            const float u = (float)(x.y >> 8) * 5.9604644775390625e-08f;
            const float span = fmaxf(__fsub_rn(P.meta[clip_cur].dur, P.dt), 0.0f);
            t_cur = __fmul_rn(u, span);
        }
        if (valid) {
            P.clip_id[env] = clip_cur;
            P.t[env] = t_cur;
            P.ep_len[env] = reset ? 0 : P.ep_len[env] + 1;
        }
        S.cur_clip[lane] = clip_cur;
        S.cur_t[lane] = t_cur;
        S.mask[lane] = reset ? 1 : 0;
        const unsigned any = __ballot_sync(0xffffffffu, reset);
        if (lane == 0) *S.any = any != 0u;
    }
    __syncthreads();

    // ---- phase 4: stage the target pose one control interval ahead and, if any env of the
    //      tile was reset, the reference state at the new phase
    const int clip_cur = S.cur_clip[lane];
    const float t_cur = S.cur_t[lane];
    const bool masked = S.mask[lane] != 0;
    const bool any_reset = *S.any != 0;
    const ClipMeta cmc = P.meta[clip_cur];
    {
        Quat qt;
        Vec3 unused;
        const float t_tgt = fminf(__fadd_rn(t_cur, P.dt), cmc.dur);
        stage_joint<false, kTgtComps>(P, cmc, t_tgt, j, lane, S.tgt, S.tgt_rootp, nullptr, qt, unused);
        if (any_reset) {
            stage_joint<true, kRefComps>(P, cmc, t_cur, j, lane, S.ref, S.rootp, S.rootv, ql_ref, wl_ref);
        }
    }
    __syncthreads();

    // ---- phase 5: target FK; state the observation is built from (simulated, or reference if reset)
    Quat q_tgt;
    Vec3 p_tgt, unused_v, unused_w;
    fk_walk<false, kTgtComps>(sk, j, lane, S.tgt, S.tgt_rootp, nullptr, q_tgt, p_tgt, unused_v, unused_w);
    Quat qx = q_sim;
    Vec3 px = p_sim, vx = v_sim, wx = w_sim;
    if (any_reset) {
        Quat qn;
        Vec3 pn, vn, wn;
        fk_walk<true, kRefComps>(sk, j, lane, S.ref, S.rootp, S.rootv, qn, pn, vn, wn);
        if (masked) { qx = qn; px = pn; vx = vn; wx = wn; }
    }
    if (j == 0) {
        const Vec3 h = qcol_x(qx);
        const float n2 = h.x * h.x + h.y * h.y;
        float hc = 1.0f, hs = 0.0f;
        if (n2 >= 1e-12f) { const float inv = 1.0f / sqrtf(n2); hc = h.x * inv; hs = h.y * inv; }
        S.head[0 * kTile + lane] = px.x;
        S.head[1 * kTile + lane] = px.y;
        S.head[2 * kTile + lane] = hc;
        S.head[3 * kTile + lane] = hs;
    }
    __syncthreads();

    // ---- phase 6: heading-local observation into the transposed tile
    {
        const float ox = S.head[0 * kTile + lane], oy = S.head[1 * kTile + lane];
        const float hc = S.head[2 * kTile + lane], hs = S.head[3 * kTile + lane];
        auto turn = [&](Vec3 a) -> Vec3 { return {hc * a.x + hs * a.y, hc * a.y - hs * a.x, a.z}; };
        float *row = S.tile + (size_t)lane * D;
        float *o = row + 15 * j;
        const Vec3 pl = turn(Vec3{px.x - ox, px.y - oy, px.z});
        const Vec3 tn = turn(qcol_x(qx)), nm = turn(qcol_z(qx));
        const Vec3 vl = turn(vx), wl = turn(wx);
        o[0] = pl.x; o[1] = pl.y; o[2] = pl.z;
        o[3] = tn.x; o[4] = tn.y; o[5] = tn.z;
        o[6] = nm.x; o[7] = nm.y; o[8] = nm.z;
        o[9] = vl.x; o[10] = vl.y; o[11] = vl.z;
        o[12] = wl.x; o[13] = wl.y; o[14] = wl.z;
        float *g = row + 15 * J + 1 + 9 * j;
        const Vec3 tp = turn(Vec3{p_tgt.x - ox, p_tgt.y - oy, p_tgt.z});
        const Vec3 tt = turn(qcol_x(q_tgt)), tm = turn(qcol_z(q_tgt));
        g[0] = tp.x; g[1] = tp.y; g[2] = tp.z;
        g[3] = tt.x; g[4] = tt.y; g[5] = tt.z;
        g[6] = tm.x; g[7] = tm.y; g[8] = tm.z;
        if (j == 0) row[15 * J] = t_cur / cmc.dur;

        if (!RESET_ALL && P.write_back && masked && valid) {
            const size_t st = (size_t)P.stride;
            P.pos[(3 * j + 0) * st + env] = px.x; P.pos[(3 * j + 1) * st + env] = px.y; P.pos[(3 * j + 2) * st + env] = px.z;
            P.quat[(4 * j + 0) * st + env] = qx.w; P.quat[(4 * j + 1) * st + env] = qx.x;
            P.quat[(4 * j + 2) * st + env] = qx.y; P.quat[(4 * j + 3) * st + env] = qx.z;
            P.lin[(3 * j + 0) * st + env] = vx.x; P.lin[(3 * j + 1) * st + env] = vx.y; P.lin[(3 * j + 2) * st + env] = vx.z;
            P.ang[(3 * j + 0) * st + env] = wx.x; P.ang[(3 * j + 1) * st + env] = wx.y; P.ang[(3 * j + 2) * st + env] = wx.z;
        }
    }
    __syncthreads();

    // ---- phase 7: rows of the tile to global memory, 128 contiguous bytes per warp store
    for (int r = j; r < kTile; r += J) {
        const int e = blockIdx.x * kTile + r;
        if (e >= P.N) break;
        float *dst = P.obs + (size_t)e * P.ld_obs;
        const float *src = S.tile + (size_t)r * D;
        for (int c = lane; c < P.ld_obs; c += 32) dst[c] = (c < D) ? src[c] : 0.0f;
    }
}

}  // namespace

size_t env_kernel_smem_bytes(int J) { return smem_floats(J) * sizeof(float); }

cudaError_t env_kernel_prepare(int J, size_t smem)
{
    (void)J;
    cudaError_t e = cudaFuncSetAttribute(env_step_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(env_step_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

cudaError_t launch_env_kernel(const EnvKernelParams &p, bool reset_all, size_t smem, cudaStream_t stream)
{
    const dim3 grid((p.N + kTile - 1) / kTile), block(32 * p.sk.J);
    if (reset_all) env_step_kernel<true><<<grid, block, smem, stream>>>(p);
    else env_step_kernel<false><<<grid, block, smem, stream>>>(p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace im
