// Fused environment step: reference lookup + slerp + forward kinematics,
// error terms and reward, flags, masked Philox reset, heading-local
// observation (the post-physics phase of the paper's Figure 2 as one kernel).
//
// Mapping: one CTA handles 32 consecutive envs; lane e handles env e of the
// tile and warp c handles kinematic chain c of the skeleton, a root-to-leaf
// path.  A thread walks its path once per pass, carrying the world transform
// (and velocities) in registers, so forward kinematics needs no exchange
// between threads; bodies shared by several paths are recomputed (pose only)
// and "owned" by one path, which alone loads their simulated state, scores them
// and writes their observation entries.  Every global load of the
// structure-of-arrays body state is one fully used 128-byte line per warp.
// The observation rows of the 32 envs are assembled in shared memory in two
// halves that reuse the same space (row stride 4 x odd: conflict-free 16-byte
// column writes, 16-byte aligned rows) and written out as whole lines.
#include <cuda_bf16.h>

#include "im_internal.h"
#include "im_device.cuh"

namespace im {

namespace {

// Four floats rounded to bf16 (nearest even), packed in column order.
__device__ __forceinline__ uint2 pack_bf16x4(float4 v)
{
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    return make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}

constexpr int kTile = 32;          // envs per CTA
constexpr int kPartials = 9;       // pose, vel, ee_pos, ee_rot, body_pos, body_vel, weighted com difference (3)

__host__ __device__ inline int tile_stride(int D)
{
    int s4 = (D + 3) / 4;
    if ((s4 & 1) == 0) ++s4;       // stride = 4 x odd floats
    return 4 * s4;
}

// The observation row is staged in two halves; the split is the end of the body blocks rounded
// up to a multiple of four columns so that both halves start on a 16-byte boundary.
__host__ __device__ inline int split_col(int J) { return (15 * J + 3) / 4 * 4; }

__host__ __device__ inline size_t smem_floats(int J, int n_chains, int extra_cols)
{
    const int D = 24 * J + 1 + extra_cols, c1 = split_col(J);
    const int s1 = tile_stride(c1), s2 = tile_stride(D - c1);
    return (size_t)kTile * (s1 > s2 ? s1 : s2) + (size_t)kPartials * n_chains * kTile;
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

// asin(y)^2 / y^2 as a series in u = y^2:  1/2 sum_n (4u)^n / (n^2 C(2n,n)) / u.
// Eight terms: relative truncation error below 1e-8 for u <= 0.15.
__device__ __forceinline__ float asin2_over_u(float u)
{
    float p = 0.03978244f;                 // n = 8
    p = fmaf(p, u, 0.04871319f);           // n = 7
    p = fmaf(p, u, 0.06156806f);           // n = 6
    p = fmaf(p, u, 0.08126984f);           // n = 5
    p = fmaf(p, u, 0.11428571f);           // n = 4
    p = fmaf(p, u, 0.17777778f);           // n = 3
    p = fmaf(p, u, 0.33333333f);           // n = 2
    return fmaf(p, u, 1.0f);               // n = 1
}

// sin(sqrt y) / sqrt y for small y (error below 1e-10 for y <= 0.07).
__device__ __forceinline__ float sinc_sqrt(float y)
{
    float p = -1.9841270e-4f;
    p = fmaf(p, y, 8.3333333e-3f);
    p = fmaf(p, y, -1.6666667e-1f);
    return fmaf(p, y, 1.0f);
}

// Shortest-arc slerp of one joint plus, if asked, the joint's angular velocity
// in the child frame, 2 log(q0* q1) fps.  The vector part of q0* q1 is formed
// from q1 - q0, which avoids the cancellation of the direct product when the
// keyframes are close and keeps the velocity accurate to ~1e-6 rad/s.
// Keyframes of a motion clip are close together, so the usual case (angle
// between the two quaternions below 0.25 rad) is evaluated without
// trigonometric calls: theta^2 from sin^2 theta by the arcsine series, and
// sin(a theta)/sin(theta) = a sinc(a theta)/sinc(theta) by short polynomials.
// Everything is normalised by |q0||q1|, so slightly non-unit keyframes give
// the same rotation as their normalised versions.
template <bool VEL>
__device__ __forceinline__ void slerp_joint(Quat q0, Quat q1, float alpha, float fps, Quat &q, Vec3 &wl)
{
    float d = q0.w * q1.w + q0.x * q1.x + q0.y * q1.y + q0.z * q1.z;
    if (d < 0.0f) { d = -d; q1 = {-q1.w, -q1.x, -q1.y, -q1.z}; }
    const Quat diff = {q1.w - q0.w, q1.x - q0.x, q1.y - q0.y, q1.z - q0.z};
    const Quat c = qmul(qconj(q0), diff);
    const float n2 = c.x * c.x + c.y * c.y + c.z * c.z;
    const float m2 = fmaf(d, d, n2);                       // (|q0||q1|)^2
    const float u = __fdividef(n2, m2);                    // sin^2 theta
    float s0, s1, vel_scale = 0.0f;
    if (u <= 0.0625f) {
        const float x = u * asin2_over_u(u);               // theta^2
        const float sc = sinc_sqrt(x);
        float inv = __fdividef(1.0f, sc);                  // theta / sin theta ...
        inv = inv * fmaf(-sc, inv, 2.0f);                  // ... refined to full precision (Newton step)
        const float a0 = 1.0f - alpha;
        s0 = a0 * sinc_sqrt(a0 * a0 * x) * inv;
        s1 = alpha * sinc_sqrt(alpha * alpha * x) * inv;
        if (VEL) {
            float rs = rsqrtf(m2);                         // 1 / (|q0||q1|), one Newton step as well:
            rs = rs * fmaf(-0.5f * m2, rs * rs, 1.5f);     // the velocity is summed down the chain
            vel_scale = 2.0f * fps * inv * rs;
        }
    } else {
        const float n = sqrtf(n2);
        const float theta = atan2f(n, d);
        const float inv = 1.0f / n;
        s0 = sinf((1.0f - alpha) * theta) * inv;
        s1 = sinf(alpha * theta) * inv;
        vel_scale = 2.0f * theta * fps * inv;
    }
    const Quat r = {s0 * q0.w + s1 * q1.w, s0 * q0.x + s1 * q1.x, s0 * q0.y + s1 * q1.y, s0 * q0.z + s1 * q1.z};
    const float rn = rsqrtf(r.w * r.w + r.x * r.x + r.y * r.y + r.z * r.z);
    q = {r.w * rn, r.x * rn, r.y * rn, r.z * rn};
    if (VEL) wl = {vel_scale * c.x, vel_scale * c.y, vel_scale * c.z};
}

// Squared rotation angle, in [0, pi^2], of the rotation taking frame a to frame b.  Small
// angles (below 0.8 rad, the usual tracking error) use the arcsine series on sin^2(theta/2).
__device__ __forceinline__ float rel_angle_sq(Quat a, Quat b)
{
    const Quat r = qmul(qconj(a), b);
    const float n2 = r.x * r.x + r.y * r.y + r.z * r.z;
    const float u = __fdividef(n2, fmaf(r.w, r.w, n2));    // sin^2(theta / 2)
    if (u <= 0.15f) return 4.0f * u * asin2_over_u(u);
    const float th = 2.0f * atan2f(sqrtf(n2), fabsf(r.w));
    return th * th;
}

// World transform (and velocities) carried down a kinematic chain (step a2).
struct Walk {
    Quat q;
    Vec3 p, v, w;
};

// One link of the chain: interpolate joint b between keyframe rows r0/r1 and
// compose it onto the running transform.  k == 0 is the root.
template <bool VEL>
__device__ __forceinline__ void joint_compose(const SkelDev &sk, const float4 *r0, const float4 *r1, float alpha,
                                              float fps, int b, int k, Walk &s, Quat ql, Vec3 wl)
{
    if (k == 0) {
        const float4 a = __ldg(r0), c = __ldg(r1);
        s.q = ql;
        s.p = {a.x + alpha * (c.x - a.x), a.y + alpha * (c.y - a.y), a.z + alpha * (c.z - a.z)};
        if (VEL) {
            s.v = {(c.x - a.x) * fps, (c.y - a.y) * fps, (c.z - a.z) * fps};
            s.w = qrot(ql, wl);
        }
    } else {
        const Vec3 arm = qrot(s.q, Vec3{sk.off[b][0], sk.off[b][1], sk.off[b][2]});
        if (VEL) s.v = s.v + cross(s.w, arm);
        s.p = s.p + arm;
        s.q = qmul(s.q, ql);
        if (VEL) s.w = s.w + qrot(s.q, wl);
    }
}

template <bool VEL>
__device__ __forceinline__ void joint_step(const SkelDev &sk, const float4 *r0, const float4 *r1, Quat k0, Quat k1,
                                           float alpha, float fps, int b, int k, Walk &s, Quat &ql, Vec3 &wl)
{
    slerp_joint<VEL>(k0, k1, alpha, fps, ql, wl);
    joint_compose<VEL>(sk, r0, r1, alpha, fps, b, k, s, ql, wl);
}

// Motion randomisation of a reset state: three standard normals of Philox counter
// (env id, step, 2, block), scaled by the configured standard deviation.
__device__ __forceinline__ Vec3 reset_noise_vec(const EnvKernelParams &P, int env, int block)
{
    const uint4 x = philox4x32_10(make_uint4(P.env_id_base + (uint32_t)env, P.step, IM_STREAM_RESET_NOISE, (uint32_t)block),
                                  make_uint2(P.seed_lo, P.seed_hi));
    float z0, z1, z2, z3;
    box_muller(x.x, x.y, z0, z1);
    box_muller(x.z, x.w, z2, z3);
    return {P.reset_noise_std * z0, P.reset_noise_std * z1, P.reset_noise_std * z2};
}
// ... as the rotation exp(n / 2) applied to joint `b` in its own frame (block b) ...
__device__ __forceinline__ Quat reset_noise_quat(const EnvKernelParams &P, int env, int b)
{
    const Vec3 n = reset_noise_vec(P, env, b);
    const float th = sqrtf(dot(n, n));
    float sn, cs;
    sincosf(0.5f * th, &sn, &cs);
    const float k = th > 1e-12f ? sn / th : 0.5f;
    return {cs, k * n.x, k * n.y, k * n.z};
}
// ... and as the shift of the root position (block J).
__device__ __forceinline__ Vec3 reset_noise_shift(const EnvKernelParams &P, int env, int J)
{
    return reset_noise_vec(P, env, J);
}

// Phase bin of time t in a clip whose start times span [0, span]: floor(t / (span / B)) in single
// fp32 operations, clamped to B - 1.
__device__ __forceinline__ int phase_bin(float t, float span, int B)
{
    const float width = __fdiv_rn(span, (float)B);
    if (!(width > 0.0f)) return 0;
    const int b = (int)floorf(__fdiv_rn(t, width));
    return min(max(b, 0), B - 1);
}

// Heading frame of the character the observation is taken from: origin at the
// root's (x, y, 0), yaw of the root's rotated x axis (step a6).
struct Heading {
    float ox, oy, c, s;
    __device__ __forceinline__ Vec3 turn(Vec3 a) const { return {c * a.x + s * a.y, c * a.y - s * a.x, a.z}; }
};

__device__ __forceinline__ Heading make_heading(Quat q_root, Vec3 p_root)
{
    const Vec3 h = qcol_x(q_root);
    const float n2 = h.x * h.x + h.y * h.y;
    Heading H = {p_root.x, p_root.y, 1.0f, 0.0f};
    if (n2 >= 1e-12f) { const float inv = rsqrtf(n2); H.c = h.x * inv; H.s = h.y * inv; }
    return H;
}

// Stores N consecutive floats at dst, whose offset from a 16-byte boundary is OFF floats,
// using 16-byte stores for the aligned middle.
template <int N, int OFF>
__device__ __forceinline__ void store_run_at(float *dst, const float (&v)[N])
{
    constexpr int head = (4 - OFF) & 3;
    constexpr int mid = (N - head) / 4;
#pragma unroll
    for (int i = 0; i < head; ++i) dst[i] = v[i];
#pragma unroll
    for (int m = 0; m < mid; ++m)
        *reinterpret_cast<float4 *>(dst + head + 4 * m) =
            make_float4(v[head + 4 * m], v[head + 4 * m + 1], v[head + 4 * m + 2], v[head + 4 * m + 3]);
#pragma unroll
    for (int i = head + 4 * mid; i < N; ++i) dst[i] = v[i];
}

template <int N>
__device__ __forceinline__ void store_run(float *row, int col, const float (&v)[N])
{
    float *dst = row + col;
    switch (col & 3) {          // uniform across the warp
    case 0: store_run_at<N, 0>(dst, v); break;
    case 1: store_run_at<N, 1>(dst, v); break;
    case 2: store_run_at<N, 2>(dst, v); break;
    default: store_run_at<N, 3>(dst, v); break;
    }
}

// The 15 observation floats of one body seen from the heading frame.
__device__ __forceinline__ void body_obs(const Heading &H, Quat q, Vec3 p, Vec3 v, Vec3 w, float *row, int b)
{
    const Vec3 pl = H.turn(Vec3{p.x - H.ox, p.y - H.oy, p.z});
    const Vec3 tn = H.turn(qcol_x(q)), nm = H.turn(qcol_z(q));
    const Vec3 vl = H.turn(v), wl = H.turn(w);
    const float o[15] = {pl.x, pl.y, pl.z, tn.x, tn.y, tn.z, nm.x, nm.y, nm.z, vl.x, vl.y, vl.z, wl.x, wl.y, wl.z};
    store_run<15>(row, 15 * b, o);
}

struct SimBody {
    Quat q;
    Vec3 p, v, w;
};

__device__ __forceinline__ Quat sanitize(Quat q, uint32_t *status)
{
    const float n2 = q.w * q.w + q.x * q.x + q.y * q.y + q.z * q.z;
    if (!(n2 > 1e-12f && n2 < 1e12f)) {
        atomicOr(status, IM_DEV_BAD_SIM_QUAT);
        return {1, 0, 0, 0};
    }
    return q;
}

// Body-state loads: `col` points at this thread's env in row 0 of the array, so a component is
// one per-thread pointer plus a warp-uniform row offset.
__device__ __forceinline__ Quat ld_sim_quat(const float *col, size_t st, int b)
{
    const float *p = col + (size_t)(4 * b) * st;
    return {p[0], p[st], p[2 * st], p[3 * st]};
}
__device__ __forceinline__ Vec3 ld_sim_vec(const float *col, size_t st, int b)
{
    const float *p = col + (size_t)(3 * b) * st;
    return {p[0], p[st], p[2 * st]};
}

// Keyframe quaternions of joint b in the two bracketing rows.
struct KeyPair {
    float4 a, b;
};
__device__ __forceinline__ KeyPair ld_keys(const float4 *r0, const float4 *r1, int b)
{
    return {__ldg(r0 + 1 + b), __ldg(r1 + 1 + b)};
}
__device__ __forceinline__ Quat as_quat(float4 v) { return {v.x, v.y, v.z, v.w}; }

// Kernel body.  The observation row is assembled in two halves that reuse the same shared
// memory: columns [0, c1) -- the body blocks and, if 15 J is not a multiple of 4, the phase and
// the first target floats -- and columns [c1, D) -- the targets.
// OPT compiles in the optional semantics (grace steps, motion randomisation, adaptive initialisation); envs that use none run
// the instantiation without them.
template <bool RESET_ALL, bool OPT>
__device__ __forceinline__ void env_step_body(const EnvKernelParams &P, float *smem_raw)
{
    // a successor launched with programmatic stream serialization (the policy's first GEMM) may be scheduled
    // onto SMs as this grid drains; it waits for this grid's completion before it reads anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const SkelDev &sk = P.sk;
    const int J = sk.J;
    const int D = 24 * J + 1;
    const int c1 = split_col(J);                    // multiple of 4
    // extended observation: end-effector targets of further future frames, then the previous action
    const int n_ee = OPT ? __popc(sk.ee_mask) : 0;
    const int ext_future = (OPT && P.n_future > 1) ? (P.n_future - 1) * 9 * n_ee : 0;
    const int D_ext = D + ext_future + (OPT ? P.act_dim : 0);
    const int S1 = tile_stride(c1), S2 = tile_stride(D_ext - c1);
    const int C = sk.n_chains;
    const int lane = threadIdx.x & 31;
    const int c = threadIdx.x >> 5;                 // this thread's chain
    const int env = blockIdx.x * kTile + lane;
    const bool valid = env < P.N;
    const int envc = valid ? env : P.N - 1;
    float *tile = smem_raw;
    float *part = smem_raw + (size_t)kTile * (S1 > S2 ? S1 : S2);
    float *row1 = tile + (size_t)lane * S1;
    float *row2 = tile + (size_t)lane * S2;
    const int len = sk.chain_len[c];
    const int first_own = sk.chain_first_own[c];
    const int RS = J + 1;

    if (c == 0)
        for (int i = 15 * J; i < S1; ++i) row1[i] = 0.0f;   // columns between the body blocks and the stride

    int clip = 0;
    float t1 = 0.0f;
    ClipMeta cm = {2, 1.0f, 1.0f, 0};
    Heading H = {0.0f, 0.0f, 1.0f, 0.0f};
    float root_z = 0.0f;

    // ---- pass A: reference at the advanced time, errors against the simulated state,
    //      observation entries of the simulated bodies
    if (!RESET_ALL) {
        clip = P.clip_id[envc];
        if (clip < 0 || clip >= P.C) {
            clip = min(max(clip, 0), P.C - 1);
            if (c == 0) atomicOr(P.status, IM_DEV_BAD_STATE);
        }
        t1 = __fadd_rn(P.t[envc], P.dt);
        cm = P.meta[clip];
        int frame;
        float alpha;
        lookup(cm, t1, frame, alpha);
        const float4 *r0 = P.frames + (size_t)frame * RS, *r1 = r0 + RS;
        KeyPair keys = ld_keys(r0, r1, sk.chain[c][0]);

        const size_t st = (size_t)P.stride;
        const float *pos_e = P.pos + envc, *quat_e = P.quat + envc, *lin_e = P.lin + envc, *ang_e = P.ang + envc;
        const Quat q_root = sanitize(ld_sim_quat(quat_e, st, 0), P.status);
        const Vec3 p_root = ld_sim_vec(pos_e, st, 0);
        H = make_heading(q_root, p_root);
        root_z = p_root.z;

        float acc[kPartials];
#pragma unroll
        for (int i = 0; i < kPartials; ++i) acc[i] = 0.0f;
        Walk s;
        Quat qa = {1, 0, 0, 0};                      // simulated state of the previous body of the chain
        Vec3 wa = {0, 0, 0};
        if (first_own > 0) {
            const int a = sk.chain[c][first_own - 1];
            qa = sanitize(ld_sim_quat(quat_e, st, a), P.status);
            wa = ld_sim_vec(ang_e, st, a);
        }
        for (int k = 0; k < len; ++k) {
            const int b = sk.chain[c][k];
            const bool own = k >= first_own;
            SimBody sim;
            if (own) {                                // issue the loads before the interpolation math
                sim.q = ld_sim_quat(quat_e, st, b);
                sim.p = ld_sim_vec(pos_e, st, b);
                sim.v = ld_sim_vec(lin_e, st, b);
                sim.w = ld_sim_vec(ang_e, st, b);
            }
            const KeyPair cur = keys;
            if (k + 1 < len) keys = ld_keys(r0, r1, sk.chain[c][k + 1]);     // next joint's keyframes in flight
            Quat ql;
            Vec3 wl;
            joint_step<true>(sk, r0, r1, as_quat(cur.a), as_quat(cur.b), alpha, cm.fps, b, k, s, ql, wl);
            if (own) {
                sim.q = sanitize(sim.q, P.status);
                Quat ql_sim = sim.q;
                Vec3 dw = sim.w;
                if (b > 0) {
                    ql_sim = qmul(qconj(qa), sim.q);
                    dw = sim.w - wa;
                }
                const Vec3 wl_sim = qrot_inv(sim.q, dw);
                const float th_sq = rel_angle_sq(ql, ql_sim);
                const Vec3 dwl = wl_sim - wl;
                const Vec3 dp = sim.p - s.p;
                const Vec3 dv = sim.v - s.v;
                const float dp2 = dot(dp, dp);
                acc[0] += th_sq;
                acc[1] += dot(dwl, dwl);
                if ((sk.ee_mask >> b) & 1u) {
                    acc[2] += dp2;
                    acc[3] += rel_angle_sq(s.q, sim.q);
                }
                acc[4] += dp2;
                acc[5] += dot(dv, dv);
                const float mf = sk.mass_frac[b];
                acc[6] += mf * dp.x;
                acc[7] += mf * dp.y;
                acc[8] += mf * dp.z;
                body_obs(H, sim.q, sim.p, sim.v, sim.w, row1, b);
                qa = sim.q;
                wa = sim.w;
            }
        }
#pragma unroll
        for (int i = 0; i < kPartials; ++i) part[(i * C + c) * kTile + lane] = acc[i];
    }
    __syncthreads();

    // ---- decision: every thread of an env adds the chains' partial sums in chain order and takes
    //      the same reward, flags and reset draw; chain 0 writes them out
    int flags = 0;
    float t_cur = t1;
    int clip_cur = clip;
    if (!RESET_ALL) {
        float e[kPartials];
#pragma unroll
        for (int i = 0; i < kPartials; ++i) {
            float a = 0.0f;
            for (int cc = 0; cc < C; ++cc) a += part[(i * C + cc) * kTile + lane];
            e[i] = a;
        }
        // term order of the configuration: pose, vel, ee_pos, ee_rot, com, body_pos, body_vel
        const float term[IM_N_TERMS] = {e[0], e[1], e[2], e[3], e[6] * e[6] + e[7] * e[7] + e[8] * e[8], e[4], e[5]};
        float r;
        if (P.reward.mode == 0) {
            float sum = 0.0f;
#pragma unroll
            for (int k = 0; k < IM_N_TERMS; ++k) sum += P.reward.w[k] * term[k];
            r = expf(-sum);
        } else {
            r = 0.0f;
#pragma unroll
            for (int k = 0; k < IM_N_TERMS; ++k) r += P.reward.a[k] * expf(-P.reward.w[k] * term[k]);
        }
        bool terminated = (root_z < P.reward.h_min) || (r < P.reward.r_min);
        if (OPT && P.ep_len[envc] < P.grace_steps) terminated = false;
        if (OPT && P.n_bins > 0 && terminated && c == 0 && valid) {
            // adaptive initialisation statistics: the (clip, phase bin) the episode failed in
            const float span = fmaxf(__fsub_rn(cm.dur, P.dt), 0.0f);
            atomicAdd(P.stat_failures + clip * P.n_bins + phase_bin(t1, span, P.n_bins), 1u);
        }
        const bool truncated = __fadd_rn(t1, P.dt) > cm.dur;
        flags = (terminated ? 1 : 0) | (truncated ? 2 : 0);
        if (c == 0 && valid) {
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
        const float u = (float)(x.y >> 8) * 5.9604644775390625e-08f;
        if (OPT && P.n_bins > 0) {
            // weighted (clip, phase bin) from the cumulative table: smallest i with x < T_i
            const int B = P.n_bins;
            int lo = 0, hi = P.C * B - 1;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if ((unsigned long long)x.x < __ldg(P.reset_cdf + mid)) hi = mid;
                else lo = mid + 1;
            }
            clip_cur = lo / B;
            const float span = fmaxf(__fsub_rn(P.meta[clip_cur].dur, P.dt), 0.0f);
            const float width = __fdiv_rn(span, (float)B);
            t_cur = fminf(__fmul_rn(__fadd_rn((float)(lo - clip_cur * B), u), width), span);
            if (c == 0 && valid) atomicAdd(P.stat_starts + lo, 1u);
        } else {
            clip_cur = (int)__umulhi(x.x, (uint32_t)P.C);
            const float span = fmaxf(__fsub_rn(P.meta[clip_cur].dur, P.dt), 0.0f);
            t_cur = __fmul_rn(u, span);
        }
    }
    if (c == 0 && valid) {
        P.clip_id[env] = clip_cur;
        P.t[env] = t_cur;
        P.ep_len[env] = reset ? 0 : P.ep_len[env] + 1;
    }
    const ClipMeta cmc = reset ? P.meta[clip_cur] : cm;

    // ---- pass C (only where an env of this warp was reset): reference state at the new phase
    //      replaces the simulated one in the observation, and optionally in the caller's arrays
    if (__any_sync(0xffffffffu, reset)) {
        int frame;
        float alpha;
        lookup(cmc, t_cur, frame, alpha);
        const float4 *r0 = P.frames + (size_t)frame * RS, *r1 = r0 + RS;
        KeyPair keys = ld_keys(r0, r1, sk.chain[c][0]);
        Walk s;
        Heading Hn = H;
        for (int k = 0; k < len; ++k) {
            const int b = sk.chain[c][k];
            const KeyPair cur = keys;
            if (k + 1 < len) keys = ld_keys(r0, r1, sk.chain[c][k + 1]);
            Quat ql;
            Vec3 wl;
            if (OPT && P.reset_noise_std > 0.0f) {
                // motion randomisation: the joint turns by a small random rotation in its own frame and
                // the root is shifted; every chain that walks a shared body draws the same numbers
                slerp_joint<true>(as_quat(cur.a), as_quat(cur.b), alpha, cmc.fps, ql, wl);
                ql = qmul(ql, reset_noise_quat(P, envc, b));
                joint_compose<true>(sk, r0, r1, alpha, cmc.fps, b, k, s, ql, wl);
                if (k == 0) s.p = s.p + reset_noise_shift(P, envc, sk.J);
            } else {
                joint_step<true>(sk, r0, r1, as_quat(cur.a), as_quat(cur.b), alpha, cmc.fps, b, k, s, ql, wl);
            }
            if (k == 0) Hn = make_heading(s.q, s.p);
            if (k >= first_own && reset) {
                body_obs(Hn, s.q, s.p, s.v, s.w, row1, b);
                if (!RESET_ALL && P.write_back && valid) {
                    const size_t st = (size_t)P.stride;
                    P.pos[(3 * b + 0) * st + env] = s.p.x; P.pos[(3 * b + 1) * st + env] = s.p.y; P.pos[(3 * b + 2) * st + env] = s.p.z;
                    P.quat[(4 * b + 0) * st + env] = s.q.w; P.quat[(4 * b + 1) * st + env] = s.q.x;
                    P.quat[(4 * b + 2) * st + env] = s.q.y; P.quat[(4 * b + 3) * st + env] = s.q.z;
                    P.lin[(3 * b + 0) * st + env] = s.v.x; P.lin[(3 * b + 1) * st + env] = s.v.y; P.lin[(3 * b + 2) * st + env] = s.v.z;
                    P.ang[(3 * b + 0) * st + env] = s.w.x; P.ang[(3 * b + 1) * st + env] = s.w.y; P.ang[(3 * b + 2) * st + env] = s.w.z;
                }
            }
        }
        if (reset) H = Hn;
    }

    // ---- the first half also holds the phase and the first floats of the root's target when 15 J
    //      is not a multiple of 4: chain 0 interpolates the root one interval ahead for them
    const float t_tgt = fminf(__fadd_rn(t_cur, P.dt), cmc.dur);
    int frame_t;
    float alpha_t;
    lookup(cmc, t_tgt, frame_t, alpha_t);
    const float4 *rt0 = P.frames + (size_t)frame_t * RS, *rt1 = rt0 + RS;
    const float phase = t_cur / cmc.dur;
    if (c == 0 && 15 * J < c1) {
        Walk s;
        Quat ql;
        Vec3 wl;
        const KeyPair kp = ld_keys(rt0, rt1, 0);
        joint_step<false>(sk, rt0, rt1, as_quat(kp.a), as_quat(kp.b), alpha_t, cmc.fps, 0, 0, s, ql, wl);
        const Vec3 tp = H.turn(Vec3{s.p.x - H.ox, s.p.y - H.oy, s.p.z});
        row1[15 * J] = phase;
        if (15 * J + 1 < c1) row1[15 * J + 1] = tp.x;
        if (15 * J + 2 < c1) row1[15 * J + 2] = tp.y;
    }
    __syncthreads();

    // ---- first half of the rows to global memory, 16-byte stores, 512 contiguous bytes per warp store
    {
        const int n4 = c1 >> 2, S4 = S1 >> 2;
        const float4 *tile4 = reinterpret_cast<const float4 *>(tile);
        for (int r = c; r < kTile; r += C) {
            const int e = blockIdx.x * kTile + r;
            if (e >= P.N) break;
            // (a policy-serving loop may ask for the bf16 rows only: obs null)
            float4 *dst = P.obs ? reinterpret_cast<float4 *>(P.obs + (size_t)e * P.ld_obs) : nullptr;
            uint2 *dst16 = P.obs_bf16 ? reinterpret_cast<uint2 *>(P.obs_bf16 + (size_t)e * P.ld_obs) : nullptr;
            for (int i = lane; i < n4; i += 32) {
                const float4 v = tile4[(size_t)r * S4 + i];
                if (dst) dst[i] = v;
                if (dst16) dst16[i] = pack_bf16x4(v);
            }
        }
    }
    __syncthreads();

    // ---- pass B: reference pose one control interval ahead, seen from the same heading frame,
    //      into the second half (which reuses the shared memory of the first)
    {
        if (c == 0) {
            for (int i = D_ext - c1; i < S2; ++i) row2[i] = 0.0f;
            if (15 * J >= c1) row2[15 * J - c1] = phase;
        }
        KeyPair keys = ld_keys(rt0, rt1, sk.chain[c][0]);
        Walk s;
        for (int k = 0; k < len; ++k) {
            const int b = sk.chain[c][k];
            const KeyPair cur = keys;
            if (k + 1 < len) keys = ld_keys(rt0, rt1, sk.chain[c][k + 1]);
            Quat ql;
            Vec3 wl;
            joint_step<false>(sk, rt0, rt1, as_quat(cur.a), as_quat(cur.b), alpha_t, cmc.fps, b, k, s, ql, wl);
            if (k >= first_own) {
                const Vec3 tp = H.turn(Vec3{s.p.x - H.ox, s.p.y - H.oy, s.p.z});
                const Vec3 tt = H.turn(qcol_x(s.q)), tm = H.turn(qcol_z(s.q));
                const float o[9] = {tp.x, tp.y, tp.z, tt.x, tt.y, tt.z, tm.x, tm.y, tm.z};
                const int col = 15 * J + 1 + 9 * b;
                if (col >= c1) {
                    store_run<9>(row2, col - c1, o);
                } else {                          // the root's block straddles the split
#pragma unroll
                    for (int i = 0; i < 9; ++i)
                        if (col + i >= c1) row2[col + i - c1] = o[i];
                }
            }
        }
        if (OPT && D_ext > D) {
            // frames f = 2 .. n_future of the reference, t + f dt (two fp32 operations, clamped to the clip's end):
            // every chain walks them again and the owner of an end effector writes its nine entries
            for (int f = 2; f <= P.n_future; ++f) {
                const float t_f = fminf(__fadd_rn(t_cur, __fmul_rn((float)f, P.dt)), cmc.dur);
                int frame_f;
                float alpha_f;
                lookup(cmc, t_f, frame_f, alpha_f);
                const float4 *rf0 = P.frames + (size_t)frame_f * RS, *rf1 = rf0 + RS;
                Walk sf;
                for (int k = 0; k < len; ++k) {
                    const int b = sk.chain[c][k];
                    const KeyPair kp = ld_keys(rf0, rf1, b);
                    Quat ql;
                    Vec3 wl;
                    joint_step<false>(sk, rf0, rf1, as_quat(kp.a), as_quat(kp.b), alpha_f, cmc.fps, b, k, sf, ql, wl);
                    if (k >= first_own && ((sk.ee_mask >> b) & 1u)) {
                        const Vec3 tp = H.turn(Vec3{sf.p.x - H.ox, sf.p.y - H.oy, sf.p.z});
                        const Vec3 tt = H.turn(qcol_x(sf.q)), tm = H.turn(qcol_z(sf.q));
                        const float o[9] = {tp.x, tp.y, tp.z, tt.x, tt.y, tt.z, tm.x, tm.y, tm.z};
                        float *dst = row2 + (D - c1) + ((f - 2) * n_ee + __popc(sk.ee_mask & ((1u << b) - 1u))) * 9;
#pragma unroll
                        for (int i = 0; i < 9; ++i) dst[i] = o[i];
                    }
                }
            }
            // the action the policy took before this step; an env that was just reset has none
            float *dst = row2 + (D - c1) + ext_future;
            for (int j = c; j < P.act_dim; j += C)
                dst[j] = (reset || !valid) ? 0.0f : __ldg(P.prev_action + (size_t)env * P.ld_action + j);
        }
    }
    __syncthreads();
    {
        const int n4 = c1 >> 2, S4 = S2 >> 2, ld4 = P.ld_obs >> 2;
        const float4 *tile4 = reinterpret_cast<const float4 *>(tile);
        for (int r = c; r < kTile; r += C) {
            const int e = blockIdx.x * kTile + r;
            if (e >= P.N) break;
            float4 *dst = P.obs ? reinterpret_cast<float4 *>(P.obs + (size_t)e * P.ld_obs) : nullptr;
            uint2 *dst16 = P.obs_bf16 ? reinterpret_cast<uint2 *>(P.obs_bf16 + (size_t)e * P.ld_obs) : nullptr;
            for (int i = n4 + lane; i < ld4; i += 32) {
                const float4 v = (i - n4 < S4) ? tile4[(size_t)r * S4 + i - n4] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                if (dst) dst[i] = v;
                if (dst16) dst16[i] = pack_bf16x4(v);
            }
        }
    }
}

// Two instantiations per mode: skeletons with at most 8 leaves (blocks of up to 256 threads) get a
// register budget that lets four blocks share an SM; wider trees fall back to 64 registers.
template <bool RESET_ALL, bool OPT>
__global__ void __maxnreg__(96) env_step_kernel_small(const __grid_constant__ EnvKernelParams P)
{
    extern __shared__ __align__(16) float smem_raw[];
    env_step_body<RESET_ALL, OPT>(P, smem_raw);
}

template <bool RESET_ALL, bool OPT>
__global__ void __launch_bounds__(1024, 1) env_step_kernel_wide(const __grid_constant__ EnvKernelParams P)
{
    extern __shared__ __align__(16) float smem_raw[];
    env_step_body<RESET_ALL, OPT>(P, smem_raw);
}

template <bool RESET_ALL, bool OPT>
cudaError_t prepare_one(size_t smem)
{
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(env_step_kernel_small<RESET_ALL, OPT>, attr, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(env_step_kernel_wide<RESET_ALL, OPT>, attr, (int)smem);
    return e;
}

template <bool RESET_ALL, bool OPT>
void launch_one(const EnvKernelParams &p, dim3 grid, dim3 block, size_t smem, cudaStream_t stream)
{
    if (block.x <= 256) env_step_kernel_small<RESET_ALL, OPT><<<grid, block, smem, stream>>>(p);
    else env_step_kernel_wide<RESET_ALL, OPT><<<grid, block, smem, stream>>>(p);
}

}  // namespace

size_t env_kernel_smem_bytes(int J, int n_chains, int extra_cols) { return smem_floats(J, n_chains, extra_cols) * sizeof(float); }

cudaError_t env_kernel_prepare(size_t smem)
{
    static bool done = false;
    if (done) return cudaSuccess;
    cudaError_t e = prepare_one<false, false>(smem);
    if (e == cudaSuccess) e = prepare_one<true, false>(smem);
    if (e == cudaSuccess) e = prepare_one<false, true>(smem);
    if (e == cudaSuccess) e = prepare_one<true, true>(smem);
    done = e == cudaSuccess;
    return e;
}

cudaError_t launch_env_kernel(const EnvKernelParams &p, bool reset_all, size_t smem, cudaStream_t stream)
{
    const dim3 grid((p.N + kTile - 1) / kTile), block(32 * p.sk.n_chains);
    const bool opt = p.grace_steps > 0 || p.reset_noise_std > 0.0f || p.n_bins > 0 || p.n_future > 1 || p.act_dim > 0;
    if (opt) {
        if (reset_all) launch_one<true, true>(p, grid, block, smem, stream);
        else launch_one<false, true>(p, grid, block, smem, stream);
    } else {
        if (reset_all) launch_one<true, false>(p, grid, block, smem, stream);
        else launch_one<false, false>(p, grid, block, smem, stream);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace im
