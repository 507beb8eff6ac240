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

// The bounds-checked build (-DIM_DEBUG, a second library next to the regular one): every index the kernel forms
// from its inputs -- keyframe row, body index of a link, body-state offset, staged observation column,
// destination row -- is tested against its limit; an index out of range sets IM_DEV_DEBUG_CHECK in the env's
// status word and is replaced by 0, so the launch always completes (no trap, no fault) and a test reads the word.
#ifdef IM_DEBUG
__device__ __forceinline__ uint32_t checked(uint32_t idx, uint32_t limit, uint32_t *status)
{
    if (idx < limit) return idx;
    atomicOr(status, IM_DEV_DEBUG_CHECK);
    return 0u;
}
#define IM_CHECKED(idx, limit) checked((uint32_t)(idx), (uint32_t)(limit), P.status)
#else
#define IM_CHECKED(idx, limit) (idx)
#endif

__host__ __device__ inline int tile_stride(int D)
{
    int s4 = (D + 3) / 4;
    if ((s4 & 1) == 0) ++s4;       // stride = 4 x odd floats
    return 4 * s4;
}

// The observation row is staged in two halves; the split is the end of the body blocks rounded
// up to a multiple of four columns so that both halves start on a 16-byte boundary.
__host__ __device__ inline int split_col(int J) { return (15 * J + 3) / 4 * 4; }

// Shared memory, in floats: the staged half rows, the chains' partial sums, the chains' link records.
__host__ __device__ inline size_t smem_floats(int J, int n_chains, int n_links, int extra_cols)
{
    const int D = 24 * J + 1 + extra_cols, c1 = split_col(J);
    const int s1 = tile_stride(c1), s2 = tile_stride(D - c1);
    return (size_t)kTile * (s1 > s2 ? s1 : s2) + (size_t)kPartials * n_chains * kTile + (size_t)8 * n_links;
}

// ---------------------------------------------------------------------------------------------
// Clip table.  Row r (one keyframe) holds 2 + 2 J 16-byte words:
//   [0]        root position (x, y, z, 0)
//   [1]        root displacement to the next keyframe (0 in a clip's last frame)
//   [2 + 2 j]  local rotation of joint j, normalised (w, x, y, z)
//   [3 + 2 j]  (h, |h|^2): h = log(q_j[k]* q_j[k+1]) on the shortest arc, the half-angle rotation
//              vector that takes this keyframe's rotation to the next one's (0 in the last frame)
// With h in the table the interpolation of step a1 needs one row instead of two and no inverse
// trigonometry per step: slerp(q0, q1, alpha) = q0 exp(alpha h), and the joint's angular velocity
// in the child frame, 2 log(q0* q1) fps, is 2 fps h.  The rows are built on the device, in double
// precision, when the clips are loaded.
// ---------------------------------------------------------------------------------------------
__global__ void clip_table_kernel(const float *__restrict__ root_pos, const float *__restrict__ local_quat,
                                  const uint8_t *__restrict__ last, long long rows, int J, float4 *__restrict__ frames)
{
    const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (i >= rows * (J + 1)) return;
    const long long r = i / (J + 1);
    const int j = (int)(i - r * (J + 1)) - 1;                  // -1: the root translation
    float4 *row = frames + r * (2 + 2 * J);
    const bool has_next = !last[r];
    if (j < 0) {
        const float *p = root_pos + 3 * r;
        row[0] = make_float4(p[0], p[1], p[2], 0.0f);
        row[1] = has_next ? make_float4((float)((double)p[3] - p[0]), (float)((double)p[4] - p[1]), (float)((double)p[5] - p[2]), 0.0f)
                          : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        return;
    }
    const float *a = local_quat + 4 * (r * J + j);
    double q0[4] = {a[0], a[1], a[2], a[3]};
    const double n0 = sqrt(q0[0] * q0[0] + q0[1] * q0[1] + q0[2] * q0[2] + q0[3] * q0[3]);
    for (int c = 0; c < 4; ++c) q0[c] /= n0;
    row[2 + 2 * j] = make_float4((float)q0[0], (float)q0[1], (float)q0[2], (float)q0[3]);
    double h[3] = {0.0, 0.0, 0.0};
    if (has_next) {
        const float *bq = a + 4 * J;
        double q1[4] = {bq[0], bq[1], bq[2], bq[3]};
        const double n1 = sqrt(q1[0] * q1[0] + q1[1] * q1[1] + q1[2] * q1[2] + q1[3] * q1[3]);
        for (int c = 0; c < 4; ++c) q1[c] /= n1;
        // rel = q0* q1, on the shortest arc
        double w = q0[0] * q1[0] + q0[1] * q1[1] + q0[2] * q1[2] + q0[3] * q1[3];
        double x = q0[0] * q1[1] - q0[1] * q1[0] - q0[2] * q1[3] + q0[3] * q1[2];
        double y = q0[0] * q1[2] + q0[1] * q1[3] - q0[2] * q1[0] - q0[3] * q1[1];
        double z = q0[0] * q1[3] - q0[1] * q1[2] + q0[2] * q1[1] - q0[3] * q1[0];
        if (w < 0.0) { w = -w; x = -x; y = -y; z = -z; }
        const double n = sqrt(x * x + y * y + z * z);
        const double k = n < 1e-12 ? 1.0 : atan2(n, w) / n;
        h[0] = k * x; h[1] = k * y; h[2] = k * z;
    }
    const float hx = (float)h[0], hy = (float)h[1], hz = (float)h[2];
    row[3 + 2 * j] = make_float4(hx, hy, hz, hx * hx + hy * hy + hz * hz);
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
    float p = fmaf(0.03978244f, u, 0.04871319f);     // n = 8, 7
    p = fmaf(p, u, 0.06156806f);           // n = 6
    p = fmaf(p, u, 0.08126984f);           // n = 5
    p = fmaf(p, u, 0.11428571f);           // n = 4
    p = fmaf(p, u, 0.17777778f);           // n = 3
    p = fmaf(p, u, 0.33333333f);           // n = 2
    return fmaf(p, u, 1.0f);               // n = 1
}

// Keyframe words of one joint: the rotation and the log of the step to the next keyframe.  The two
// 16-byte words are one aligned 32-byte sector, fetched with a single 256-bit load: every lane gathers from a
// row of its own, so each load instruction costs the load pipe one pass per lane.  The loads ask L2 to evict the
// table last: it is a few MB that every step gathers from, while hundreds of MB of body states and observation
// rows (and the policy's activations between two steps) stream through the same cache.
struct KeyPair {
    float4 a, b;
};
__device__ __forceinline__ KeyPair ld_pair(const float4 *p)
{
    KeyPair k;
    uint64_t keep;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
    asm("ld.global.nc.L2::cache_hint.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8], %9;"
        : "=f"(k.a.x), "=f"(k.a.y), "=f"(k.a.z), "=f"(k.a.w), "=f"(k.b.x), "=f"(k.b.y), "=f"(k.b.z), "=f"(k.b.w)
        : "l"(p), "l"(keep));
    return k;
}
__device__ __forceinline__ KeyPair ld_keys(const float4 *r0, int b) { return ld_pair(r0 + 2 + 2 * b); }

// Shortest-arc slerp of one joint from the table's (keyframe, half-angle log) pair: q0 exp(alpha h), with
// exp(alpha h) = (cos(alpha theta), sin(alpha theta) / theta h), theta = |h| <= pi / 2.  Keyframes of a motion
// clip are close together, so the usual case (theta <= 0.5) takes cos and sin(x)/x from their Taylor
// polynomials in (alpha theta)^2 (truncation below 2e-8); a larger step goes through sincosf.  If asked, also
// the joint's angular velocity in the child frame, which is constant over the interval: 2 fps h.
template <bool VEL>
__device__ __forceinline__ void slerp_joint(const KeyPair &key, float alpha, float fps2, Quat &q, Vec3 &wl)
{
    const Quat k0 = {key.a.x, key.a.y, key.a.z, key.a.w};
    const Vec3 h = {key.b.x, key.b.y, key.b.z};
    const float th2 = key.b.w;
    const float x = alpha * alpha * th2;
    float p = fmaf(x, -1.9841270e-4f, 8.3333333e-3f);
    p = fmaf(p, x, -1.6666667e-1f);
    float s = alpha * fmaf(p, x, 1.0f);
    float g = fmaf(x, 2.4801587e-5f, -1.3888889e-3f);
    g = fmaf(g, x, 4.1666667e-2f);
    g = fmaf(g, x, -0.5f);
    float c = fmaf(g, x, 1.0f);
    if (th2 > 0.25f) {
        const float th = sqrtf(th2);
        float sn;
        sincosf(alpha * th, &sn, &c);
        s = sn / th;
    }
    q = qmul(k0, Quat{c, s * h.x, s * h.y, s * h.z});
    if (VEL) wl = {fps2 * h.x, fps2 * h.y, fps2 * h.z};
}

// Squared rotation angle, in [0, pi^2], of the rotation r (a quaternion of any positive norm).  Small
// angles (below 0.8 rad, the usual tracking error) use the arcsine series on sin^2(theta/2).
__device__ __forceinline__ float angle_sq(Quat r)
{
    const float n2 = fmaf(r.z, r.z, fmaf(r.y, r.y, r.x * r.x));
    const float u = __fdividef(n2, fmaf(r.w, r.w, n2));    // sin^2(theta / 2)
    float th_sq = 4.0f * u * asin2_over_u(u);
    if (!(u <= 0.15f)) {
        const float th = 2.0f * atan2f(sqrtf(n2), fabsf(r.w));
        th_sq = th * th;
    }
    return th_sq;
}

// World transform (and velocities) carried down a kinematic chain (step a2).
struct Walk {
    Quat q;
    Vec3 p, v, w;
};

// One link of the chain as read from shared memory.
struct LinkRec {
    Vec3 off;
    float mass_frac;
    int b, flags;
};
__device__ __forceinline__ LinkRec ld_link(const float4 *links, int k)
{
    const float4 a = links[2 * k];
    const int4 i = *reinterpret_cast<const int4 *>(links + 2 * k + 1);
    return {{a.x, a.y, a.z}, a.w, i.x, i.y};
}
#ifdef IM_DEBUG
// (checked build: position within the chain and the body index it holds)
#define ld_link(links, k) ld_link_checked(links, k, len, J, P.status)
__device__ __forceinline__ LinkRec ld_link_checked(const float4 *links, int k, int len, int J, uint32_t *status)
{
    LinkRec L = (ld_link)(links, (int)checked((uint32_t)k, (uint32_t)len, status));
    L.b = (int)checked((uint32_t)L.b, (uint32_t)J, status);
    return L;
}
#endif

// Compose the interpolated joint onto the running transform.  k == 0 is the root, whose position is the
// lerp of the row's root position along its displacement.
template <bool VEL>
__device__ __forceinline__ void joint_compose(const float4 *r0, float alpha, float fps, const LinkRec &L, int k, Walk &s,
                                              Quat ql, Vec3 wl)
{
    if (k == 0) {
        const KeyPair root = ld_pair(r0);
        const float4 a = root.a, d = root.b;
        s.q = ql;
        s.p = {fmaf(alpha, d.x, a.x), fmaf(alpha, d.y, a.y), fmaf(alpha, d.z, a.z)};
        if (VEL) {
            s.v = {d.x * fps, d.y * fps, d.z * fps};
            s.w = qrot(ql, wl);
        }
    } else {
        const Vec3 arm = qrot(s.q, L.off);
        if (VEL) s.v = cross_add(s.w, arm, s.v);
        s.p = s.p + arm;
        s.q = qmul(s.q, ql);
        if (VEL) s.w = qrot_add(s.q, wl, s.w);
    }
}

template <bool VEL>
__device__ __forceinline__ void joint_step(const float4 *r0, const KeyPair &key, float alpha, float fps, const LinkRec &L,
                                           int k, Walk &s, Quat &ql, Vec3 &wl)
{
    slerp_joint<VEL>(key, alpha, fps + fps, ql, wl);
    joint_compose<VEL>(r0, alpha, fps, L, k, s, ql, wl);
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

// Phase bin of time t in a clip whose start times span [0, span]: floor(t / (span / B)) in single
// fp32 operations, clamped to B - 1.
__device__ __forceinline__ int phase_bin(float t, float span, int B)
{
    const float width = __fdiv_rn(span, (float)B);
    if (!(width > 0.0f)) return 0;
    const int b = (int)floorf(__fdiv_rn(t, width));
    return min(max(b, 0), B - 1);
}

// Looped clips: root displacement after `cyc` completed cycles, and a time moved `ahead` seconds on -- clamped to
// the clip's end, or, on a looped clip, wrapped (one fp32 subtraction per completed cycle, counted in cyc).
__device__ __forceinline__ Vec3 loop_shift(const ClipLoop &loop, int cyc)
{
    const float n = (float)cyc;
    return {n * loop.sx, n * loop.sy, n * loop.sz};
}
template <bool OPT>
__device__ __forceinline__ float time_ahead(const ClipLoop &loop, float dur, float t, float ahead, int &cyc)
{
    float t2 = __fadd_rn(t, ahead);
    if (!(OPT && loop.on)) return fminf(t2, dur);
    for (int i = 0; i < 64 && t2 >= dur; ++i) { t2 = __fsub_rn(t2, dur); ++cyc; }
    return t2;
}

// Heading frame of the character the observation is taken from: origin at the
// root's (x, y, 0), yaw of the root's rotated x axis (step a6).
struct Heading {
    float ox, oy, c, s;
    __device__ __forceinline__ Vec3 turn(Vec3 a) const { return {fmaf(s, a.y, c * a.x), fmaf(-s, a.x, c * a.y), a.z}; }
    // the same for a position: relative to the origin first
    __device__ __forceinline__ Vec3 local(Vec3 p) const { return turn(Vec3{p.x - ox, p.y - oy, p.z}); }
};

__device__ __forceinline__ Heading make_heading(Quat q_root, Vec3 p_root)
{
    const Vec3 h = qcol_x(q_root);
    const float n2 = fmaf(h.y, h.y, h.x * h.x);
    const float inv = rsqrtf(n2);
    const bool ok = n2 >= 1e-12f;
    return {p_root.x, p_root.y, ok ? h.x * inv : 1.0f, ok ? h.y * inv : 0.0f};
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
    const Vec3 pl = H.local(p);
    const Vec3 tn = H.turn(qcol_x(q)), nm = H.turn(qcol_z(q));
    const Vec3 vl = H.turn(v), wl = H.turn(w);
    const float o[15] = {pl.x, pl.y, pl.z, tn.x, tn.y, tn.z, nm.x, nm.y, nm.z, vl.x, vl.y, vl.z, wl.x, wl.y, wl.z};
    store_run<15>(row, 15 * b, o);
}
// The 9 target floats of one body of the reference: position and orientation columns in the heading frame.
__device__ __forceinline__ void target_obs(const Heading &H, Quat q, Vec3 p, float (&o)[9])
{
    const Vec3 tp = H.local(p);
    const Vec3 tt = H.turn(qcol_x(q)), tm = H.turn(qcol_z(q));
    o[0] = tp.x; o[1] = tp.y; o[2] = tp.z; o[3] = tt.x; o[4] = tt.y; o[5] = tt.z; o[6] = tm.x; o[7] = tm.y; o[8] = tm.z;
}

struct SimBody {
    Quat q;
    Vec3 p, v, w;
};

// A simulated quaternion of zero or non-finite norm is replaced by the identity and reported.
__device__ __forceinline__ Quat sanitize(Quat q, uint32_t *status)
{
    const float n2 = fmaf(q.z, q.z, fmaf(q.y, q.y, fmaf(q.x, q.x, q.w * q.w)));
    if (!(n2 > 1e-12f && n2 < 1e12f)) {
        atomicOr(status, IM_DEV_BAD_SIM_QUAT);
        return {1, 0, 0, 0};
    }
    return q;
}

// Body-state access of one thread (one env).  Two layouts:
//   component rows (AOS = false): element (row, env) of an array lies at row * stride + env, rows 3 b + c (4 b + c for
//     the quaternions); a warp load is one full line.  Offsets are 32-bit (the launcher checks the array sizes).
//   simulator records (AOS = true): element (env, body b, component c) lies at base + env * env_stride +
//     b * body_stride + c, read where the simulator keeps it; every lane walks its own record, the components of a
//     body are adjacent words.
template <bool AOS>
struct SimView {
    float *pos, *quat, *lin, *ang;        // rows: array bases; records: this env's record in each array
    uint32_t st, e;                       // rows
    int bs_pos, bs_quat, bs_lin, bs_ang;  // records: floats between two bodies

    __device__ __forceinline__ SimView(const EnvKernelParams &P, int envc)
    {
        if (AOS) {
            pos = P.pos + (long long)envc * P.aos_env_stride[0];
            quat = P.quat + (long long)envc * P.aos_env_stride[1];
            lin = P.lin + (long long)envc * P.aos_env_stride[2];
            ang = P.ang + (long long)envc * P.aos_env_stride[3];
            bs_pos = P.aos_body_stride[0]; bs_quat = P.aos_body_stride[1]; bs_lin = P.aos_body_stride[2]; bs_ang = P.aos_body_stride[3];
            st = 0; e = 0;
        } else {
            pos = P.pos; quat = P.quat; lin = P.lin; ang = P.ang;
            st = (uint32_t)P.stride; e = (uint32_t)envc;
            bs_pos = bs_quat = bs_lin = bs_ang = 0;
        }
    }
    __device__ __forceinline__ Quat ld_quat(int b) const
    {
        if (AOS) { const float *p = quat + (long long)b * bs_quat; return {p[0], p[1], p[2], p[3]}; }
        const uint32_t o = 4 * (uint32_t)b * st + e;
        // streaming loads (evict first): the body states are read once, the keyframe table should stay in L2
        return {__ldcs(quat + o), __ldcs(quat + o + st), __ldcs(quat + o + 2 * st), __ldcs(quat + o + 3 * st)};
    }
    __device__ __forceinline__ Vec3 ld_vec(const float *base, int bs, int b) const
    {
        if (AOS) { const float *p = base + (long long)b * bs; return {p[0], p[1], p[2]}; }
        const uint32_t o = 3 * (uint32_t)b * st + e;
        return {__ldcs(base + o), __ldcs(base + o + st), __ldcs(base + o + 2 * st)};
    }
    __device__ __forceinline__ Vec3 ld_pos(int b) const { return ld_vec(pos, bs_pos, b); }
    __device__ __forceinline__ Vec3 ld_lin(int b) const { return ld_vec(lin, bs_lin, b); }
    __device__ __forceinline__ Vec3 ld_ang(int b) const { return ld_vec(ang, bs_ang, b); }
    __device__ __forceinline__ void st_vec(float *base, int bs, int b, Vec3 v) const
    {
        if (AOS) { float *p = base + (long long)b * bs; p[0] = v.x; p[1] = v.y; p[2] = v.z; return; }
        const uint32_t o = 3 * (uint32_t)b * st + e;
        base[o] = v.x; base[o + st] = v.y; base[o + 2 * st] = v.z;
    }
    __device__ __forceinline__ void st_body(int b, Quat q, Vec3 p, Vec3 v, Vec3 w) const
    {
        st_vec(pos, bs_pos, b, p); st_vec(lin, bs_lin, b, v); st_vec(ang, bs_ang, b, w);
        if (AOS) { float *d = quat + (long long)b * bs_quat; d[0] = q.w; d[1] = q.x; d[2] = q.y; d[3] = q.z; return; }
        const uint32_t o = 4 * (uint32_t)b * st + e;
        quat[o] = q.w; quat[o + st] = q.x; quat[o + 2 * st] = q.y; quat[o + 3 * st] = q.z;
    }
};

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// Copies the staged half rows to the observation buffers.  Warp w takes rows w, w + n_warps, ..; a row leaves as
// 16-byte stores, 512 contiguous bytes per warp store.  `quads` 16-byte words of each staged row (row stride S
// floats) go to float4 positions [first, first + quads) of the destination row, positions up to `last` are
// zero-filled (the padding of the row).  F32 / BF16 select the destinations at compile time.
template <bool F32, bool BF16>
__device__ __forceinline__ void copy_out(const EnvKernelParams &P, const float *tile, int S, int rows, int quads, int first,
                                         int last, int warp, int n_warps, int lane)
{
    const uint32_t src_lane = (uint32_t)__cvta_generic_to_shared(tile) + 16u * lane;
    const int e0 = blockIdx.x * kTile;
    quads = min(quads, last - first);             // the staged stride may be wider than what is left of the row
    for (int r = warp; r < rows; r += n_warps) {
        const size_t row_off = (size_t)IM_CHECKED(e0 + r, P.N) * P.ld_obs + 4 * (first + lane);
        float4 *dst = F32 ? reinterpret_cast<float4 *>(P.obs + row_off) : nullptr;
        uint2 *dst16 = BF16 ? reinterpret_cast<uint2 *>(P.obs_bf16 + row_off) : nullptr;
        uint32_t src = src_lane + (uint32_t)(r * S) * 4u;
        int i = lane;
        for (; i < quads; i += 32, src += 512u) {
            const float4 v = lds128(src);
            if (F32) { __stcs(dst, v); dst += 32; }                 // streamed: written once, not read by this kernel
            if (BF16) { *dst16 = pack_bf16x4(v); dst16 += 32; }
        }
        for (; i < last - first; i += 32) {
            if (F32) { *dst = make_float4(0.0f, 0.0f, 0.0f, 0.0f); dst += 32; }
            if (BF16) { *dst16 = make_uint2(0u, 0u); dst16 += 32; }
        }
    }
}
__device__ __forceinline__ void copy_out_any(const EnvKernelParams &P, const float *tile, int S, int quads, int first, int last,
                                             int warp, int n_warps, int lane)
{
    const int rows = min(kTile, P.N - (int)blockIdx.x * kTile);
    // (a policy-serving loop may ask for the bf16 rows only: obs null)
    if (P.obs && P.obs_bf16) copy_out<true, true>(P, tile, S, rows, quads, first, last, warp, n_warps, lane);
    else if (P.obs) copy_out<true, false>(P, tile, S, rows, quads, first, last, warp, n_warps, lane);
    else copy_out<false, true>(P, tile, S, rows, quads, first, last, warp, n_warps, lane);
}

// Kernel body.  The observation row is assembled in two halves that reuse the same shared
// memory: columns [0, c1) -- the body blocks and, if 15 J is not a multiple of 4, the phase and
// the first target floats -- and columns [c1, D) -- the targets.
// OPT compiles in the optional semantics (grace steps, motion randomisation, adaptive initialisation, extended
// observation); envs that use none run the instantiation without them.
template <bool RESET_ALL, bool OPT, bool AOS>
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
    const int RS = 2 + 2 * J;

    // this chain's link records: global -> shared, private to the warp
    float4 *links = reinterpret_cast<float4 *>(part + (size_t)kPartials * C * kTile) + 2 * sk.link_start[c];
    for (int i = lane; i < 2 * len; i += 32) links[i] = __ldg(P.links + 2 * sk.link_start[c] + i);
    __syncwarp();

    if (c == 0)
        for (int i = 15 * J; i < c1; ++i) row1[i] = 0.0f;   // columns between the body blocks and the split

    int clip = 0, cyc = 0;
    float t1 = 0.0f;
    ClipMeta cm = {2, 1.0f, 1.0f, 0};
    ClipLoop loop = {0.0f, 0.0f, 0.0f, 0};
    Heading H = {0.0f, 0.0f, 1.0f, 0.0f};
    float root_z = 0.0f;
    const SimView<AOS> sv(P, envc);

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
        if (OPT && P.loops) {
            // a clip played in a loop: the time wraps at the clip's end and the env's cycle count goes up
            loop = P.loops[clip];
            cyc = P.cycle[envc];
            if (loop.on && t1 >= cm.dur) { t1 = __fsub_rn(t1, cm.dur); ++cyc; }
        }
        int frame;
        float alpha;
        lookup(cm, t1, frame, alpha);
        const float4 *r0 = P.frames + (size_t)IM_CHECKED(frame, P.n_rows) * RS;
        LinkRec L = ld_link(links, 0);
        KeyPair keys = ld_keys(r0, L.b);

        const Quat q_root = sanitize(sv.ld_quat(0), P.status);
        const Vec3 p_root = sv.ld_pos(0);
        H = make_heading(q_root, p_root);
        root_z = p_root.z;

        float acc[kPartials];
#pragma unroll
        for (int i = 0; i < kPartials; ++i) acc[i] = 0.0f;
        Walk s;
        Quat qa = {1, 0, 0, 0};                      // simulated state of the previous body of the chain
        Vec3 wa = {0, 0, 0};
        if (first_own > 0) {
            const int a = ld_link(links, first_own - 1).b;
            qa = sanitize(sv.ld_quat(a), P.status);
            wa = sv.ld_ang(a);
        }
        for (int k = 0; k < len; ++k) {
            const LinkRec Lc = L;
            const int b = Lc.b;
            const bool own = Lc.flags & LINK_OWN;
            SimBody sim;
            if (own) {                                // issue the loads before the interpolation math
                if (!AOS) (void)IM_CHECKED((4 * (uint32_t)b + 3) * sv.st + sv.e, 4u * (uint32_t)J * sv.st);
                sim.q = sv.ld_quat(b);
                sim.p = sv.ld_pos(b);
                sim.v = sv.ld_lin(b);
                sim.w = sv.ld_ang(b);
            }
            const KeyPair cur = keys;
            if (k + 1 < len) {                        // next joint's link and keyframe words in flight
                L = ld_link(links, k + 1);
                keys = ld_keys(r0, L.b);
            }
            Quat ql;
            Vec3 wl;
            joint_step<true>(r0, cur, alpha, cm.fps, Lc, k, s, ql, wl);
            if (OPT && k == 0) s.p = s.p + loop_shift(loop, cyc);    // completed cycles of a looped clip move the root
            if (own) {
                sim.q = sanitize(sim.q, P.status);
                // the root's "parent" is the identity: qa = (1, 0, 0, 0), wa = 0 on the chain that owns it
                const Quat ql_sim = qmul_conj(qa, sim.q);
                const Vec3 wl_sim = qrot_inv(sim.q, sim.w - wa);
                const float th_sq = angle_sq(qmul_conj(ql, ql_sim));
                const Vec3 dwl = wl_sim - wl;
                const Vec3 dp = sim.p - s.p;
                const Vec3 dv = sim.v - s.v;
                const float dp2 = dot(dp, dp);
                acc[0] += th_sq;
                acc[1] += dot(dwl, dwl);
                if (Lc.flags & LINK_EE) {
                    acc[2] += dp2;
                    acc[3] += angle_sq(qmul_conj(s.q, sim.q));
                }
                acc[4] += dp2;
                acc[5] += dot(dv, dv);
                acc[6] = fmaf(Lc.mass_frac, dp.x, acc[6]);
                acc[7] = fmaf(Lc.mass_frac, dp.y, acc[7]);
                acc[8] = fmaf(Lc.mass_frac, dp.z, acc[8]);
                (void)IM_CHECKED(15 * b + 14, c1);
                body_obs(H, sim.q, sim.p, sim.v, sim.w, row1, b);
                qa = sim.q;
                wa = sim.w;
            }
        }
#pragma unroll
        for (int i = 0; i < kPartials; ++i) part[(i * C + c) * kTile + lane] = acc[i];
    }
    __syncthreads();

    // ---- decision.  Chain 0 adds the chains' partial sums in chain order, forms the reward and writes reward,
    //      flags and the new per-env state.  Every other thread of the env needs the flags as well: it repeats the
    //      reward only if the reward can terminate an episode (r_min above -inf), else the root height and the
    //      clip end decide alone.  The reset draw is a function of (env, step) and is repeated by every thread.
    int flags = 0;
    float t_cur = t1;
    int clip_cur = clip;
    float reward_val = 0.0f;
    if (!RESET_ALL) {
        float r = 0.0f;
        const bool need_r = c == 0 || P.reward.r_min > -INFINITY;
        if (need_r) {
            float e[kPartials];
#pragma unroll
            for (int i = 0; i < kPartials; ++i) {
                float a = 0.0f;
                for (int cc = 0; cc < C; ++cc) a += part[(i * C + cc) * kTile + lane];
                e[i] = a;
            }
            // term order of the configuration: pose, vel, ee_pos, ee_rot, com, body_pos, body_vel
            const float term[IM_N_TERMS] = {e[0], e[1], e[2], e[3], e[6] * e[6] + e[7] * e[7] + e[8] * e[8], e[4], e[5]};
            if (P.reward.mode == 0) {
                float sum = 0.0f;
#pragma unroll
                for (int k = 0; k < IM_N_TERMS; ++k) sum += P.reward.w[k] * term[k];
                r = expf(-sum);
            } else {
#pragma unroll
                for (int k = 0; k < IM_N_TERMS; ++k) r += P.reward.a[k] * expf(-P.reward.w[k] * term[k]);
            }
            if (c == 0 && valid) {
                P.reward_out[env] = r;
                if (P.terms_out) {
#pragma unroll
                    for (int k = 0; k < IM_N_TERMS; ++k) P.terms_out[(size_t)k * P.N + env] = term[k];
                }
            }
        }
        bool terminated = (root_z < P.reward.h_min) || (r < P.reward.r_min);
        if (OPT && P.ep_len[envc] < P.grace_steps) terminated = false;
        if (OPT && P.n_bins > 0 && terminated && c == 0 && valid) {
            // adaptive initialisation statistics: the (clip, phase bin) the episode failed in
            const float span = fmaxf(__fsub_rn(cm.dur, P.dt), 0.0f);
            atomicAdd(P.stat_failures + clip * P.n_bins + phase_bin(t1, span, P.n_bins), 1u);
        }
        const bool truncated = !(OPT && loop.on) && __fadd_rn(t1, P.dt) > cm.dur;    // a looped clip has no end
        flags = (terminated ? 1 : 0) | (truncated ? 2 : 0);
        reward_val = r;
        if (c == 0 && valid) P.flags_out[env] = (uint8_t)flags;
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
    if (reset) cyc = 0;
    if (c == 0) {
        int ep_done = 0;                    // steps of the episode this step ended (0 where none ended)
        if (valid) {
            const int len_now = P.ep_len[env] + 1;
            P.clip_id[env] = clip_cur;
            P.t[env] = t_cur;
            if (OPT && P.loops) P.cycle[env] = cyc;
            P.ep_len[env] = reset ? 0 : len_now;
            ep_done = reset ? len_now : 0;
        }
        if (OPT && !RESET_ALL && P.summary) {
            // training summaries: integer sums over the tile (one warp), then one atomic per quantity
            unsigned long long v[4] = {valid ? (unsigned long long)__float2ll_rn(reward_val * 1099511627776.0f) : 0ull,
                                       (unsigned long long)(valid ? (flags & 1) : 0), (unsigned long long)(valid ? (flags >> 1) & 1 : 0),
                                       (unsigned long long)ep_done};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v[i] += __shfl_xor_sync(0xffffffffu, v[i], o);
                if (lane == 0 && v[i]) atomicAdd(P.summary + i, v[i]);
            }
        }
    }
    const ClipMeta cmc = reset ? P.meta[clip_cur] : cm;
    if (OPT && P.loops && reset) loop = P.loops[clip_cur];

    // ---- pass C (only where an env of this warp was reset): reference state at the new phase
    //      replaces the simulated one in the observation, and optionally in the caller's arrays
    if (__any_sync(0xffffffffu, reset)) {
        int frame;
        float alpha;
        lookup(cmc, t_cur, frame, alpha);
        const float4 *r0 = P.frames + (size_t)IM_CHECKED(frame, P.n_rows) * RS;
        LinkRec L = ld_link(links, 0);
        KeyPair keys = ld_keys(r0, L.b);
        Walk s;
        Heading Hn = H;
        for (int k = 0; k < len; ++k) {
            const LinkRec Lc = L;
            const int b = Lc.b;
            const KeyPair cur = keys;
            if (k + 1 < len) {
                L = ld_link(links, k + 1);
                keys = ld_keys(r0, L.b);
            }
            Quat ql;
            Vec3 wl;
            if (OPT && P.reset_noise_std > 0.0f) {
                // motion randomisation: the joint turns by a small random rotation in its own frame and
                // the root is shifted; every chain that walks a shared body draws the same numbers
                slerp_joint<true>(cur, alpha, cmc.fps + cmc.fps, ql, wl);
                ql = qmul(ql, reset_noise_quat(P, envc, b));
                joint_compose<true>(r0, alpha, cmc.fps, Lc, k, s, ql, wl);
                if (k == 0) s.p = s.p + reset_noise_vec(P, envc, sk.J);
            } else {
                joint_step<true>(r0, cur, alpha, cmc.fps, Lc, k, s, ql, wl);
            }
            if (k == 0) Hn = make_heading(s.q, s.p);
            if ((Lc.flags & LINK_OWN) && reset) {
                body_obs(Hn, s.q, s.p, s.v, s.w, row1, b);
                if (!RESET_ALL && P.write_back && valid) {
                    sv.st_body(b, s.q, s.p, s.v, s.w);
                }
            }
        }
        if (reset) H = Hn;
    }

    // ---- the first half also holds the phase and the first floats of the root's target when 15 J
    //      is not a multiple of 4: chain 0 interpolates the root one interval ahead for them
    int cyc_t = cyc;
    const float t_tgt = time_ahead<OPT>(loop, cmc.dur, t_cur, P.dt, cyc_t);
    int frame_t;
    float alpha_t;
    lookup(cmc, t_tgt, frame_t, alpha_t);
    const float4 *rt0 = P.frames + (size_t)IM_CHECKED(frame_t, P.n_rows) * RS;
    float phase = 0.0f;
    if (c == 0) {
        phase = t_cur / cmc.dur;
        if (15 * J < c1) {
            const KeyPair root = ld_pair(rt0);
            Vec3 rp = {fmaf(alpha_t, root.b.x, root.a.x), fmaf(alpha_t, root.b.y, root.a.y), 0.0f};
            if (OPT) rp = rp + loop_shift(loop, cyc_t);
            const Vec3 tp = H.local(rp);
            row1[15 * J] = phase;
            if (15 * J + 1 < c1) row1[15 * J + 1] = tp.x;
            if (15 * J + 2 < c1) row1[15 * J + 2] = tp.y;
        }
    }
    __syncthreads();

    // ---- first half of the rows to global memory
    copy_out_any(P, tile, S1, c1 >> 2, 0, c1 >> 2, c, C, lane);
    __syncthreads();

    // ---- pass B: reference pose one control interval ahead, seen from the same heading frame,
    //      into the second half (which reuses the shared memory of the first)
    {
        if (c == 0) {
            for (int i = D_ext - c1; i < S2; ++i) row2[i] = 0.0f;
            if (15 * J >= c1) row2[15 * J - c1] = phase;
        }
        LinkRec L = ld_link(links, 0);
        KeyPair keys = ld_keys(rt0, L.b);
        Walk s;
        for (int k = 0; k < len; ++k) {
            const LinkRec Lc = L;
            const int b = Lc.b;
            const KeyPair cur = keys;
            if (k + 1 < len) {
                L = ld_link(links, k + 1);
                keys = ld_keys(rt0, L.b);
            }
            Quat ql;
            Vec3 wl;
            joint_step<false>(rt0, cur, alpha_t, cmc.fps, Lc, k, s, ql, wl);
            if (OPT && k == 0) s.p = s.p + loop_shift(loop, cyc_t);
            if (Lc.flags & LINK_OWN) {
                float o[9];
                target_obs(H, s.q, s.p, o);
                const int col = 15 * J + 1 + 9 * b;
                (void)IM_CHECKED(col + 8 - c1, S2);
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
                int cyc_f = cyc;
                const float t_f = time_ahead<OPT>(loop, cmc.dur, t_cur, __fmul_rn((float)f, P.dt), cyc_f);
                int frame_f;
                float alpha_f;
                lookup(cmc, t_f, frame_f, alpha_f);
                const float4 *rf0 = P.frames + (size_t)IM_CHECKED(frame_f, P.n_rows) * RS;
                Walk sf;
                for (int k = 0; k < len; ++k) {
                    const LinkRec Lf = ld_link(links, k);
                    const int b = Lf.b;
                    const KeyPair kp = ld_keys(rf0, b);
                    Quat ql;
                    Vec3 wl;
                    joint_step<false>(rf0, kp, alpha_f, cmc.fps, Lf, k, sf, ql, wl);
                    if (k == 0) sf.p = sf.p + loop_shift(loop, cyc_f);
                    if ((Lf.flags & LINK_OWN) && (Lf.flags & LINK_EE)) {
                        float o[9];
                        target_obs(H, sf.q, sf.p, o);
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
    copy_out_any(P, tile, S2, S2 >> 2, c1 >> 2, P.ld_obs >> 2, c, C, lane);
}

// Diagnostic kernel: the scalar building blocks of the env kernel on caller-given inputs, one thread per item.
__global__ void debug_math_kernel(int op, int n, const float *__restrict__ in, float *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (op == 0) {                                   // squared rotation angle of a quaternion of any norm
        const float *q = in + 4 * i;
        out[i] = angle_sq(Quat{q[0], q[1], q[2], q[3]});
    } else {                                         // slerp from (keyframe, half-angle log, blend factor), fps = 1
        const float *v = in + 8 * i;
        const KeyPair key = {make_float4(v[0], v[1], v[2], v[3]),
                             make_float4(v[4], v[5], v[6], v[4] * v[4] + v[5] * v[5] + v[6] * v[6])};
        Quat q;
        Vec3 wl;
        slerp_joint<true>(key, v[7], 2.0f, q, wl);
        float *o = out + 7 * i;
        o[0] = q.w; o[1] = q.x; o[2] = q.y; o[3] = q.z; o[4] = wl.x; o[5] = wl.y; o[6] = wl.z;
    }
}

// Two instantiations per mode: skeletons with at most 8 leaves (blocks of up to 256 threads) get a
// register budget that lets four blocks share an SM; wider trees fall back to 64 registers.
#ifndef IM_ENV_MAXNREG
#define IM_ENV_MAXNREG 96
#endif
template <bool RESET_ALL, bool OPT, bool AOS>
__global__ void __maxnreg__(IM_ENV_MAXNREG) env_step_kernel_small(const __grid_constant__ EnvKernelParams P)
{
    extern __shared__ __align__(16) float smem_raw[];
    env_step_body<RESET_ALL, OPT, AOS>(P, smem_raw);
}

template <bool RESET_ALL, bool OPT, bool AOS>
__global__ void __launch_bounds__(1024, 1) env_step_kernel_wide(const __grid_constant__ EnvKernelParams P)
{
    extern __shared__ __align__(16) float smem_raw[];
    env_step_body<RESET_ALL, OPT, AOS>(P, smem_raw);
}

template <bool RESET_ALL, bool OPT, bool AOS>
cudaError_t prepare_one(size_t smem)
{
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = cudaFuncSetAttribute(env_step_kernel_small<RESET_ALL, OPT, AOS>, attr, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(env_step_kernel_wide<RESET_ALL, OPT, AOS>, attr, (int)smem);
    return e;
}

template <bool RESET_ALL, bool OPT, bool AOS>
void launch_one(const EnvKernelParams &p, dim3 grid, dim3 block, size_t smem, cudaStream_t stream)
{
    if (block.x <= 256) env_step_kernel_small<RESET_ALL, OPT, AOS><<<grid, block, smem, stream>>>(p);
    else env_step_kernel_wide<RESET_ALL, OPT, AOS><<<grid, block, smem, stream>>>(p);
}

}  // namespace

size_t env_kernel_smem_bytes(int J, int n_chains, int n_links, int extra_cols)
{
    return smem_floats(J, n_chains, n_links, extra_cols) * sizeof(float);
}

cudaError_t env_kernel_prepare(size_t smem)
{
    static DeviceOnce once;
    return once.run([&] {
        cudaError_t e = prepare_one<false, false, false>(smem);
        if (e == cudaSuccess) e = prepare_one<true, false, false>(smem);
        if (e == cudaSuccess) e = prepare_one<false, true, false>(smem);
        if (e == cudaSuccess) e = prepare_one<true, true, false>(smem);
        if (e == cudaSuccess) e = prepare_one<false, false, true>(smem);
        if (e == cudaSuccess) e = prepare_one<false, true, true>(smem);
        return e;
    });
}

cudaError_t launch_clip_table(const float *root_pos, const float *local_quat, const uint8_t *last, int64_t rows, int J,
                              float4 *frames, cudaStream_t stream)
{
    const long long n = (long long)rows * (J + 1);
    clip_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(root_pos, local_quat, last, (long long)rows, J, frames);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

cudaError_t launch_debug_math(int op, int n, const float *in, float *out, cudaStream_t stream)
{
    debug_math_kernel<<<(n + 127) / 128, 128, 0, stream>>>(op, n, in, out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

cudaError_t launch_env_kernel(const EnvKernelParams &p, bool reset_all, size_t smem, cudaStream_t stream)
{
    const dim3 grid((p.N + kTile - 1) / kTile), block(32 * p.sk.n_chains);
    const bool opt = p.grace_steps > 0 || p.reset_noise_std > 0.0f || p.n_bins > 0 || p.n_future > 1 || p.act_dim > 0 ||
                     p.summary != nullptr || p.loops != nullptr;
    if (p.aos && !reset_all) {               // simulator records read in place (the reset-all launch reads no body states)
        if (opt) launch_one<false, true, true>(p, grid, block, smem, stream);
        else launch_one<false, false, true>(p, grid, block, smem, stream);
    } else if (opt) {
        if (reset_all) launch_one<true, true, false>(p, grid, block, smem, stream);
        else launch_one<false, true, false>(p, grid, block, smem, stream);
    } else {
        if (reset_all) launch_one<true, false, false>(p, grid, block, smem, stream);
        else launch_one<false, false, false>(p, grid, block, smem, stream);
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError();
}

}  // namespace im
