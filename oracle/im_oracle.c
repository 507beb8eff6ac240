/*
 * CPU oracle for the imitation-step hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, scalar restatement of what one control step computes outside
 * the physics solver in the paper's training loop (Figure 2: reward and dones,
 * masked reset, observation building, policy inference), written to be checked
 * against the paper by eye.  It is not part of the product: only the tests,
 * the smoke check and the benchmark's CPU-baseline leg call it, and it shares
 * no code with the CUDA library.
 *
 * Precision: every quantity that is compared within a tolerance (observations,
 * rewards, error terms, policy means, Gaussian draws) is computed in fp64.
 * Every quantity that is compared bit for bit (the per-env time, keyframe
 * index, flags, reset clip id and phase, Philox words) is computed with single
 * IEEE fp32 operations or integers, so that any conforming fp32 implementation
 * reproduces it exactly.  Build with -ffp-contract=off.
 *
 * Conventions (the paper fixes only the quaternion order, Figure 3a): right
 * handed, z up, metres / seconds / radians, unit Hamilton quaternions stored
 * w,x,y,z, R(q)v = q v q*, parent[0] = -1, parent[j] < j.
 *
 * Every function below has at least one pin in tests/ that does not restate
 * its formula (closed forms, invariants, brute force with 3x3 matrices, the
 * paper's Figure 5 constants, published Philox known answers; for the advantage
 * estimator: the discounted-sum form of its definition and geometric series).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_BODIES 32
#define ORC_N_TERMS 7
#define ORC_STREAM_RESET 0u
#define ORC_STREAM_ACTION 1u
#define ORC_STREAM_RESET_NOISE 2u

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al. 2011): counter-based generator the method    */
/* draws its reset phases and action noise from.                             */
/* ------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------------------------------------ */
/* Quaternion algebra, fp64.                                                 */
/* ------------------------------------------------------------------------ */
void orc_quat_mul(const double a[4], const double b[4], double out[4])
{
    double w = a[0]*b[0] - a[1]*b[1] - a[2]*b[2] - a[3]*b[3];
    double x = a[0]*b[1] + a[1]*b[0] + a[2]*b[3] - a[3]*b[2];
    double y = a[0]*b[2] - a[1]*b[3] + a[2]*b[0] + a[3]*b[1];
    double z = a[0]*b[3] + a[1]*b[2] - a[2]*b[1] + a[3]*b[0];
    out[0] = w; out[1] = x; out[2] = y; out[3] = z;
}

static void quat_conj(const double a[4], double out[4])
{
    out[0] = a[0]; out[1] = -a[1]; out[2] = -a[2]; out[3] = -a[3];
}

/* R(q) v = q (0,v) q*  written out as the product of the three quaternions. */
void orc_quat_rotate(const double q[4], const double v[3], double out[3])
{
    double p[4] = {0.0, v[0], v[1], v[2]}, qc[4], t[4], r[4];
    quat_conj(q, qc);
    orc_quat_mul(q, p, t);
    orc_quat_mul(t, qc, r);
    out[0] = r[1]; out[1] = r[2]; out[2] = r[3];
}

static void quat_rotate_inv(const double q[4], const double v[3], double out[3])
{
    double qc[4];
    quat_conj(q, qc);
    orc_quat_rotate(qc, v, out);
}

static void quat_normalize(double q[4])
{
    double n = sqrt(q[0]*q[0] + q[1]*q[1] + q[2]*q[2] + q[3]*q[3]);
    if (n > 0.0) { q[0] /= n; q[1] /= n; q[2] /= n; q[3] /= n; }
    else { q[0] = 1.0; q[1] = q[2] = q[3] = 0.0; }
}

/* Half-angle rotation vector of a unit quaternion on the shortest arc:
 * log(q) = v/|v| * atan2(|v|, w), with q negated first when w < 0. */
void orc_quat_log(const double q_in[4], double out[3])
{
    double q[4] = {q_in[0], q_in[1], q_in[2], q_in[3]};
    if (q[0] < 0.0) { q[0] = -q[0]; q[1] = -q[1]; q[2] = -q[2]; q[3] = -q[3]; }
    double n = sqrt(q[1]*q[1] + q[2]*q[2] + q[3]*q[3]);
    if (n < 1e-12) { out[0] = out[1] = out[2] = 0.0; return; }
    double h = atan2(n, q[0]);
    out[0] = q[1] / n * h; out[1] = q[2] / n * h; out[2] = q[3] / n * h;
}

/* Rotation angle in [0, pi] of a unit quaternion: 2 atan2(|v|, |w|). */
double orc_geodesic_angle(const double q[4])
{
    double n = sqrt(q[1]*q[1] + q[2]*q[2] + q[3]*q[3]);
    return 2.0 * atan2(n, fabs(q[0]));
}

/* Angle of the rotation taking frame a to frame b: theta(a* b). */
static double rel_angle(const double a[4], const double b[4])
{
    double ac[4], r[4];
    quat_conj(a, ac);
    orc_quat_mul(ac, b, r);
    return orc_geodesic_angle(r);
}

/* Shortest-arc spherical interpolation; normalised lerp when nearly equal. */
void orc_slerp(const double q0[4], const double q1_in[4], double alpha, double out[4])
{
    double q1[4] = {q1_in[0], q1_in[1], q1_in[2], q1_in[3]};
    double d = q0[0]*q1[0] + q0[1]*q1[1] + q0[2]*q1[2] + q0[3]*q1[3];
    if (d < 0.0) { d = -d; for (int i = 0; i < 4; ++i) q1[i] = -q1[i]; }
    double s0, s1;
    if (d > 1.0 - 1e-6) { s0 = 1.0 - alpha; s1 = alpha; }
    else {
        double theta = acos(d), s = sin(theta);
        s0 = sin((1.0 - alpha) * theta) / s;
        s1 = sin(alpha * theta) / s;
    }
    for (int i = 0; i < 4; ++i) out[i] = s0 * q0[i] + s1 * q1[i];
    quat_normalize(out);
}

/* ------------------------------------------------------------------------ */
/* Skeleton and clip library.                                                */
/* ------------------------------------------------------------------------ */
typedef struct {
    int J;
    int parent[ORC_MAX_BODIES];
    double offset[ORC_MAX_BODIES][3];
    double mass[ORC_MAX_BODIES];
    int n_ee;
    int ee[ORC_MAX_BODIES];
} orc_skeleton;

typedef struct {
    int C, J;
    int *K;            /* keyframes per clip */
    float *fps;        /* fp32, as given */
    float *dur;        /* D_c = (K_c - 1) / fps_c, one fp32 division */
    int64_t *start;    /* first frame of each clip in the packed tables */
    double *root;      /* [sum K][3] */
    double *quat;      /* [sum K][J][4], renormalised */
    int *cyclic;       /* per clip: the motion repeats (orc_clips_set_cyclic); 0 by default */
    double *shift;     /* [C][3] root displacement of one cycle, P[K-1] - P[0] */
} orc_clips;

orc_skeleton *orc_skeleton_create(int J, const int32_t *parents, const float *offsets,
                                  const float *masses, const int32_t *ee_ids, int n_ee)
{
    if (J < 1 || J > ORC_MAX_BODIES || parents[0] != -1) return NULL;
    orc_skeleton *s = (orc_skeleton *)calloc(1, sizeof(*s));
    s->J = J;
    for (int j = 0; j < J; ++j) {
        if (j > 0 && (parents[j] < 0 || parents[j] >= j)) { free(s); return NULL; }
        s->parent[j] = parents[j];
        for (int c = 0; c < 3; ++c) s->offset[j][c] = (double)offsets[3*j + c];
        s->mass[j] = masses ? (double)masses[j] : 1.0;
    }
    if (ee_ids && n_ee > 0) {
        s->n_ee = n_ee;
        for (int i = 0; i < n_ee; ++i) s->ee[i] = ee_ids[i];
    } else {            /* default end-effectors: bodies without children */
        int has_child[ORC_MAX_BODIES] = {0};
        for (int j = 1; j < J; ++j) has_child[parents[j]] = 1;
        for (int j = 0; j < J; ++j) if (!has_child[j]) s->ee[s->n_ee++] = j;
    }
    return s;
}

void orc_skeleton_destroy(orc_skeleton *s) { free(s); }

orc_clips *orc_clips_create(const orc_skeleton *skel, int C, const int32_t *n_frames,
                            const float *fps, const float *root_pos, const float *local_quat)
{
    orc_clips *c = (orc_clips *)calloc(1, sizeof(*c));
    int J = skel->J;
    c->C = C; c->J = J;
    c->K = (int *)malloc(sizeof(int) * C);
    c->fps = (float *)malloc(sizeof(float) * C);
    c->dur = (float *)malloc(sizeof(float) * C);
    c->start = (int64_t *)malloc(sizeof(int64_t) * C);
    int64_t total = 0;
    for (int i = 0; i < C; ++i) {
        c->K[i] = n_frames[i];
        c->fps[i] = fps[i];
        c->dur[i] = (float)(n_frames[i] - 1) / fps[i];
        c->start[i] = total;
        total += n_frames[i];
    }
    c->root = (double *)malloc(sizeof(double) * total * 3);
    c->quat = (double *)malloc(sizeof(double) * total * J * 4);
    c->cyclic = (int *)calloc(C, sizeof(int));
    c->shift = (double *)calloc((size_t)3 * (size_t)C, sizeof(double));
    for (int64_t i = 0; i < total * 3; ++i) c->root[i] = (double)root_pos[i];
    for (int i = 0; i < C; ++i)
        for (int k = 0; k < 3; ++k)
            c->shift[3*i + k] = (double)root_pos[3 * (c->start[i] + n_frames[i] - 1) + k] - (double)root_pos[3 * c->start[i] + k];
    for (int64_t i = 0; i < total * J; ++i) {
        double q[4] = {local_quat[4*i], local_quat[4*i+1], local_quat[4*i+2], local_quat[4*i+3]};
        quat_normalize(q);
        memcpy(c->quat + 4*i, q, sizeof(q));
    }
    return c;
}

void orc_clips_destroy(orc_clips *c)
{
    if (!c) return;
    free(c->K); free(c->fps); free(c->dur); free(c->start); free(c->root); free(c->quat); free(c->cyclic); free(c->shift); free(c);
}

/* Cyclic clips (periodic motions such as the paper's walk and run): a clip flagged cyclic is played in a loop.
 * Its last keyframe is the pose of the first one, displaced by the root translation of one cycle,
 * shift = P[K-1] - P[0].  An env on such a clip never truncates: when its time reaches the clip's duration it
 * wraps (one fp32 subtraction of the duration) and the env's cycle count goes up by one; the reference at cycle
 * n is the clip's pose with n * shift added to the root (and so to every body).  flags: [C] bytes, or NULL to
 * clear all. */
void orc_clips_set_cyclic(orc_clips *c, const uint8_t *flags)
{
    for (int i = 0; i < c->C; ++i) c->cyclic[i] = flags ? (flags[i] != 0) : 0;
}

float orc_clip_duration(const orc_clips *c, int clip) { return c->dur[clip]; }

/* ------------------------------------------------------------------------ */
/* Step a1: keyframe index and blend factor at time t.                       */
/* f = fl32(t * fps); k = min(floor(f), K-2); alpha = f - k in [0,1].        */
/* ------------------------------------------------------------------------ */
void orc_lookup_index(float t, float fps, int K, int32_t *k_out, double *alpha_out)
{
    volatile float f = t * fps;           /* one fp32 multiply, round to nearest */
    int k = (int)floorf(f);
    if (k > K - 2) k = K - 2;
    if (k < 0) k = 0;
    double a = (double)f - (double)k;
    if (a < 0.0) a = 0.0;
    if (a > 1.0) a = 1.0;
    *k_out = k; *alpha_out = a;
}

/* Reference character state at (clip, t): steps a1 + a2. */
typedef struct {
    double ql[ORC_MAX_BODIES][4];   /* local (parent-relative) rotations   */
    double wl[ORC_MAX_BODIES][3];   /* joint angular velocity, child frame  */
    double p[ORC_MAX_BODIES][3];    /* world positions                      */
    double q[ORC_MAX_BODIES][4];    /* world rotations                      */
    double v[ORC_MAX_BODIES][3];    /* world linear velocities              */
    double w[ORC_MAX_BODIES][3];    /* world angular velocities             */
    double com[3];
} orc_ref;

static void cross3(const double a[3], const double b[3], double out[3])
{
    out[0] = a[1]*b[2] - a[2]*b[1];
    out[1] = a[2]*b[0] - a[0]*b[2];
    out[2] = a[0]*b[1] - a[1]*b[0];
}

static void center_of_mass(const orc_skeleton *s, double p[][3], double com[3])
{
    double m = 0.0;
    com[0] = com[1] = com[2] = 0.0;
    for (int j = 0; j < s->J; ++j) {
        m += s->mass[j];
        for (int c = 0; c < 3; ++c) com[c] += s->mass[j] * p[j][c];
    }
    for (int c = 0; c < 3; ++c) com[c] /= m;
}

static void forward_kinematics(const orc_skeleton *s, orc_ref *r);

void orc_reference_state(const orc_skeleton *s, const orc_clips *cl, int clip, float t, orc_ref *r)
{
    int J = s->J, K = cl->K[clip], k;
    double alpha, fps = (double)cl->fps[clip];
    orc_lookup_index(t, cl->fps[clip], K, &k, &alpha);
    const double *P0 = cl->root + 3 * (cl->start[clip] + k), *P1 = P0 + 3;
    const double *Q0 = cl->quat + 4 * (int64_t)J * (cl->start[clip] + k), *Q1 = Q0 + 4 * J;

    /* a1: slerp each joint, lerp the root, finite-difference velocities */
    for (int j = 0; j < J; ++j) {
        double q0c[4], rel[4], lg[3];
        orc_slerp(Q0 + 4*j, Q1 + 4*j, alpha, r->ql[j]);
        quat_conj(Q0 + 4*j, q0c);
        orc_quat_mul(q0c, Q1 + 4*j, rel);
        orc_quat_log(rel, lg);
        for (int c = 0; c < 3; ++c) r->wl[j][c] = 2.0 * lg[c] * fps;
    }
    for (int c = 0; c < 3; ++c) {
        r->p[0][c] = (1.0 - alpha) * P0[c] + alpha * P1[c];
        r->v[0][c] = (P1[c] - P0[c]) * fps;
    }
    forward_kinematics(s, r);
}

/* a2: forward kinematics with velocity propagation from the local rotations ql, the joint
 * angular velocities wl and the root's position and linear velocity (p[0], v[0]). */
static void forward_kinematics(const orc_skeleton *s, orc_ref *r)
{
    int J = s->J;
    memcpy(r->q[0], r->ql[0], sizeof(double) * 4);
    orc_quat_rotate(r->q[0], r->wl[0], r->w[0]);
    for (int j = 1; j < J; ++j) {
        int a = s->parent[j];
        double arm[3], wj[3], wxr[3];
        orc_quat_mul(r->q[a], r->ql[j], r->q[j]);
        orc_quat_rotate(r->q[a], s->offset[j], arm);
        orc_quat_rotate(r->q[j], r->wl[j], wj);
        cross3(r->w[a], arm, wxr);
        for (int c = 0; c < 3; ++c) {
            r->p[j][c] = r->p[a][c] + arm[c];
            r->w[j][c] = r->w[a][c] + wj[c];
            r->v[j][c] = r->v[a][c] + wxr[c];
        }
    }
    center_of_mass(s, r->p, r->com);
}

/* Reference state of a cyclic clip in its cycle `cyc`: the clip's own state with cyc * shift added to every
 * position (rotations and velocities repeat). */
static void reference_state_cyc(const orc_skeleton *s, const orc_clips *cl, int clip, float t, int cyc, orc_ref *r)
{
    orc_reference_state(s, cl, clip, t, r);
    if (cyc == 0) return;
    for (int c = 0; c < 3; ++c) {
        double d = (double)cyc * cl->shift[3*clip + c];
        for (int j = 0; j < s->J; ++j) r->p[j][c] += d;
        r->com[c] += d;
    }
}

/* Time `t_in` moved `ahead` seconds on in a clip (fp32: one addition, and for a cyclic clip one subtraction
 * of the duration per completed cycle): a non-cyclic clip clamps at its end.  *cyc is advanced. */
static float time_ahead(const orc_clips *cl, int clip, float t_in, float ahead, int *cyc)
{
    volatile float t = t_in + ahead;
    float dur = cl->dur[clip];
    if (!cl->cyclic[clip]) return t < dur ? t : dur;
    while (t >= dur) { t = t - dur; *cyc += 1; }
    return t;
}

/* Flat export of orc_reference_state for the tests. */
void orc_reference_state_flat(const orc_skeleton *s, const orc_clips *cl, int clip, float t,
                              double *p, double *q, double *v, double *w,
                              double *ql, double *wl, double *com)
{
    orc_ref r;
    orc_reference_state(s, cl, clip, t, &r);
    for (int j = 0; j < s->J; ++j) {
        for (int c = 0; c < 3; ++c) {
            p[3*j+c] = r.p[j][c]; v[3*j+c] = r.v[j][c]; w[3*j+c] = r.w[j][c]; wl[3*j+c] = r.wl[j][c];
        }
        for (int c = 0; c < 4; ++c) { q[4*j+c] = r.q[j][c]; ql[4*j+c] = r.ql[j][c]; }
    }
    for (int c = 0; c < 3; ++c) com[c] = r.com[c];
}

/* ------------------------------------------------------------------------ */
/* Environment configuration (mirrors what a caller of the method chooses).  */
/* ------------------------------------------------------------------------ */
typedef struct {
    int32_t mode;                   /* 0 multiplicative, 1 additive */
    float a[ORC_N_TERMS];           /* additive coefficients */
    float w[ORC_N_TERMS];           /* error scales; order: pose, vel, ee_pos, ee_rot, com, body_pos, body_vel */
    float h_min;                    /* terminate when root height < h_min */
    float r_min;                    /* terminate when reward < r_min (-inf: off) */
} orc_reward_config;

typedef struct {
    float dt;
    uint32_t seed_lo, seed_hi;
    orc_reward_config reward;
    int32_t write_back_reset;
    int32_t grace_steps;            /* no early termination while fewer than this many steps of the episode are done */
    float reset_noise_std;          /* motion randomisation of the state an env is reset to (0: off) */
    /* adaptive episode initialisation: B phase bins per clip with a cumulative table over the C*B
     * (clip, bin) pairs; n_bins = 0 keeps the uniform draw */
    int32_t n_bins;
    const uint64_t *reset_cdf;      /* [C*B] exclusive upper thresholds in [0, 2^32], see orc_reset_cdf */
    uint32_t *stat_starts;          /* [C*B] episodes started in the bin (or NULL) */
    uint32_t *stat_failures;        /* [C*B] early terminations that happened in the bin (or NULL) */
    /* extended observation (Section 6: "future reference end-effector frames, and the previous action"), appended
     * after the 24J+1 entries; zero fields switch it off:
     *   n_future F > 1: for f = 2..F and each end effector in body order, position (3) and first and third
     *     rotation column (3 + 3) of the reference at min(t + f dt, D_clip), seen from the observed root's heading frame
     *   act_dim A > 0: the A entries of prev_action[i] (zeros for an env that was just reset) */
    int32_t n_future;
    int32_t act_dim;
    const float *prev_action;       /* [n][ld_action] */
    int64_t ld_action;
    int32_t *cycle;                 /* [n] per-env cycle count of cyclic clips (state, updated by the step), or NULL */
} orc_env_config;

/* Cumulative table of a weight table w[n] >= 0 (not all zero): T_i = floor(2^32 (w_0 + .. + w_i) / total)
 * with the sums taken in order in fp64, T_{n-1} = 2^32.  A 32-bit uniform word x selects the smallest
 * i with x < T_i, so bin i is drawn with probability (T_i - T_{i-1}) / 2^32 and a bin of weight 0 never. */
int orc_reset_cdf(int n, const float *w, uint64_t *T)
{
    double total = 0.0, cum = 0.0;
    for (int i = 0; i < n; ++i) {
        if (!(w[i] >= 0.0f) || isinf(w[i])) return -1;
        total += (double)w[i];
    }
    if (!(total > 0.0)) return -1;
    for (int i = 0; i < n; ++i) {
        cum += (double)w[i];
        T[i] = (uint64_t)floor(cum / total * 4294967296.0);
    }
    T[n - 1] = 4294967296ull;
    return 0;
}

/* Phase bin of time t in a clip whose start times span [0, span]: floor(t / (span / B)) in single
 * fp32 operations, clamped to B - 1 (times past the last start time fall in the last bin). */
static int phase_bin(float t, float span, int B)
{
    volatile float width = span / (float)B;
    if (!(width > 0.0f)) return 0;
    volatile float f = t / width;
    int b = (int)floorf(f);
    return b < 0 ? 0 : (b > B - 1 ? B - 1 : b);
}

/* Body state of one env, fp64 working copy. */
typedef struct {
    double p[ORC_MAX_BODIES][3], q[ORC_MAX_BODIES][4], v[ORC_MAX_BODIES][3], w[ORC_MAX_BODIES][3];
} orc_body_state;

/* Step a3: the seven error terms between a simulated state and the reference
 * (Section 6.1 names pose, velocity, COM, end-effector position/orientation;
 * Figure 5 adds whole-body position and velocity sums). */
static void error_terms(const orc_skeleton *s, const orc_body_state *x, const orc_ref *r, double e[ORC_N_TERMS])
{
    int J = s->J;
    for (int k = 0; k < ORC_N_TERMS; ++k) e[k] = 0.0;
    for (int j = 0; j < J; ++j) {
        int a = s->parent[j];
        double ql_sim[4], wl_sim[3], dw[3];
        if (a < 0) {
            memcpy(ql_sim, x->q[j], sizeof(ql_sim));
            dw[0] = x->w[j][0]; dw[1] = x->w[j][1]; dw[2] = x->w[j][2];
        } else {
            double qc[4];
            quat_conj(x->q[a], qc);
            orc_quat_mul(qc, x->q[j], ql_sim);
            for (int c = 0; c < 3; ++c) dw[c] = x->w[j][c] - x->w[a][c];
        }
        quat_rotate_inv(x->q[j], dw, wl_sim);
        double th = rel_angle(r->ql[j], ql_sim);
        e[0] += th * th;
        for (int c = 0; c < 3; ++c) {
            double d = wl_sim[c] - r->wl[j][c];
            e[1] += d * d;
            double dp = x->p[j][c] - r->p[j][c];
            e[5] += dp * dp;
            double dv = x->v[j][c] - r->v[j][c];
            e[6] += dv * dv;
        }
    }
    for (int i = 0; i < s->n_ee; ++i) {
        int b = s->ee[i];
        for (int c = 0; c < 3; ++c) {
            double d = x->p[b][c] - r->p[b][c];
            e[2] += d * d;
        }
        double th = rel_angle(r->q[b], x->q[b]);
        e[3] += th * th;
    }
    double com_sim[3];
    center_of_mass(s, (double (*)[3])x->p, com_sim);
    for (int c = 0; c < 3; ++c) {
        double d = com_sim[c] - r->com[c];
        e[4] += d * d;
    }
}

/* Reward from the error terms: prod_k exp(-w_k e_k) = exp(-sum_k w_k e_k)
 * (Section 6.1) or sum_k a_k exp(-w_k e_k) (Figure 5). */
double orc_reward(const orc_reward_config *rc, const double e[ORC_N_TERMS])
{
    if (rc->mode == 0) {
        double s = 0.0;
        for (int k = 0; k < ORC_N_TERMS; ++k) s += (double)rc->w[k] * e[k];
        return exp(-s);
    }
    double r = 0.0;
    for (int k = 0; k < ORC_N_TERMS; ++k) r += (double)rc->a[k] * exp(-(double)rc->w[k] * e[k]);
    return r;
}

/* Step a5: uniform reset draw for env id `env` at step `step`. */
void orc_reset_draw(const orc_clips *cl, const orc_env_config *cfg, uint32_t env, uint32_t step,
                    int32_t *clip_out, float *t_out)
{
    uint32_t ctr[4] = {env, step, ORC_STREAM_RESET, 0u}, key[2] = {cfg->seed_lo, cfg->seed_hi}, x[4];
    orc_philox4x32_10(ctr, key, x);
    float u = (float)(x[1] >> 8) * 5.9604644775390625e-08f;       /* 2^-24, exact */
    if (cfg->n_bins > 0) {
        /* adaptive initialisation: (clip, bin) from the cumulative table, then uniform inside the bin */
        int B = cfg->n_bins, n = cl->C * B, i = 0;
        while (i < n - 1 && !((uint64_t)x[0] < cfg->reset_cdf[i])) ++i;
        int32_t clip = i / B, b = i % B;
        volatile float span = cl->dur[clip] - cfg->dt;
        if (span < 0.0f) span = 0.0f;
        volatile float width = span / (float)B;
        volatile float pos = (float)b + u;
        volatile float t = pos * width;
        if (t > span) t = span;
        *clip_out = clip; *t_out = t;
        if (cfg->stat_starts) {
#pragma omp atomic
            cfg->stat_starts[i] += 1u;
        }
        return;
    }
    int32_t clip = (int32_t)(((uint64_t)x[0] * (uint64_t)(uint32_t)cl->C) >> 32);
    volatile float span = cl->dur[clip] - cfg->dt;                  /* one fp32 subtract */
    if (span < 0.0f) span = 0.0f;
    volatile float t = u * span;                                    /* one fp32 multiply */
    *clip_out = clip; *t_out = t;
}

/* Four standard normals from one Philox block: (x0,x1) and (x2,x3) each feed one Box-Muller pair. */
static void normal4(const uint32_t ctr[4], const uint32_t key[2], double z[4])
{
    uint32_t x[4];
    orc_philox4x32_10(ctr, key, x);
    for (int h = 0; h < 2; ++h) {
        double u1 = ((double)(x[2*h] >> 8) + 1.0) * 5.9604644775390625e-08;
        double u2 = (double)(x[2*h+1] >> 8) * 5.9604644775390625e-08;
        double rad = sqrt(-2.0 * log(u1));
        z[2*h] = rad * cos(2.0 * M_PI * u2);
        z[2*h+1] = rad * sin(2.0 * M_PI * u2);
    }
}

/* Motion randomisation of a reset state (the hyper-parameter "motion randomization std" of the
 * paper's configuration table; the paper does not say what is perturbed -- reading: every joint's
 * local rotation is turned by a rotation vector n ~ N(0, std^2 I) given in the joint's own frame,
 * ql' = ql exp(n/2), and the root position is shifted by N(0, std^2 I); local joint velocities and
 * the root's linear velocity are kept, and the world state follows by forward kinematics).
 * Joint j draws from Philox counter (env, step, 2, j), the root shift from (env, step, 2, J);
 * the first three normals of a block are used. */
void orc_reset_noise(const orc_skeleton *s, const orc_env_config *cfg, uint32_t env, uint32_t step, orc_ref *r)
{
    double std = (double)cfg->reset_noise_std, z[4];
    uint32_t key[2] = {cfg->seed_lo, cfg->seed_hi};
    if (!(std > 0.0)) return;
    for (int j = 0; j <= s->J; ++j) {
        uint32_t ctr[4] = {env, step, ORC_STREAM_RESET_NOISE, (uint32_t)j};
        normal4(ctr, key, z);
        if (j == s->J) {
            for (int c = 0; c < 3; ++c) r->p[0][c] += std * z[c];
        } else {
            double n[3] = {std * z[0], std * z[1], std * z[2]};
            double th = sqrt(n[0]*n[0] + n[1]*n[1] + n[2]*n[2]);
            double k = th > 1e-12 ? sin(0.5 * th) / th : 0.5;
            double dq[4] = {cos(0.5 * th), k * n[0], k * n[1], k * n[2]}, out[4];
            orc_quat_mul(r->ql[j], dq, out);
            memcpy(r->ql[j], out, sizeof(out));
        }
    }
    forward_kinematics(s, r);
}

/* Flat export for the tests: the randomised reset state of (clip, t). */
void orc_reset_state_flat(const orc_skeleton *s, const orc_clips *cl, const orc_env_config *cfg, uint32_t env,
                          uint32_t step, int clip, float t, double *p, double *q, double *v, double *w, double *ql)
{
    orc_ref r;
    orc_reference_state(s, cl, clip, t, &r);
    orc_reset_noise(s, cfg, env, step, &r);
    for (int j = 0; j < s->J; ++j) {
        for (int c = 0; c < 3; ++c) { p[3*j+c] = r.p[j][c]; v[3*j+c] = r.v[j][c]; w[3*j+c] = r.w[j][c]; }
        for (int c = 0; c < 4; ++c) { q[4*j+c] = r.q[j][c]; ql[4*j+c] = r.ql[j][c]; }
    }
}

static void ref_to_state(const orc_skeleton *s, const orc_ref *r, orc_body_state *x)
{
    memcpy(x->p, r->p, sizeof(double) * 3 * s->J);
    memcpy(x->q, r->q, sizeof(double) * 4 * s->J);
    memcpy(x->v, r->v, sizeof(double) * 3 * s->J);
    memcpy(x->w, r->w, sizeof(double) * 3 * s->J);
}

/* Step a6: heading-local observation of state x at (clip, t), D = 24J + 1. */
static void build_obs(const orc_skeleton *s, const orc_clips *cl, const orc_env_config *cfg,
                      const orc_body_state *x, int clip, float t, int cyc, double *obs, int i, int was_reset)
{
    int J = s->J;
    const double ex[3] = {1.0, 0.0, 0.0}, ez[3] = {0.0, 0.0, 1.0};
    double hx[3];
    orc_quat_rotate(x->q[0], ex, hx);
    double psi = 0.0;
    if (sqrt(hx[0]*hx[0] + hx[1]*hx[1]) >= 1e-6) psi = atan2(hx[1], hx[0]);
    double qh_inv[4] = {cos(0.5 * psi), 0.0, 0.0, -sin(0.5 * psi)};   /* rotation by -psi about z */
    double origin[3] = {x->p[0][0], x->p[0][1], 0.0};

    for (int j = 0; j < J; ++j) {
        double *o = obs + 15 * j, d[3], ql[4];
        for (int c = 0; c < 3; ++c) d[c] = x->p[j][c] - origin[c];
        orc_quat_rotate(qh_inv, d, o + 0);
        orc_quat_mul(qh_inv, x->q[j], ql);
        orc_quat_rotate(ql, ex, o + 3);
        orc_quat_rotate(ql, ez, o + 6);
        orc_quat_rotate(qh_inv, x->v[j], o + 9);
        orc_quat_rotate(qh_inv, x->w[j], o + 12);
    }
    obs[15 * J] = (double)t / (double)cl->dur[clip];

    int cyc_tgt = cyc;
    float t_tgt = time_ahead(cl, clip, t, cfg->dt, &cyc_tgt);      /* one fp32 add; clamped, or wrapped on a cyclic clip */
    orc_ref tgt;
    reference_state_cyc(s, cl, clip, t_tgt, cyc_tgt, &tgt);
    for (int j = 0; j < J; ++j) {
        double *o = obs + 15 * J + 1 + 9 * j, d[3], ql[4];
        for (int c = 0; c < 3; ++c) d[c] = tgt.p[j][c] - origin[c];
        orc_quat_rotate(qh_inv, d, o + 0);
        orc_quat_mul(qh_inv, tgt.q[j], ql);
        orc_quat_rotate(ql, ex, o + 3);
        orc_quat_rotate(ql, ez, o + 6);
    }

    /* extended entries */
    double *o = obs + 24 * J + 1;
    for (int f = 2; f <= cfg->n_future; ++f) {
        volatile float ahead = (float)f * cfg->dt;          /* one fp32 multiplication, */
        int cyc_f = cyc;
        float t_c = time_ahead(cl, clip, t, ahead, &cyc_f);  /* one fp32 addition; clamped or wrapped */
        orc_ref fut;
        reference_state_cyc(s, cl, clip, t_c, cyc_f, &fut);
        for (int j = 0; j < J; ++j) {
            int is_ee = 0;
            for (int k = 0; k < s->n_ee; ++k) is_ee |= (s->ee[k] == j);
            if (!is_ee) continue;
            double d[3], ql[4];
            for (int c = 0; c < 3; ++c) d[c] = fut.p[j][c] - origin[c];
            orc_quat_rotate(qh_inv, d, o + 0);
            orc_quat_mul(qh_inv, fut.q[j], ql);
            orc_quat_rotate(ql, ex, o + 3);
            orc_quat_rotate(ql, ez, o + 6);
            o += 9;
        }
    }
    for (int a = 0; a < cfg->act_dim; ++a)
        *o++ = was_reset ? 0.0 : (double)cfg->prev_action[(int64_t)i * cfg->ld_action + a];
}

static void load_sim(const orc_skeleton *s, const float *pos, const float *quat, const float *lin,
                     const float *ang, int64_t stride, int64_t i, orc_body_state *x)
{
    for (int j = 0; j < s->J; ++j) {
        for (int c = 0; c < 3; ++c) {
            x->p[j][c] = (double)pos[(3*j+c) * stride + i];
            x->v[j][c] = (double)lin[(3*j+c) * stride + i];
            x->w[j][c] = (double)ang[(3*j+c) * stride + i];
        }
        for (int c = 0; c < 4; ++c) x->q[j][c] = (double)quat[(4*j+c) * stride + i];
    }
}

static void store_sim(const orc_skeleton *s, const orc_body_state *x, float *pos, float *quat,
                      float *lin, float *ang, int64_t stride, int64_t i)
{
    for (int j = 0; j < s->J; ++j) {
        for (int c = 0; c < 3; ++c) {
            pos[(3*j+c) * stride + i] = (float)x->p[j][c];
            lin[(3*j+c) * stride + i] = (float)x->v[j][c];
            ang[(3*j+c) * stride + i] = (float)x->w[j][c];
        }
        for (int c = 0; c < 4; ++c) quat[(4*j+c) * stride + i] = (float)x->q[j][c];
    }
}

/* Step 0: every env is reset (counter step 0) and its first observation is
 * built from the reference state; no reward. */
void orc_env_reset_all(const orc_skeleton *s, const orc_clips *cl, const orc_env_config *cfg,
                       int n, const uint32_t *env_ids, uint32_t step,
                       int32_t *clip_id, float *t, int32_t *ep_len,
                       double *obs, int64_t ld_obs, int n_threads)
{
    if (n_threads < 1) n_threads = 1;
#pragma omp parallel for num_threads(n_threads) schedule(static)
    for (int i = 0; i < n; ++i) {
        orc_ref r;
        orc_body_state x;
        orc_reset_draw(cl, cfg, env_ids[i], step, &clip_id[i], &t[i]);
        ep_len[i] = 0;
        if (cfg->cycle) cfg->cycle[i] = 0;
        orc_reference_state(s, cl, clip_id[i], t[i], &r);
        orc_reset_noise(s, cfg, env_ids[i], step, &r);
        ref_to_state(s, &r, &x);
        build_obs(s, cl, cfg, &x, clip_id[i], t[i], 0, obs + (int64_t)i * ld_obs, i, 1);
    }
}

/* One control step for n envs (Figure 2's post-physics phase, in its order:
 * reward and dones, masked reset, observation).  State arrays are updated in
 * place.  sim arrays are structure-of-arrays: component c of env i at
 * c*comp_stride + i.  terms may be NULL. */
void orc_env_step(const orc_skeleton *s, const orc_clips *cl, const orc_env_config *cfg,
                  int n, const uint32_t *env_ids, uint32_t step,
                  int32_t *clip_id, float *t, int32_t *ep_len,
                  float *pos, float *quat, float *linvel, float *angvel, int64_t comp_stride,
                  double *obs, int64_t ld_obs, double *reward, uint8_t *flags, double *terms,
                  int n_threads)
{
    if (n_threads < 1) n_threads = 1;
#pragma omp parallel for num_threads(n_threads) schedule(static)
    for (int i = 0; i < n; ++i) {
        orc_ref r;
        orc_body_state x;
        double e[ORC_N_TERMS];
        int clip = clip_id[i];

        int cyc = cfg->cycle ? cfg->cycle[i] : 0;
        volatile float t_adv = t[i] + cfg->dt;                      /* a0: one fp32 add */
        float t1 = t_adv;
        if (cl->cyclic[clip] && t1 >= cl->dur[clip]) {              /* a cyclic clip wraps: one fp32 subtract */
            volatile float t_wrap = t1 - cl->dur[clip];
            t1 = t_wrap;
            cyc += 1;
        }
        reference_state_cyc(s, cl, clip, t1, cyc, &r);               /* a1, a2 */
        load_sim(s, pos, quat, linvel, angvel, comp_stride, i, &x);
        error_terms(s, &x, &r, e);                                   /* a3 */
        double rew = orc_reward(&cfg->reward, e);
        reward[i] = rew;
        if (terms) for (int k = 0; k < ORC_N_TERMS; ++k) terms[(int64_t)k * n + i] = e[k];

        /* a4: flags.  Root height is compared as the fp32 input value. */
        float root_z = pos[2 * comp_stride + i];
        int terminated = (root_z < cfg->reward.h_min) || (rew < (double)cfg->reward.r_min);
        if (ep_len[i] < cfg->grace_steps) terminated = 0;           /* early-termination grace steps */
        if (terminated && cfg->n_bins > 0 && cfg->stat_failures) {  /* where the episode failed */
            volatile float span = cl->dur[clip] - cfg->dt;
            if (span < 0.0f) span = 0.0f;
            int b = phase_bin(t1, span, cfg->n_bins);
#pragma omp atomic
            cfg->stat_failures[clip * cfg->n_bins + b] += 1u;
        }
        volatile float t2 = t1 + cfg->dt;
        int truncated = !cl->cyclic[clip] && t2 > cl->dur[clip];    /* a cyclic clip has no end */
        flags[i] = (uint8_t)(terminated | (truncated << 1));

        float t_cur = t1;
        if (flags[i]) {                                              /* a5 */
            orc_reset_draw(cl, cfg, env_ids[i], step, &clip, &t_cur);
            ep_len[i] = 0;
            cyc = 0;
            orc_reference_state(s, cl, clip, t_cur, &r);
            orc_reset_noise(s, cfg, env_ids[i], step, &r);
            ref_to_state(s, &r, &x);
            if (cfg->write_back_reset) store_sim(s, &x, pos, quat, linvel, angvel, comp_stride, i);
        } else {
            ep_len[i] += 1;
        }
        clip_id[i] = clip;
        t[i] = t_cur;
        if (cfg->cycle) cfg->cycle[i] = cyc;
        build_obs(s, cl, cfg, &x, clip, t_cur, cyc, obs + (int64_t)i * ld_obs, i, flags[i] != 0);   /* a6 */
    }
}

/* ------------------------------------------------------------------------ */
/* Step e: policy MLP forward and Gaussian action sampling.                  */
/* ------------------------------------------------------------------------ */

/* Standard normals for env `env` at step `step`: Philox block i gives four
 * words; (x0,x1) and (x2,x3) each feed one Box-Muller pair. */
void orc_action_noise(uint32_t seed_lo, uint32_t seed_hi, uint32_t env, uint32_t step, int A, double *z)
{
    uint32_t key[2] = {seed_lo, seed_hi};
    for (int blk = 0; 4 * blk < A; ++blk) {
        uint32_t ctr[4] = {env, step, ORC_STREAM_ACTION, (uint32_t)blk}, x[4];
        orc_philox4x32_10(ctr, key, x);
        for (int h = 0; h < 2; ++h) {
            double u1 = ((double)(x[2*h] >> 8) + 1.0) * 5.9604644775390625e-08;
            double u2 = (double)(x[2*h+1] >> 8) * 5.9604644775390625e-08;
            double rad = sqrt(-2.0 * log(u1));
            double zc = rad * cos(2.0 * M_PI * u2), zs = rad * sin(2.0 * M_PI * u2);
            if (4*blk + 2*h < A) z[4*blk + 2*h] = zc;
            if (4*blk + 2*h + 1 < A) z[4*blk + 2*h + 1] = zs;
        }
    }
}

/* Nearest-even rounding of a value to bf16 (through fp32), as a double. */
double orc_round_bf16(double x)
{
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return (double)f;      /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* h_{l+1} = relu(W_l h_l + b_l), last layer linear -> mean; a = mean + sigma z.
 * Weights W_l are [dims[l+1]][dims[l]] fp32 values (bf16 weights widened
 * exactly by the caller); accumulation in fp64.  With bf16_operands the
 * operands of every layer are bf16 values, as the bf16 configurations
 * prescribe ("bf16 operands, fp32 accumulation"): the observation and each
 * hidden activation are rounded to bf16 before they enter the next layer;
 * otherwise activations are never rounded. */
void orc_policy_forward_std(int n_layers, const int32_t *dims, const float *const *W, const float *const *b,
                            double sigma, const float *log_std, uint32_t seed_lo, uint32_t seed_hi, uint32_t step,
                            int n, const uint32_t *env_ids, const double *obs, int64_t ld_obs,
                            double *mean, double *action, double *logp, double *z_out, int n_threads,
                            int bf16_operands);

void orc_policy_forward(int n_layers, const int32_t *dims, const float *const *W, const float *const *b,
                        double sigma, uint32_t seed_lo, uint32_t seed_hi, uint32_t step,
                        int n, const uint32_t *env_ids, const double *obs, int64_t ld_obs,
                        double *mean, double *action, double *logp, double *z_out, int n_threads,
                        int bf16_operands)
{
    orc_policy_forward_std(n_layers, dims, W, b, sigma, NULL, seed_lo, seed_hi, step, n, env_ids, obs, ld_obs,
                           mean, action, logp, z_out, n_threads, bf16_operands);
}

/* The same with a state-independent standard deviation per action dimension, sigma_i =
 * exp(log_std[i]) (the "policy log std" parameter of the paper's hyper-parameter table);
 * log_std == NULL uses the scalar sigma for every dimension.
 * a_i = mean_i + sigma_i z_i;  logp = -0.5 sum z^2 - sum_i ln sigma_i - (A/2) ln 2 pi. */
void orc_policy_forward_std(int n_layers, const int32_t *dims, const float *const *W, const float *const *b,
                            double sigma, const float *log_std, uint32_t seed_lo, uint32_t seed_hi, uint32_t step,
                            int n, const uint32_t *env_ids, const double *obs, int64_t ld_obs,
                            double *mean, double *action, double *logp, double *z_out, int n_threads,
                            int bf16_operands)
{
    int maxd = 0, A = dims[n_layers];
    for (int l = 0; l <= n_layers; ++l) if (dims[l] > maxd) maxd = dims[l];
    if (n_threads < 1) n_threads = 1;
#pragma omp parallel for num_threads(n_threads) schedule(static)
    for (int i = 0; i < n; ++i) {
        double *h0 = (double *)malloc(sizeof(double) * maxd), *h1 = (double *)malloc(sizeof(double) * maxd);
        double *z = (double *)malloc(sizeof(double) * (A + 4));
        for (int k = 0; k < dims[0]; ++k) {
            h0[k] = obs[(int64_t)i * ld_obs + k];
            if (bf16_operands) h0[k] = orc_round_bf16(h0[k]);
        }
        for (int l = 0; l < n_layers; ++l) {
            int in = dims[l], out = dims[l+1];
            for (int o = 0; o < out; ++o) {
                double acc = (double)b[l][o];
                const float *w = W[l] + (int64_t)o * in;
                for (int k = 0; k < in; ++k) acc += (double)w[k] * h0[k];
                if (l < n_layers - 1) {
                    if (acc < 0.0) acc = 0.0;
                    if (bf16_operands) acc = orc_round_bf16(acc);
                }
                h1[o] = acc;
            }
            double *tmp = h0; h0 = h1; h1 = tmp;
        }
        orc_action_noise(seed_lo, seed_hi, env_ids[i], step, A, z);
        double zz = 0.0;
        for (int o = 0; o < A; ++o) {
            mean[(int64_t)i * A + o] = h0[o];
            action[(int64_t)i * A + o] = h0[o] + (log_std ? exp((double)log_std[o]) : sigma) * z[o];
            if (z_out) z_out[(int64_t)i * A + o] = z[o];
            zz += z[o] * z[o];
        }
        double sum_log = (double)A * log(sigma);
        if (log_std) { sum_log = 0.0; for (int o = 0; o < A; ++o) sum_log += (double)log_std[o]; }
        if (logp) logp[i] = -0.5 * zz - sum_log - 0.5 * (double)A * log(2.0 * M_PI);
        free(h0); free(h1); free(z);
    }
}

/* Error terms and reward of one explicit (state, reference) pair; lets the
 * tests feed hand-made states. */
void orc_error_terms_flat(const orc_skeleton *s, const orc_clips *cl, int clip, float t,
                          const double *p, const double *q, const double *v, const double *w, double *e)
{
    orc_ref r;
    orc_body_state x;
    orc_reference_state(s, cl, clip, t, &r);
    for (int j = 0; j < s->J; ++j) {
        for (int c = 0; c < 3; ++c) { x.p[j][c] = p[3*j+c]; x.v[j][c] = v[3*j+c]; x.w[j][c] = w[3*j+c]; }
        for (int c = 0; c < 4; ++c) x.q[j][c] = q[4*j+c];
    }
    error_terms(s, &x, &r, e);
}

/* ------------------------------------------------------------------------
 * Generalised advantage estimation over one rollout of T control steps (the
 * estimator whose discount factor and parameter lambda the paper's Table of
 * training hyper-parameters lists; the rollout loop of the paper's training-loop
 * figure stores reward, terminated and truncated per step for it).
 *
 *   done_t  = terminated_t or truncated_t            (flags bit 0 / bit 1)
 *   r'_t    = r_t + gamma V_t   if bootstrap_truncated and truncated_t and not terminated_t
 *           = r_t               otherwise
 *   delta_t = r'_t + gamma V_{t+1} (1 - done_t) - V_t
 *   A_t     = delta_t + gamma lambda (1 - done_t) A_{t+1},      A_T = 0
 *   R_t     = A_t + V_t
 *
 * Arrays are [T][ld] (value: [T+1][ld]; row T is the value of the observation after the last
 * step), env index fastest.  fp32 inputs, fp64 arithmetic and outputs. */
void orc_gae(int T, int N, int64_t ld, const float *reward, const float *value, const uint8_t *flags,
             double gamma, double lambda, int bootstrap_truncated, double *adv, double *ret)
{
    for (int e = 0; e < N; ++e) {
        double a_next = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            const int64_t i = (int64_t)t * ld + e;
            const int terminated = flags[i] & 1, truncated = (flags[i] >> 1) & 1;
            const double live = (terminated || truncated) ? 0.0 : 1.0;
            const double v = (double)value[i], v_next = (double)value[i + ld];
            double r = (double)reward[i];
            if (bootstrap_truncated && truncated && !terminated) r += gamma * v;
            const double delta = r + gamma * v_next * live - v;
            const double a = delta + gamma * lambda * live * a_next;
            adv[i] = a;
            ret[i] = a + v;
            a_next = a;
        }
    }
}

/* ------------------------------------------------------------------------
 * PPO minibatch loss and its gradients with respect to the network outputs (the paper's
 * hyper-parameter table lists the ratio clip, the value-loss and entropy coefficients and the KL
 * threshold; the objective is the clipped surrogate of Schulman et al. 2017 as the usual on-policy
 * runners implement it).  For sample i of M, action dimension k of A, sigma_k = exp(log_std_k):
 *
 *   logp_i   = -1/2 sum_k ((a_ik - mu_ik) / sigma_k)^2 - sum_k log_std_k - A/2 ln 2 pi
 *   r_i      = exp(logp_i - logp_old_i),      Ahat_i = (adv_i - adv_mean) adv_rstd
 *   surr_i   = -min(r_i Ahat_i, clip(r_i, 1 - eps, 1 + eps) Ahat_i)
 *   vl_i     = (V_i - R_i)^2, or with value clipping max((V_i - R_i)^2, (Vc_i - R_i)^2),
 *              Vc_i = Vold_i + clip(V_i - Vold_i, -eps, eps)
 *   H        = sum_k (log_std_k + 1/2 ln(2 pi e))                 (entropy, the same for every sample)
 *   L        = mean_i surr_i + c_v mean_i vl_i - c_e H
 *   kl_i     = sum_k [log_std_k - log_std_old_k + (sigma_old_k^2 + (mu_old_ik - mu_ik)^2) / (2 sigma_k^2) - 1/2]
 *
 * Outputs: dL/dmu [M][A], dL/dlog_std [A], dL/dV [M], and summary = {L, mean surr, mean vl, H,
 * mean kl, fraction of samples with |r - 1| > eps}.  The branch of min / max that is active decides
 * the gradient (on a tie both branches have the same derivative here). */
typedef struct {
    float clip, value_coef, entropy_coef;
    int32_t clip_value_loss;
} orc_ppo_config;

void orc_ppo_loss(const orc_ppo_config *cfg, int64_t M, int A, const float *mean, const float *log_std,
                  const float *action, const float *logp_old, const float *mean_old, const float *log_std_old,
                  const float *adv, double adv_mean, double adv_rstd, const float *value, const float *value_old,
                  const float *returns, double *d_mean, double *d_log_std, double *d_value, double *summary)
{
    const double eps = (double)cfg->clip, cv = (double)cfg->value_coef, ce = (double)cfg->entropy_coef;
    double sum_log = 0.0, H = 0.0, s_surr = 0.0, s_vl = 0.0, s_kl = 0.0, s_clip = 0.0;
    for (int k = 0; k < A; ++k) {
        sum_log += (double)log_std[k];
        H += (double)log_std[k] + 0.5 * log(2.0 * M_PI * exp(1.0));
        d_log_std[k] = -ce;
    }
    for (int64_t i = 0; i < M; ++i) {
        double zz = 0.0, kl = 0.0;
        for (int k = 0; k < A; ++k) {
            double sg = exp((double)log_std[k]), so = exp((double)log_std_old[k]);
            double z = ((double)action[i * A + k] - (double)mean[i * A + k]) / sg;
            double dm = (double)mean_old[i * A + k] - (double)mean[i * A + k];
            zz += z * z;
            kl += (double)log_std[k] - (double)log_std_old[k] + (so * so + dm * dm) / (2.0 * sg * sg) - 0.5;
        }
        double logp = -0.5 * zz - sum_log - 0.5 * (double)A * log(2.0 * M_PI);
        double r = exp(logp - (double)logp_old[i]);
        double ah = ((double)adv[i] - adv_mean) * adv_rstd;
        double rc = r < 1.0 - eps ? 1.0 - eps : (r > 1.0 + eps ? 1.0 + eps : r);
        double s1 = r * ah, s2 = rc * ah;
        double g_r = s1 <= s2 ? -ah : 0.0;                 /* d surr / d r */
        s_surr += -(s1 <= s2 ? s1 : s2);
        s_clip += fabs(r - 1.0) > eps ? 1.0 : 0.0;
        s_kl += kl;
        for (int k = 0; k < A; ++k) {
            double sg = exp((double)log_std[k]);
            double z = ((double)action[i * A + k] - (double)mean[i * A + k]) / sg;
            d_mean[i * A + k] = g_r * r * z / sg / (double)M;            /* dlogp/dmu = z / sigma */
            d_log_std[k] += g_r * r * (z * z - 1.0) / (double)M;         /* dlogp/dlog_std = z^2 - 1 */
        }
        double v = (double)value[i], R = (double)returns[i], e1 = v - R, vl = e1 * e1, gv = 2.0 * e1;
        if (cfg->clip_value_loss) {
            double d = v - (double)value_old[i];
            double dc = d < -eps ? -eps : (d > eps ? eps : d);
            double e2 = (double)value_old[i] + dc - R;
            if (e2 * e2 > vl) { vl = e2 * e2; gv = (d == dc) ? 2.0 * e2 : 0.0; }
        }
        s_vl += vl;
        d_value[i] = cv * gv / (double)M;
    }
    summary[1] = s_surr / (double)M;
    summary[2] = s_vl / (double)M;
    summary[3] = H;
    summary[4] = s_kl / (double)M;
    summary[5] = s_clip / (double)M;
    summary[0] = summary[1] + cv * summary[2] - ce * H;
}

/* Mean and 1 / (std + 1e-8) of n values, std with the n - 1 divisor (advantage normalisation). */
void orc_moments(const float *x, int64_t n, double *mean_out, double *rstd_out)
{
    double s = 0.0, q = 0.0;
    for (int64_t i = 0; i < n; ++i) s += (double)x[i];
    double m = s / (double)n;
    for (int64_t i = 0; i < n; ++i) q += ((double)x[i] - m) * ((double)x[i] - m);
    *mean_out = m;
    *rstd_out = 1.0 / (sqrt(n > 1 ? q / (double)(n - 1) : 0.0) + 1e-8);
}

/* ------------------------------------------------------------------------
 * Optimiser step of the update (Adam, Kingma & Ba 2015, with bias correction, as in the usual
 * deep-learning libraries), global-norm gradient clipping and the KL-adaptive learning rate
 * that the paper's "KL threshold" hyper-parameter belongs to.
 *
 *   g      = grad * grad_scale
 *   m      = b1 m + (1 - b1) g,    v = b2 v + (1 - b2) g^2
 *   param -= lr (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps)            t = 1, 2, ...
 *
 *   grad_scale = min(1, max_norm / (||all grads||_2 + 1e-6))                (norm over every tensor)
 *
 *   lr' = max(lr / 1.5, lr_min) if kl > 2 kl_target;  min(lr * 1.5, lr_max) if 0 < kl < kl_target / 2;
 *         lr otherwise                                                      (the adaptive schedule of
 *                                                                            common on-policy runners)
 * fp32 inputs and state, fp64 arithmetic, results rounded to fp32 once. */
void orc_adam_step(int64_t n, float *param, const float *grad, float *m, float *v, double lr, double b1,
                   double b2, double eps, int t, double grad_scale)
{
    const double c1 = 1.0 - pow(b1, (double)t), c2 = 1.0 - pow(b2, (double)t);
    for (int64_t i = 0; i < n; ++i) {
        const double g = (double)grad[i] * grad_scale;
        const double mi = b1 * (double)m[i] + (1.0 - b1) * g;
        const double vi = b2 * (double)v[i] + (1.0 - b2) * g * g;
        m[i] = (float)mi;
        v[i] = (float)vi;
        param[i] = (float)((double)param[i] - lr * (mi / c1) / (sqrt(vi / c2) + eps));
    }
}

double orc_grad_scale(int n_tensors, const float *const *grads, const int64_t *sizes, double max_norm)
{
    double q = 0.0;
    for (int k = 0; k < n_tensors; ++k)
        for (int64_t i = 0; i < sizes[k]; ++i) q += (double)grads[k][i] * (double)grads[k][i];
    const double s = max_norm / (sqrt(q) + 1e-6);
    return s < 1.0 ? s : 1.0;
}

double orc_adaptive_lr(double lr, double kl, double kl_target, double lr_min, double lr_max)
{
    if (kl > 2.0 * kl_target) { lr = lr / 1.5; return lr > lr_min ? lr : lr_min; }
    if (kl > 0.0 && kl < 0.5 * kl_target) { lr = lr * 1.5; return lr < lr_max ? lr : lr_max; }
    return lr;
}

/* ------------------------------------------------------------------------
 * Backward pass of the MLP h_l = relu(W_l h_{l-1} + b_l) (last layer linear) for a batch: given
 * g = dL/d(output) per sample, the gradients of L with respect to every W_l and b_l by the chain
 * rule:  gz_L = g;  dW_l = sum_i gz_l,i h_{l-1,i}^T;  db_l = sum_i gz_l,i;
 *        gh_{l-1} = W_l^T gz_l;  gz_{l-1} = gh_{l-1} where h_{l-1} > 0, else 0.
 * With bf16_operands the tensors that enter a matrix product are bf16 values, as on the
 * tensor-core path: the input and every hidden activation (as in orc_policy_forward), the output
 * gradient, every gh (rounded when it is formed) and the resulting dW; the bias gradient of the
 * last layer sums the unrounded g.  Sums are exact (fp64).
 * dW is a flat array, layer after layer, each [dims[l+1]][dims[l]]; db likewise. */
void orc_mlp_backward(int n_layers, const int32_t *dims, const float *const *W, const float *const *b, int n,
                      const double *obs, int64_t ld_obs, const double *g_out, double *dW, double *db,
                      int bf16_operands)
{
    int maxd = 0;
    int64_t w_total = 0, b_total = 0, act_total = 0;
    for (int l = 0; l <= n_layers; ++l) { if (dims[l] > maxd) maxd = dims[l]; act_total += dims[l]; }
    for (int l = 0; l < n_layers; ++l) { w_total += (int64_t)dims[l] * dims[l + 1]; b_total += dims[l + 1]; }
    memset(dW, 0, sizeof(double) * (size_t)w_total);
    memset(db, 0, sizeof(double) * (size_t)b_total);
    double *h = (double *)malloc(sizeof(double) * (size_t)act_total);      /* activations of one sample, all layers */
    double *gz = (double *)malloc(sizeof(double) * (size_t)maxd), *gh = (double *)malloc(sizeof(double) * (size_t)maxd);
    for (int i = 0; i < n; ++i) {
        /* forward, keeping every layer's activation */
        double *h0 = h;
        for (int k = 0; k < dims[0]; ++k) h0[k] = bf16_operands ? orc_round_bf16(obs[(int64_t)i * ld_obs + k]) : obs[(int64_t)i * ld_obs + k];
        double *hin = h0;
        for (int l = 0; l < n_layers; ++l) {
            double *hout = hin + dims[l];
            for (int o = 0; o < dims[l + 1]; ++o) {
                double acc = (double)b[l][o];
                for (int k = 0; k < dims[l]; ++k) acc += (double)W[l][(int64_t)o * dims[l] + k] * hin[k];
                if (l < n_layers - 1) { acc = acc > 0.0 ? acc : 0.0; if (bf16_operands) acc = orc_round_bf16(acc); }
                hout[o] = acc;
            }
            hin = hout;
        }
        /* backward */
        const int A = dims[n_layers];
        for (int o = 0; o < A; ++o) gz[o] = g_out[(int64_t)i * A + o];
        int64_t w_off = w_total, b_off = b_total;
        double *hl = h + act_total - A;                                       /* output layer's slot */
        for (int l = n_layers - 1; l >= 0; --l) {
            const int N = dims[l + 1], K = dims[l];
            double *hprev = hl - K;
            w_off -= (int64_t)N * K; b_off -= N;
            for (int o = 0; o < N; ++o) db[b_off + o] += gz[o];                /* before operand rounding */
            if (bf16_operands) for (int o = 0; o < N; ++o) gz[o] = orc_round_bf16(gz[o]);
            for (int o = 0; o < N; ++o)
                for (int k = 0; k < K; ++k) dW[w_off + (int64_t)o * K + k] += gz[o] * hprev[k];
            if (l > 0) {
                for (int k = 0; k < K; ++k) {
                    double acc = 0.0;
                    for (int o = 0; o < N; ++o) acc += (double)W[l][(int64_t)o * K + k] * gz[o];
                    if (bf16_operands) acc = orc_round_bf16(acc);
                    gh[k] = hprev[k] > 0.0 ? acc : 0.0;
                }
                for (int k = 0; k < K; ++k) gz[k] = gh[k];
            }
            hl = hprev;
        }
    }
    if (bf16_operands) for (int64_t j = 0; j < w_total; ++j) dW[j] = orc_round_bf16(dW[j]);
    free(h); free(gz); free(gh);
}

int orc_openmp_enabled(void)
{
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}
