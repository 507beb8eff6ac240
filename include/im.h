/*
 * im.h -- C ABI of the B200 imitation-step library.
 *
 * The library implements, for N environments at once, everything a
 * DeepMimic-style training loop does per control step outside the physics
 * solver (paper Figure 2: policy inference, then the post-physics phase --
 * reward and dones, masked reset, observation building).  The simulated body
 * states are an input; physics is not part of this library.
 *
 * Conventions: right handed, z up, metres / seconds / radians.  Quaternions
 * are unit Hamilton quaternions stored w,x,y,z (paper Figure 3a), R(q)v = qvq*.
 * Bodies are ordered so that parent[0] = -1 and parent[j] < j.
 *
 * Pointer kinds: every pointer is marked HOST or DEVICE.  Set-up calls take
 * HOST pointers, copy what they need, and keep no reference.  Per-step calls
 * take DEVICE pointers that the caller owns; the library only enqueues work on
 * the CUDA stream given at creation and holds no reference once the call
 * returns.  Per-step calls never synchronise, never read device data on the
 * host, never branch on device data and never allocate (paper Section 4.2:
 * no CPU access on the rollout step; reset is unconditional with a device-side
 * mask), so a sequence of them can be captured in a CUDA graph (Section 2.2).
 *
 * Threads and devices: a handle may be used from one host thread at a time;
 * different handles may be created and used from different threads.  A handle
 * belongs to the CUDA device that was current when it was created and must be
 * used with that device current; the kernels' one-time set-up (shared-memory
 * limits, SM count) is done once per device, guarded against concurrent first
 * calls.
 *
 * Errors: a call that returns a negative status has had no effect.  Anomalies
 * found on the device (a non-finite quaternion, a wait that ran out) set bits
 * in a sticky status word, the kernel carries on with a defined fallback and
 * never traps; read the word with im_poll_device_status.
 */
#ifndef IM_H_
#define IM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif
#if defined(__GNUC__)
#pragma GCC visibility push(default)   /* the entry points below are the library's only exports */
#endif

typedef int32_t im_status;
#define IM_OK                  0
#define IM_ERR_INVALID_ARG    (-1)  /* null pointer, size out of range, misaligned buffer   */
#define IM_ERR_BAD_TOPOLOGY   (-2)  /* parent[0] != -1, parent[j] >= j, J > IM_MAX_BODIES   */
#define IM_ERR_BAD_QUAT       (-3)  /* keyframe quaternion non-finite or |q| off 1 by > 1e-3 */
#define IM_ERR_ALLOC          (-4)  /* device or host allocation failed                      */
#define IM_ERR_CUDA           (-5)  /* a CUDA runtime or driver call failed                  */
#define IM_ERR_UNSUPPORTED    (-6)  /* layer sizes / device the kernels do not cover         */

/* bits of the sticky device status word */
#define IM_DEV_BAD_SIM_QUAT    1u   /* a simulated quaternion had zero or non-finite norm; identity used */
#define IM_DEV_WAIT_TIMEOUT    2u   /* a bounded wait inside a kernel ran out; that tile's output is invalid */
#define IM_DEV_BAD_STATE       4u   /* a per-env clip id was out of range; clamped */
#define IM_DEV_DEBUG_CHECK     8u   /* bounds-checked build only: an index formed inside the env kernel was out of range */

#define IM_MAX_BODIES   32
#define IM_N_TERMS       7          /* pose, vel, ee_pos, ee_rot, com, body_pos, body_vel */
#define IM_MAX_LAYERS    8

#define IM_FLAG_TERMINATED 1u
#define IM_FLAG_TRUNCATED  2u

typedef struct im_skeleton im_skeleton;
typedef struct im_clips    im_clips;
typedef struct im_env      im_env;
typedef struct im_policy   im_policy;

const char *im_status_string(im_status s);

/* ---- skeleton -------------------------------------------------------------
 * The articulated character the reference motion is played on (forward
 * kinematics of step (a): q[j] = q[parent] * q_local[j],
 * p[j] = p[parent] + R(q[parent]) offset[j]).
 *   J         number of bodies, 1..IM_MAX_BODIES
 *   parents   HOST [J]      parent[0] = -1, parent[j] < j
 *   offsets   HOST [J][3]   body origin in the parent's frame, metres (offsets[0] ignored)
 *   masses    HOST [J] or NULL (all 1): weights of the centre of mass, which is the
 *             mass-weighted mean of the body origins
 *   ee_ids    HOST [n_ee] or NULL: end-effector bodies; NULL/0 selects every body without children
 * Returns a host-side handle; free with im_destroy_skeleton. */
im_status im_create_skeleton(int32_t J, const int32_t *parents, const float *offsets,
                             const float *masses, const int32_t *ee_ids, int32_t n_ee,
                             im_skeleton **out);
void im_destroy_skeleton(im_skeleton *s);

/* ---- reference motion clips -----------------------------------------------
 * A library of C keyframed clips (the paper's reference motions, Section 6.2).
 * Frame k of clip c holds the root position and one local (parent-relative)
 * quaternion per body.  Between keyframes the library interpolates: shortest
 * arc slerp per joint, lerp for the root.
 *   n_frames   HOST [C]            K_c >= 2
 *   fps        HOST [C]            > 0; clip duration D_c = (K_c - 1) / fps_c (one fp32 division)
 *   root_pos   HOST [sum K][3]
 *   local_quat HOST [sum K][J][4]  w,x,y,z; must be finite with | |q| - 1 | <= 1e-3; used as given (the
 *                                 interpolation and velocity formulas do not depend on the small scale error)
 * The device table is built on the current CUDA device from these arrays (fp64 arithmetic, stored as fp32): per
 * keyframe one row of 2 + 2J 16-byte words -- root position, root displacement to the next keyframe, and per
 * joint the normalised quaternion and the half-angle logarithm of the shorter-arc rotation to the next keyframe
 * -- so that interpolating a joint is one 32-byte read.  Free with im_destroy_clips. */
im_status im_load_clips(const im_skeleton *skel, int32_t C, const int32_t *n_frames, const float *fps,
                        const float *root_pos, const float *local_quat, im_clips **out);
void im_destroy_clips(im_clips *c);

/* Looped playback of periodic motions (the paper's Section 6 tracks walk and run cycles among its clips; it does
 * not say how a clip's end is handled -- this is the library's reading).  flags: HOST [C] bytes, non-zero marks a
 * clip as cyclic; NULL clears all.  A cyclic clip's last keyframe is taken to be the pose of its first one moved by
 * the root translation of one cycle, shift_c = P_c[K-1] - P_c[0].  An env on such a clip never truncates: when its
 * time reaches D_c it wraps, t <- fl32(t - D_c), and the env's cycle count n goes up by one; the reference at
 * (c, t, n) is the clip's own state at t with n shift_c added to the root position (rotations and velocities
 * repeat).  Look-ahead times (the target frame, further future frames) wrap the same way instead of clamping
 * at D_c, each with the cycle count it reaches.  A reset starts a new episode at cycle 0.  The call waits for the
 * device and takes effect for every env created on these clips, from its next step on. */
im_status im_clips_set_cyclic(im_clips *c, const uint8_t *flags);

/* ---- environment ----------------------------------------------------------
 * Reward (paper Section 6.1 and Figure 5) from seven error terms e_k between
 * the simulated character and the reference at the env's time:
 *   0 pose      sum over joints of the squared geodesic angle between reference and simulated
 *               local rotations (rad^2), root included
 *   1 vel       sum over joints of |difference of child-frame joint angular velocities|^2
 *   2 ee_pos    sum over end-effectors of |world position difference|^2
 *   3 ee_rot    sum over end-effectors of the squared geodesic angle of the world rotations
 *   4 com       |centre-of-mass difference|^2
 *   5 body_pos  sum over bodies of |world position difference|^2      (Figure 5 pose_err)
 *   6 body_vel  sum over bodies of |world linear velocity difference|^2 (Figure 5 vel_err)
 * mode 0: r = prod_k exp(-w_k e_k) (Section 6.1);  mode 1: r = sum_k a_k exp(-w_k e_k) (Figure 5). */
typedef struct {
    int32_t mode;
    float a[IM_N_TERMS];
    float w[IM_N_TERMS];
    float h_min;      /* terminated if simulated root height (z) < h_min                        */
    float r_min;      /* ... or reward < r_min; -INFINITY switches the reward test off          */
} im_reward_config;

typedef struct {
    int32_t n_envs;           /* N >= 1                                                             */
    uint32_t env_id_base;     /* env i draws random numbers as env id env_id_base + i, so a batch   */
                              /* split across devices reproduces the unsplit run                    */
    float dt;                 /* control interval, 0 < dt <= shortest clip duration                 */
    uint64_t seed;            /* Philox key                                                         */
    im_reward_config reward;
    int32_t ld_obs;           /* row stride of obs buffers in floats: >= 24J+1 and a multiple of 4; */
                              /* columns [24J+1, ld_obs) are written as zeros                       */
    int32_t write_back_reset; /* non-zero: a reset env's reference state is also stored into the    */
                              /* caller's body-state arrays (masked store)                          */
    /* Optional semantics named in the paper's hyper-parameter table; 0 switches them off.         */
    int32_t grace_steps;      /* early-termination grace steps: the terminated flag is suppressed   */
                              /* while the episode has completed fewer than this many steps         */
                              /* (truncation at the clip end is not affected)                       */
    float reset_noise_std;    /* motion randomisation: an env is reset to the reference state with  */
                              /* every joint turned, in its own frame, by a rotation vector         */
                              /* n ~ N(0, std^2 I) (q_local' = q_local exp(n/2), radians) and the   */
                              /* root shifted by N(0, std^2 I) metres; velocities of the joints and */
                              /* of the root are kept and the world state follows by forward        */
                              /* kinematics.  Joint j draws from Philox counter (env id, step, 2,   */
                              /* j), the root shift from (env id, step, 2, J); Box-Muller as for    */
                              /* the actions, first three normals of the block.  The observation    */
                              /* targets stay those of the unperturbed reference.                   */
} im_env_config;

/* Simulated body states, DEVICE, structure of arrays: component c of env e at
 * base[c * comp_stride + e]; per body 3 position rows (x,y,z), 4 quaternion
 * rows (w,x,y,z), 3 linear and 3 angular velocity rows (world frame), so pos,
 * linvel, angvel have 3J rows and quat 4J rows.  comp_stride >= N.  Each base
 * pointer and comp_stride*4 must be multiples of 16 bytes. */
typedef struct {
    float *pos;
    float *quat;
    float *linvel;
    float *angvel;
    int64_t comp_stride;
} im_body_state;

/* Creates the per-env state (clip id, time, episode length) on the current
 * device.  cuda_stream is a cudaStream_t (NULL = legacy default stream); every
 * later call on this handle enqueues there.  skel and clips must outlive it. */
im_status im_env_create(const im_skeleton *skel, const im_clips *clips, const im_env_config *cfg,
                        void *cuda_stream, im_env **out);
void im_env_destroy(im_env *e);

/* Step 0: every env is reset with Philox counter (env id, step, 0, 0) to a
 * uniform clip and a uniform start time in [0, D_clip - dt), and its first
 * observation is built from the reference state.
 *   obs_out DEVICE [N][ld_obs] */
im_status im_env_reset_all(im_env *e, uint32_t step, float *obs_out);

/* One control step (post-physics phase of Figure 2), in this order per env:
 * t += dt; reference lookup + slerp + forward kinematics at t; error terms and
 * reward; flags (terminated: root height / reward test; truncated: t + dt
 * would pass the clip end); masked reset with Philox counter (env id, step,
 * 0, 0) -- only flagged envs change clip/time, the others count one more
 * step; observation of the (possibly reset) state in the character's heading
 * frame plus the reference pose one control interval ahead.
 *   sim        DEVICE, see im_body_state (read; written only for reset envs if write_back_reset)
 *   obs_out    DEVICE [N][ld_obs]; row: J x (pos3, tangent3, normal3, linvel3, angvel3), phase t/D,
 *              J x (target pos3, tangent3, normal3), zero padding
 *   reward_out DEVICE [N]
 *   flags_out  DEVICE [N] bytes: IM_FLAG_TERMINATED | IM_FLAG_TRUNCATED
 *   terms_out  DEVICE [IM_N_TERMS][N] or NULL: the seven error terms */
im_status im_env_step(im_env *e, uint32_t step, const im_body_state *sim,
                      float *obs_out, float *reward_out, uint8_t *flags_out, float *terms_out);

/* The same step on a simulator's own arrays (array of structures), read where they
 * are (the paper's Section 4.2: post-physics kernels take simulator state from the
 * GPU-resident arrays, no host copy).  Element (env e, body j, component c) of an
 * array is base[e * env_stride + j * body_stride + c]; strides in floats, so arrays
 * with a leading world body (point base at body 1), or spatial velocities stored as
 * six floats per body (point linvel and angvel into the same array, body_stride 6),
 * are described without copying.  pos, linvel, angvel have 3 components, quat 4
 * (w,x,y,z).  DEVICE; no alignment requirement.
 * The env kernel reads the records where they lie (every thread walks the record of its env; with
 * write_back_reset the states of reset envs are stored back the same way): nothing is staged, nothing
 * allocated, the call is capturable like im_env_step, and the results are those of im_env_step on the
 * transposed data, bit for bit.  Per-thread record reads are not coalesced, so the step is slower than on
 * component rows (measured at 65536 envs x 24 bodies: 213 us against 126 us).  im_env_set_aos_staging(e, 1)
 * trades memory for time: it allocates a [13J][N] buffer once (outside any capture), after which
 * im_env_step_aos first transposes the records into it with one gather kernel and runs the env kernel on the
 * rows (168 us in the same measurement), scattering reset envs back; im_env_set_aos_staging(e, 0) frees the
 * buffer and returns to in-place reading. */
typedef struct {
    float *base;
    int64_t env_stride;
    int32_t body_stride;
} im_aos_array;

typedef struct {
    im_aos_array pos, quat, linvel, angvel;
} im_body_state_aos;

im_status im_env_step_aos(im_env *e, uint32_t step, const im_body_state_aos *sim,
                          float *obs_out, float *reward_out, uint8_t *flags_out, float *terms_out);
im_status im_env_set_aos_staging(im_env *e, int32_t on);

/* Copies the per-env state to / from DEVICE arrays of N elements (stream
 * ordered); with the step number this is all that is needed to resume a
 * rollout bit-exactly.  Any pointer may be NULL to skip that array. */
im_status im_env_get_state(im_env *e, int32_t *clip_id, float *t, int32_t *ep_len);
im_status im_env_set_state(im_env *e, const int32_t *clip_id, const float *t, const int32_t *ep_len);
/* The cycle counts of envs on cyclic clips (0 elsewhere), DEVICE int32 [N]: the fourth piece of per-env state. */
im_status im_env_get_cycles(im_env *e, int32_t *cycle);
im_status im_env_set_cycles(im_env *e, const int32_t *cycle);

/* ---- extended observation ---------------------------------------------------
 * (Section 6: observations also hold "future reference end-effector frames, and the
 * previous action"; the paper gives no layout, this one appends to the 24J+1 row.)
 *   columns [24J+1, 24J+1 + (n_future-1) * 9 * n_ee):  for each further reference frame
 *       f = 2 .. n_future, at time min(fl32(t + fl32(f * dt)), D_clip), and each end effector
 *       in body order: position (3), first and third column of the rotation (3 + 3), seen
 *       from the heading frame of the observed root exactly like the frame-1 targets
 *   then act_dim columns: prev_action[env][0..act_dim), the action the policy took before
 *       this step (DEVICE float [n_envs][ld_action], read by every later step: the caller
 *       keeps it alive and fills it, normally with the policy's action output); zeros for
 *       an env that this step reset, and after im_env_reset_all.
 * n_future = 1 and act_dim = 0 restore the 24J+1 layout.  ld_obs must hold the extended
 * row, else IM_ERR_INVALID_ARG; a policy attached for another width is detached.  Takes
 * effect with the next launch (host state only).  im_step_host does not support act_dim > 0. */
im_status im_env_set_obs_extension(im_env *e, int32_t n_future, int32_t act_dim, const float *prev_action, int32_t ld_action);

/* ---- training summaries kept on the device ------------------------------------
 * (Section 4.2 of the paper: logging must not put a host read on the rollout step, so the summaries a
 * trainer plots stay on the GPU and are read whenever convenient.)  With an accumulator attached every
 * im_env_step adds, over its N envs:
 *   acc[0] += sum of round(reward * 2^40)      (a fixed-point sum: exact, the same whatever order the
 *                                               thread blocks finish in; divide by 2^40 and the step count)
 *   acc[1] += envs flagged terminated          acc[2] += envs flagged truncated
 *   acc[3] += sum over envs reset by this step of the length, in steps, of the episode that ended
 * acc: DEVICE uint64 [4], owned by the caller (who zeroes it when a logging window starts and reads it
 * stream-ordered, e.g. once per rollout); NULL detaches.  Host state only, takes effect with the next
 * launch; the additions are integer atomics enqueued with the step (capturable).  im_env_reset_all does
 * not touch the accumulator. */
#define IM_SUMMARY_REWARD_SCALE 1099511627776.0    /* 2^40 */
im_status im_env_set_summary(im_env *e, uint64_t *acc);

/* ---- adaptive episode initialisation --------------------------------------
 * (The paper trains "with early termination and adaptive episode-initialization
 * sampling", Section 6, without giving the rule; this is the mechanism such rules
 * need, kept on the device: a weighted reset distribution and failure counts.)
 * Each clip's start times [0, D_c - dt] are cut into n_bins equal phase bins.
 * A reset draws the pair (clip, bin) with probability proportional to its weight
 * and the start time uniformly inside the bin:
 *   T_i = floor(2^32 (w_0 + ... + w_i) / sum w)   (sums in order, fp64; T_last = 2^32)
 *   i   = smallest index with x0 < T_i, clip = i / n_bins, b = i % n_bins
 *   t   = min(fl32(fl32(b + u) * fl32(span / n_bins)), span),  span = max(D_clip - dt, 0)
 * with x0 and u = (x1 >> 8) 2^-24 from the same Philox block as the uniform draw,
 * every operation a single fp32 one.  A bin of weight 0 is never drawn.
 *   weights  HOST [C][n_bins], finite, >= 0, not all zero.  n_bins = 0 restores the
 *            uniform draw (weights ignored).
 * Changing n_bins reallocates the tables and clears the counts; the call waits for
 * the env's stream (not capturable).  Counts, per (clip, bin): `starts`, episodes begun
 * there by a reset (im_env_reset_all included); `failures`, early terminations
 * (IM_FLAG_TERMINATED) whose time fell there, bin = min(floor(t / (span / n_bins)),
 * n_bins - 1).  Integer atomics, so the counts do not depend on execution order.
 * im_env_get_reset_stats copies them to DEVICE arrays of C * n_bins uint32 (either may
 * be NULL), stream-ordered, and zeroes them afterwards if clear != 0;
 * IM_ERR_UNSUPPORTED while n_bins == 0. */
im_status im_env_set_reset_bins(im_env *e, int32_t n_bins, const float *weights);
/* The adaptive part, on the device and stream-ordered (capturable): the weight of (clip, bin) i becomes
 * fl32(fl32(failures_i) + floor_weight) -- bins where more episodes ended early are started more
 * often, floor_weight > 0 keeps every bin reachable -- and the cumulative table is rebuilt from
 * those weights by the rule above; clear != 0 zeroes both counts afterwards.  IM_ERR_UNSUPPORTED
 * while n_bins == 0 or with more than 12288 (clip, bin) pairs. */
im_status im_env_adapt_reset_bins(im_env *e, float floor_weight, int32_t clear);
im_status im_env_get_reset_stats(im_env *e, uint32_t *starts, uint32_t *failures, int32_t clear);

/* ---- policy ---------------------------------------------------------------
 * Multi-layer perceptron h_{l+1} = relu(W_l h_l + b_l), last layer linear,
 * giving the mean of a Gaussian with fixed standard deviation sigma (paper
 * Figure 2 `policy(obs)`; Table 4 initial log-std).  action = mean + sigma z
 * with z standard normal from Philox counter (env id, step, 1, block) and
 * Box-Muller: block i feeds z[4i..4i+3].
 *   dims    HOST [n_layers + 1]: input width, hidden widths, action width
 *   W       HOST [n_layers] pointers, W[l] is [dims[l+1]][dims[l]] row-major,
 *           float (dtype 0) or bf16 bit patterns as uint16 (dtype 1)
 *   b       HOST [n_layers] pointers to float [dims[l+1]]
 * dtype 0 runs fp32 SIMT kernels.  dtype 1 runs the tensor-core path: bf16
 * operands (observations and hidden activations are rounded to bf16), fp32
 * accumulation; it needs n_layers >= 2, hidden widths that are multiples of 64 and an action
 * width of at most 80. */
typedef struct {
    int32_t n_layers;
    int32_t dims[IM_MAX_LAYERS + 1];
    int32_t dtype;
    float sigma;
    uint64_t seed;
    uint32_t env_id_base;
    int32_t max_batch;       /* largest n a forward call will pass; sizes the activation buffers */
    int32_t impl;            /* 0: default for dtype; 1: force the SIMT kernels (debug cross-check);    */
                             /* 2: tensor path with CTA-pair GEMMs even for small batches (tests)         */
} im_policy_config;

im_status im_load_policy(const im_policy_config *cfg, const void *const *W, const float *const *b,
                         void *cuda_stream, im_policy **out);
void im_destroy_policy(im_policy *p);

/* One standard deviation per action dimension, sigma_i = exp(log_std[i]) (the learnable,
 * state-independent "policy log std" of the paper's hyper-parameter table): afterwards
 * action_i = mean_i + sigma_i z_i and logp = -0.5 sum z^2 - sum_i log_std[i] - (A/2) ln 2 pi.
 *   log_std  DEVICE [A]; copied (stream-ordered) into the policy, so an optimiser can hand
 *            over its updated parameter between rollouts without touching the host.
 *            NULL returns to the scalar sigma of the configuration (waits for the stream).
 * The first call allocates the A floats. */
im_status im_policy_set_log_std(im_policy *p, const float *log_std);

/*   obs        DEVICE [n][ld_obs] float, ld_obs >= dims[0], multiple of 4, 16-byte aligned
 *   mean_out   DEVICE [n][A]     action_out DEVICE [n][A] or NULL     logp_out DEVICE [n] or NULL
 *              (mean_out and action_out 16-byte aligned on the tensor-core path)
 * logp = -0.5 sum z^2 - A ln sigma - (A/2) ln 2 pi.
 * action_out == NULL (logp_out must then be NULL too, else IM_ERR_INVALID_ARG) evaluates the
 * mean only: no noise is drawn. */
im_status im_policy_forward(im_policy *p, uint32_t step, int32_t n, const float *obs, int32_t ld_obs,
                            float *mean_out, float *action_out, float *logp_out);

/* ---- env -> policy staging ----------------------------------------------------
 * The tensor-core policy consumes bf16 observations.  An env attached to such a
 * policy writes, besides the fp32 rows the caller asked for, the same rows
 * rounded to bf16 (nearest even) straight into the policy's input staging
 * buffer during im_env_reset_all / im_env_step, and im_policy_forward_staged
 * then runs the policy on rows [0, n) of that buffer -- the same result as
 * im_policy_forward on the fp32 rows, without the conversion pass over the
 * observations.  Requirements: tensor-core policy, same stream, policy input
 * width 24J+1, max_batch >= N, and ld_obs equal to 24J+1 rounded up to a
 * multiple of 64.  Passing NULL detaches.  While a policy is attached,
 * im_env_reset_all and im_env_step accept obs_out == NULL: only the bf16 rows
 * are written then (a policy-serving loop that never reads the fp32
 * observation saves their 4 (24J+1) bytes of stores per env). */
im_status im_env_attach_policy(im_env *e, im_policy *p);
im_status im_policy_forward_staged(im_policy *p, uint32_t step, int32_t n,
                                   float *mean_out, float *action_out, float *logp_out);

/* ---- rollout-side plumbing: value head and advantage estimation ------------------
 * (The paper's training loop, its Figure 2, stores obs, action, reward, terminated and
 * truncated per step and hands the storage to the PPO update; its hyper-parameter table
 * lists the discount factor and the GAE parameter.  The storage itself is plain device
 * memory: callers pass pointers into their [T][N] arrays to the per-step calls.)
 *
 * Value head: a critic is an im_policy (any output width, normally 1) read without
 * sampling.  im_policy_forward with action_out == NULL (and logp_out == NULL) does the
 * same thing; these two are the named form.
 *   value_out  DEVICE [n][dims[last]] (16-byte aligned on the tensor-core path)
 * im_value_forward_staged runs on the bf16 observation rows an attached environment has
 * written into the staging buffer of `src` (the actor the env is attached to; NULL: the
 * critic's own buffer).  Both must be tensor-core policies with the same input width,
 * created on the same stream; src->max_batch >= n. */
im_status im_value_forward(im_policy *critic, int32_t n, const float *obs, int32_t ld_obs, float *value_out);
im_status im_value_forward_staged(im_policy *critic, im_policy *src, int32_t n, float *value_out);

/* Generalised advantage estimation (Schulman et al. 2016) over T control steps of N envs:
 *   done_t  = flags_t != 0        (the flag bytes im_env_step writes)
 *   r'_t    = r_t + gamma V_t     if bootstrap_truncated and step t is truncated, not terminated
 *   delta_t = r'_t + gamma V_{t+1} (1 - done_t) - V_t
 *   A_t     = delta_t + gamma lambda (1 - done_t) A_{t+1},  A_T = 0        R_t = A_t + V_t
 * All arrays DEVICE, time-major with row stride ld >= N elements, env index fastest:
 *   reward [T][ld] float   value [T+1][ld] float (row T: value of the observation after the
 *   last step)   flags [T][ld] uint8   advantage, returns [T][ld] float (written; padding
 *   columns are not touched).
 * fp32 arithmetic; chunks of the horizon are folded in parallel, so results differ from the
 * plain backward recursion by rounding only.  Asynchronous on cuda_stream, allocates nothing,
 * capturable.  gamma and lambda must lie in [0, 1] (IM_ERR_INVALID_ARG otherwise). */
typedef struct {
    float gamma, lambda;
    int32_t bootstrap_truncated;
} im_gae_config;

im_status im_gae(const im_gae_config *cfg, int32_t T, int32_t N, int64_t ld, const float *reward,
                 const float *value, const uint8_t *flags, float *advantage, float *returns,
                 void *cuda_stream);

/* ---- PPO minibatch loss -------------------------------------------------------
 * (The paper's update phase, "update_policy(storage)" in its Figure 2, with the
 * coefficients of its hyper-parameter table: PPO ratio clip, value-loss and entropy
 * coefficients; the mean KL below is what its KL threshold is compared with.  This
 * call covers the part of the update between the forward and the backward GEMMs.)
 * For sample i of M and action dimension k of A (A <= 128), sigma_k = exp(log_std_k):
 *   logp_i = -1/2 sum_k ((a_ik - mu_ik)/sigma_k)^2 - sum_k log_std_k - A/2 ln 2 pi
 *   r_i    = exp(logp_i - logp_old_i),   Ahat_i = (adv_i - adv_mean) adv_rstd
 *   surr_i = -min(r_i Ahat_i, clip(r_i, 1-clip, 1+clip) Ahat_i)
 *   vl_i   = (V_i - R_i)^2, or with clip_value_loss max(vl_i, (Vold_i + clip(V_i - Vold_i, -clip, clip) - R_i)^2)
 *   L      = mean_i surr_i + value_coef mean_i vl_i - entropy_coef sum_k (log_std_k + 1/2 ln(2 pi e))
 * Inputs, all DEVICE float: mean, action, mean_old [M][A]; log_std, log_std_old [A];
 * logp_old, advantage, value, value_old (may be NULL without clip_value_loss), returns [M];
 * adv_moments [2] = (adv_mean, adv_rstd) as im_moments writes them, or NULL for (0, 1).
 * Outputs, DEVICE: d_mean [M][A] = dL/dmu, d_log_std [A], d_value [M] = dL/dV, and
 * summary [6] = {L, mean surr, mean vl, entropy, mean KL(old || new), fraction of samples
 * with |r - 1| > clip}.  fp32 arithmetic, batch sums finished in fp64 in a fixed order
 * (bit-reproducible).  workspace: DEVICE, im_ppo_workspace_bytes() bytes, 8-byte aligned,
 * contents irrelevant.  Two or three launches on cuda_stream; nothing is allocated or read on the
 * host.  When the [M] and [M][A] arrays are 16-byte aligned, whole 32-row tiles travel as bulk
 * asynchronous copies (the fast path); otherwise, and for the rows after the last full tile, rows
 * are fetched element by element.  Per-row results do not depend on the path.
 *
 * im_moments: out2 = (mean, 1 / (std + 1e-8)) of n floats, std with the n - 1 divisor
 * (advantage normalisation), accumulated in fp64; same workspace rules. */
typedef struct {
    float clip, value_coef, entropy_coef;
    int32_t clip_value_loss;
} im_ppo_config;

typedef struct {
    const float *mean, *log_std, *action, *logp_old, *mean_old, *log_std_old;
    const float *advantage, *adv_moments, *value, *value_old, *returns;
} im_ppo_batch;

size_t im_ppo_workspace_bytes(void);
im_status im_moments(const float *x, int64_t n, float *out2, void *workspace, void *cuda_stream);
im_status im_ppo_loss(const im_ppo_config *cfg, int64_t M, int32_t A, const im_ppo_batch *batch, float *d_mean,
                      float *d_log_std, float *d_value, float *summary, void *workspace, void *cuda_stream);

/* ---- optimiser step -----------------------------------------------------------
 * (Adam with bias correction as in the common deep-learning libraries; the learning
 * rate follows the mean KL against the paper's "KL threshold"; the gradient is
 * clipped by its global norm.  Learning rate and gradient scale are DEVICE scalars,
 * so a whole update runs without the host reading anything back.)
 *   g = grad * grad_scale;   m = beta1 m + (1 - beta1) g;   v = beta2 v + (1 - beta2) g^2
 *   param -= lr (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)          t = 1, 2, ...
 * im_adam_step: param, grad, m, v DEVICE float [n] (param, m, v updated in place);
 *   lr DEVICE float [1]; grad_scale DEVICE float [1] or NULL (1).  bf16_out, if not NULL,
 *   receives the new parameters rounded to bf16 (nearest even) as a [n / cols][cols] matrix
 *   with row stride ld_bf16 elements -- e.g. a layer's padded weight matrix from
 *   im_policy_layer_buffers, so the next forward uses the updated weights.
 * im_grad_scale: scale_out DEVICE float [2] <- (min(1, max_norm / (norm + 1e-6)), norm), norm
 *   the L2 norm over all n_tensors gradient tensors (HOST arrays of DEVICE pointers and
 *   sizes, at most 64 tensors); fp64 sums in a fixed order.  workspace as for im_ppo_loss.
 * im_adaptive_lr: lr <- max(lr / 1.5, lr_min) if kl > 2 kl_target; min(1.5 lr, lr_max) if
 *   0 < kl < kl_target / 2; unchanged otherwise.  lr, kl DEVICE float [1] (kl is
 *   summary[4] of im_ppo_loss).
 * All asynchronous on cuda_stream, no allocation, capturable.
 * im_policy_layer_buffers: the DEVICE weight matrix of a layer ([dims[l+1]][dims[l]] with
 *   row stride *ld elements; bf16 on the tensor-core path and for dtype 1, else float) and
 *   its float bias, for in-place updates by an optimiser running on the policy's stream. */
typedef struct {
    float beta1, beta2, eps;
} im_adam_config;

im_status im_adam_step(const im_adam_config *cfg, int32_t t, int64_t n, float *param, const float *grad, float *m,
                       float *v, const float *lr, const float *grad_scale, uint16_t *bf16_out, int32_t cols,
                       int32_t ld_bf16, void *cuda_stream);
im_status im_grad_scale(int32_t n_tensors, const float *const *grads, const int64_t *sizes, float max_norm,
                        float *scale_out, void *workspace, void *cuda_stream);
im_status im_adaptive_lr(float *lr, const float *kl, float kl_target, float lr_min, float lr_max, void *cuda_stream);
im_status im_policy_layer_buffers(im_policy *p, int32_t layer, void **W, int32_t *ld, float **bias);

/* ---- backward-pass building blocks ---------------------------------------------
 * (The GEMMs and glue kernels of the update's backward pass; the paper runs this
 * phase through torch.compile.)  With H_l = relu(H_{l-1} W_l^T + b_l) and dZ_l the
 * gradient at layer l's pre-activation:  dW_l = dZ_l^T H_{l-1},  db_l = column sums of
 * dZ_l,  dH_{l-1} = dZ_l W_l,  dZ_{l-1} = dH_{l-1} masked by H_{l-1} > 0.
 * All matrices DEVICE, row-major bf16 bit patterns (uint16) unless stated; ld* are row
 * strides in elements.  Everything is asynchronous on cuda_stream and allocates nothing.
 *
 * im_gemm_bf16: C[M][N] = act(A[M][K] B[N][K]^T + bias[N]) on the tcgen05 kernels of the
 *   forward path (fp32 accumulation, output rounded to bf16; relu != 0: act = max(., 0)).
 *   N and K multiples of 64; lda, ldb, ldc multiples of 8; all pointers 16-byte aligned;
 *   bias float [N] (pass zeros for none); status DEVICE uint32 [1] receives
 *   IM_DEV_WAIT_TIMEOUT if a bounded wait inside the kernel runs out.
 * im_gemm_bf16_tn: the transposed product of two row-major matrices without transposing either:
 *   C_s[Mo][No] = sum over rows r of slice s of A[r][0..Mo) (x) B[r][0..No), for `slices` equal
 *   ranges of the R rows (R a multiple of 64 * slices), partial results stacked c_pitch rows apart
 *   (c_pitch >= Mo, a multiple of 128; rows Mo..c_pitch of a slice are written as zeros).  The
 *   tensor cores read both operands M/N-major.  No a multiple of 64.  The slices split the long
 *   batch-dimension contraction of dW so that it fills the machine; im_sum_slices_bf16_to_f32 then adds
 *   them (in order, fp32) into a dense float matrix: out[r][c] = sum_s in[s * slice_stride + r * ld_in + c].
 * im_gemm_bf16_f32out: C[M][N] float, dense = A[M][K] B[N][K]^T + bias, N <= 80; B and bias
 *   must hold ceil(N / 16) * 16 rows / floats (the extra ones zero).
 * im_transpose_bf16: out[c][r] = in[r][c] for a [rows][cols] matrix.
 * im_gemm_bf16_dgrad: the backward product through a linear layer fused with what follows it,
 *   dH[r][c] = (H[r][c] > 0) * sum_k dZ[r][k] Wt[c][k]  as bf16 [M][N] (Wt = the layer's weights transposed,
 *   bf16 [N][K]; H = the forward activations the ReLU produced, bf16 [M][N], or NULL for no mask), and
 *   colsum_partial[(r / 32) * ld_partial + c] = the sum of the fp32 values of dH over the 32-row block
 *   (float [M / 32][ld_partial], or NULL); summing those rows with im_colsum_f32 gives the bias gradient
 *   of the layer below.  M a multiple of 32; the product has no bias; the other rules of im_gemm_bf16 apply.
 * im_f32_to_bf16_padded: out[r][c] = bf16(in[r][c]) for c < cols, 0 for cols <= c < ld_out.
 * im_gather_rows_f32: out[i][0..cols) = in[idx[i]][0..cols) for i < rows (shuffled minibatches); idx
 *   DEVICE int32 [rows] with values in [0, n_src); out is float [rows][ld_out], or with to_bf16 != 0
 *   bf16 [rows][ld_out] with columns cols..ld_out written as zeros.  An index out of range is clamped
 *   and sets IM_DEV_BAD_STATE in *status (DEVICE uint32).
 * im_copy_f32: dst[0..n) = src[0..n), DEVICE to DEVICE on the stream (e.g. a trained bias vector
 *   into the buffer im_policy_layer_buffers returns).
 * im_colsum_f32: out[c] = sum_r x[r][c], float [cols]; rows are summed in
 *   fp32 within slices of 256 rows and the slices in a fixed order in fp64 (bit-reproducible);
 *   workspace DEVICE, at least ceil(rows / 256) * cols * 4 bytes. */
im_status im_gemm_bf16(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, uint16_t *C, int64_t ldc,
                       int32_t M, int32_t N, int32_t K, const float *bias, int32_t relu, uint32_t *status,
                       void *cuda_stream);
im_status im_gemm_bf16_dgrad(const uint16_t *dZ, int64_t ld_dz, const uint16_t *Wt, int64_t ld_wt, uint16_t *dH, int64_t ld_dh,
                             int32_t M, int32_t N, int32_t K, const uint16_t *H, int64_t ld_h, float *colsum_partial,
                             int32_t ld_partial, uint32_t *status, void *cuda_stream);
im_status im_gemm_bf16_tn(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, uint16_t *C, int64_t ldc,
                          int32_t R, int32_t Mo, int32_t No, int32_t slices, int32_t c_pitch, uint32_t *status,
                          void *cuda_stream);
im_status im_sum_slices_bf16_to_f32(const uint16_t *in, int64_t slice_stride, int64_t ld_in, int32_t slices, int32_t rows,
                                    int32_t cols, float *out, void *cuda_stream);
im_status im_gemm_bf16_f32out(const uint16_t *A, int64_t lda, const uint16_t *B, int64_t ldb, float *C, int32_t M,
                              int32_t N, int32_t K, const float *bias, uint32_t *status, void *cuda_stream);
im_status im_transpose_bf16(const uint16_t *in, int64_t ld_in, int32_t rows, int32_t cols, uint16_t *out, int64_t ld_out,
                            void *cuda_stream);
im_status im_f32_to_bf16_padded(const float *in, int64_t ld_in, int32_t rows, int32_t cols, uint16_t *out, int32_t ld_out,
                                void *cuda_stream);
im_status im_gather_rows_f32(const float *in, int64_t ld_in, const int32_t *idx, int64_t n_src, int32_t rows, int32_t cols,
                             void *out, int32_t ld_out, int32_t to_bf16, uint32_t *status, void *cuda_stream);
im_status im_copy_f32(float *dst, const float *src, int64_t n, void *cuda_stream);
im_status im_colsum_f32(const float *x, int64_t ld, int64_t rows, int32_t cols, float *out, void *workspace,
                        size_t workspace_bytes, void *cuda_stream);

/* ---- the update phase as handles ------------------------------------------------
 * (The paper's training loop, Figure 2: `update_policy(storage)` after every rollout; Section 4.1 runs
 * the PPO update as one compiled unit, and Section 4.2 keeps the host out of it.  The hyper-parameter
 * table names what im_ppo_update_config holds: learning rate, ratio clip, value-loss and entropy
 * coefficients, KL threshold, gradient clipping.)
 *
 * im_trainer: one MLP in training form -- fp32 master weights and Adam moments, bf16 working copies of the
 * weights and of their transposes (padded to the 64-column tiles of the tensor-core kernels), one bf16
 * activation buffer per layer, gradient buffers, and the scratch of the backward pass -- for minibatches of up
 * to max_rows rows.  Hidden widths must be multiples of 64, the output width at most 80, max_rows a multiple
 * of 64.  W, b: HOST arrays of n_layers HOST pointers (W[l] float [dims[l+1]][dims[l]], b[l] float
 * [dims[l+1]]), copied.  All later calls only enqueue kernels on cuda_stream: no host read, no allocation,
 * capturable.
 *   im_trainer_forward   runs the net on the first M rows of the input buffer (IM_TRAINER_H of layer 0: bf16
 *                        [max_rows][ld], filled by the caller, columns beyond dims[0] zero) and leaves the fp32
 *                        outputs in IM_TRAINER_OUT; every layer's activation is kept for the backward pass.
 *   im_trainer_backward  d_out DEVICE float [M][dims[last]] = dL/d(outputs) of that forward; M a multiple of 64.
 *                        Fills the gradients IM_TRAINER_DW / IM_TRAINER_DB of every layer:
 *                        dW_l = dZ_l^T H_{l-1} (im_gemm_bf16_tn over row slices + im_sum_slices_bf16_to_f32),
 *                        dZ_{l-1} = (H_{l-1} > 0) (dZ_l W_l) and its column sums (im_gemm_bf16_dgrad + im_colsum_f32).
 *   im_trainer_step      one Adam step on every tensor (im_adam_step; lr and grad_scale DEVICE float [1],
 *                        grad_scale may be NULL); the bf16 copies and their transposes follow.
 *   im_trainer_push_to_policy  writes the current weights and biases into a loaded im_policy of the same
 *                        shape and stream, so the next rollout acts with the trained network.
 *   im_trainer_tensor    DEVICE address and shape of one of the trainer's arrays (IM_TRAINER_*; `layer` is
 *                        ignored for OUT and STATUS).  *dtype: IM_DTYPE_F32 / IM_DTYPE_BF16 / IM_DTYPE_U32.  The
 *                        arrays stay owned by the trainer; a caller may read them, and may write the input rows.
 *   im_trainer_set_step_count  sets the Adam step counter (bias correction) -- 0 restarts the optimiser.
 *   im_trainer_dw_slices the number of row slices the dW product of a layer with Np x Kp (padded) weights takes
 *                        on M rows: the power of two that minimises a small time model (waves of output tiles on
 *                        the SMs x rows per slice, plus the pass that adds the partial products).  Host only. */
typedef struct im_trainer im_trainer;
#define IM_TRAINER_W        0   /* float [dims[l+1]][dims[l]]                      */
#define IM_TRAINER_B        1   /* float [dims[l+1]] (buffer padded to 64 floats)   */
#define IM_TRAINER_W_BF16   2   /* bf16 [Np][Kp], zero padded                       */
#define IM_TRAINER_WT_BF16  3   /* bf16 [Kp][Np], its transpose                     */
#define IM_TRAINER_M_W      4
#define IM_TRAINER_V_W      5
#define IM_TRAINER_M_B      6
#define IM_TRAINER_V_B      7
#define IM_TRAINER_DW       8
#define IM_TRAINER_DB       9
#define IM_TRAINER_H       10   /* bf16 [max_rows][Kp]: input of layer l (layer 0: the observations) */
#define IM_TRAINER_OUT     11   /* float [max_rows][dims[last]]                     */
#define IM_TRAINER_STATUS  12   /* uint32 [1]: sticky device status word            */
#define IM_DTYPE_F32  0
#define IM_DTYPE_BF16 1
#define IM_DTYPE_U32  2
im_status im_trainer_create(int32_t n_layers, const int32_t *dims, const float *const *W, const float *const *b,
                            int32_t max_rows, void *cuda_stream, im_trainer **out);
void im_trainer_destroy(im_trainer *tr);
im_status im_trainer_forward(im_trainer *tr, int32_t M);
im_status im_trainer_backward(im_trainer *tr, const float *d_out, int32_t M);
im_status im_trainer_step(im_trainer *tr, const im_adam_config *adam, const float *lr, const float *grad_scale);
im_status im_trainer_push_to_policy(im_trainer *tr, im_policy *p);
im_status im_trainer_tensor(im_trainer *tr, int32_t which, int32_t layer, void **ptr, int64_t *rows, int64_t *cols,
                            int64_t *ld, int32_t *dtype);
im_status im_trainer_set_step_count(im_trainer *tr, int32_t t);
int32_t im_trainer_dw_slices(int32_t Np, int32_t Kp, int64_t M, int32_t max_split, int32_t any_rows);

/* im_ppo_updater: one actor, one critic (a trainer with a single output) and the learnable per-dimension
 * log-std, sharing a stream and max_rows.  log_std: HOST float [A], the initial value (also the first
 * "old" log-std).
 *   im_ppo_update  one minibatch update on M rows (a multiple of 64): forward of both nets on their input
 *     rows, advantage moments (if normalize_advantage), im_ppo_loss, both backward passes, im_grad_scale
 *     over every gradient tensor (global-norm clip at max_grad_norm), Adam on every tensor and on the
 *     log-std, im_adaptive_lr from the mean KL.  The minibatch's observations must already sit in both
 *     trainers' input rows.  mb: DEVICE float arrays -- action, mean_old [M][A]; logp_old, advantage,
 *     value_old (needed with clip_value_loss), returns [M]; log_std_old [A] or NULL for the updater's own copy.
 *   im_ppo_update_rollout  the whole update phase over a collected rollout: `epochs` passes over
 *     `n_minibatches` blocks of the T * N samples (row t * N + e of the time-major arrays of `view`;
 *     T * N / n_minibatches must be a multiple of 64 within max_rows).  perm NULL: contiguous blocks, the
 *     observations converted into both nets' input rows by im_f32_to_bf16_padded, everything else read in
 *     place.  perm: DEVICE int32 [epochs][T * N], a permutation of the sample indices per epoch: every array
 *     of a block is gathered by im_gather_rows_f32 (the first shuffled call of a given size allocates the
 *     gather buffers; make it outside a capture).
 *   im_ppo_updater_tensor  DEVICE address of a state array (IM_PPO_*): the log-std and its Adam moments [A],
 *     the frozen behaviour log-std [A], the learning rate [1], (clip factor, gradient norm) [2], the loss
 *     summary of the last minibatch [6] as im_ppo_loss writes it. */
typedef struct im_ppo_updater im_ppo_updater;
typedef struct {
    float lr;                     /* initial learning rate; adapted between lr_min and lr_max            */
    float clip, value_coef, entropy_coef;
    int32_t clip_value_loss;
    float max_grad_norm;
    float kl_target, lr_min, lr_max;
    int32_t normalize_advantage;
    im_adam_config adam;
} im_ppo_update_config;
typedef struct {
    const float *action, *mean_old, *log_std_old, *logp_old, *advantage, *value_old, *returns;
} im_ppo_minibatch;
typedef struct {
    int32_t T, N, A, ld_obs;
    const float *obs;             /* [T * N][ld_obs]                                                      */
    const float *action, *mean;   /* [T * N][A]: the behaviour policy's actions and means                 */
    const float *logp, *advantage, *returns, *value;   /* [T * N]                                          */
} im_rollout_view;
#define IM_PPO_LOG_STD      0
#define IM_PPO_LOG_STD_OLD  1
#define IM_PPO_M_LOG_STD    2
#define IM_PPO_V_LOG_STD    3
#define IM_PPO_LR           4
#define IM_PPO_GRAD_SCALE   5
#define IM_PPO_SUMMARY      6
im_status im_ppo_updater_create(im_trainer *actor, im_trainer *critic, const float *log_std,
                                const im_ppo_update_config *cfg, im_ppo_updater **out);
void im_ppo_updater_destroy(im_ppo_updater *u);
im_status im_ppo_update(im_ppo_updater *u, int32_t M, const im_ppo_minibatch *mb);
im_status im_ppo_update_rollout(im_ppo_updater *u, const im_rollout_view *view, int32_t epochs, int32_t n_minibatches,
                                const int32_t *perm);
im_status im_ppo_updater_tensor(im_ppo_updater *u, int32_t which, float **ptr, int64_t *n);
im_status im_ppo_updater_set_step_count(im_ppo_updater *u, int32_t t);

/* ---- whole step from host buffers ------------------------------------------
 * Convenience for callers whose simulator lives in host memory: copies one
 * step's body states HOST -> device, runs im_policy_forward on the current
 * observation and then im_env_step, and copies action, reward and flags back,
 * then waits until everything has arrived.  The upload runs beside the policy
 * forward and the actions travel back beside the env step (two internal copy
 * streams); the kernels run on the env's stream.  From 49152 envs on, the upload
 * is cut into four env ranges and each range's env kernel starts when its
 * columns have arrived.  The first call allocates the
 * device staging buffers and the copy streams (so it is not capturable).  Call
 * im_env_reset_all_host first.  sim_host is [13J][N] (pos rows, quat rows,
 * linvel rows, angvel rows); pinned memory gives the copies full speed.
 *   action_host HOST [N][A]   reward_host HOST [N]   flags_host HOST [N] */
im_status im_env_reset_all_host(im_env *e, uint32_t step);
im_status im_step_host(im_env *e, im_policy *p, uint32_t step, const float *sim_host,
                       float *action_host, float *reward_host, uint8_t *flags_host);

/* Reads the sticky device status word of an env or a policy handle (exactly
 * one of them non-NULL).  This is the only call besides the *_host ones that
 * waits for the stream. */
im_status im_poll_device_status(im_env *e, im_policy *p, uint32_t *out);

/* Number of kernel launches the library has enqueued since it was loaded. */
uint64_t im_launch_count(void);

/* ---- diagnostics: the env kernel's approximations in isolation -----------------
 * (No counterpart in the paper.)  The env kernel evaluates the interpolation of step (a) and the
 * geodesic angles of the reward without inverse trigonometry where the angles are small: the squared
 * rotation angle from an arcsine series on sin^2(theta/2) (up to sin^2 = 0.15, atan2 beyond), and
 * slerp as q0 exp(alpha h) with cos and sin(x)/x from Taylor polynomials (up to |h| = 0.5, sincos
 * beyond).  This call runs those two device functions on n items so that a test can sweep them across
 * both branches against closed forms.
 *   op = IM_DEBUG_ANGLE_SQ   in DEVICE [n][4] quaternions of any positive norm -> out DEVICE [n] angle^2
 *   op = IM_DEBUG_SLERP      in DEVICE [n][8] = q0 (w,x,y,z), h (3), alpha       -> out DEVICE [n][7] =
 *                            q0 exp(alpha h) (4) and 2 h (the joint velocity at 1 frame per second) */
/* im_debug_set_wait: every wait inside the tensor-core GEMM kernels and the bulk-copy PPO loss kernel (on an
 * mbarrier that a copy or an MMA completes) is bounded: when limit_ns (2 s by default) runs out the kernel sets
 * IM_DEV_WAIT_TIMEOUT in the handle's status word (the PPO loss: a NaN summary), stops issuing, lets what is in
 * flight land, frees its tensor memory and returns, so the context stays usable.  This call sets the limit for
 * the current device and, with skip_loads != 0, makes the copy-issuing threads of the single-CTA GEMM kernels
 * and of the PPO loss kernel issue nothing -- the only way to see a wait run out without a fault: nothing is in
 * flight, the consumers give up after limit_ns.  For tests of the failure path; synchronises the device. */
im_status im_debug_set_wait(uint64_t limit_ns, int32_t skip_loads);
#define IM_DEBUG_ANGLE_SQ 0
#define IM_DEBUG_SLERP    1
im_status im_debug_math(int32_t op, int32_t n, const float *in, float *out, void *cuda_stream);

/* ---- allocation-free policy forward ------------------------------------------
 * (The paper has no counterpart of this call; it exists for deployment.)
 * For callers that may not allocate device memory when they need an action: a
 * control loop that cannot afford an allocation's device-wide stall, a process
 * whose memory was all handed out at start-up, a plug-in living inside another
 * program's allocator.  The fp32 policy chain of im_policy_forward (same
 * kernels, same results) runs on weights the CALLER keeps in device memory,
 * and the only memory the library adds -- the hidden activations -- is a fixed
 * array inside the library image, IM_NOALLOC_SCRATCH_BYTES per GPU that loads
 * the library, held until the process exits.  The call allocates and frees
 * nothing and needs no handle.
 *   dims        HOST [n_layers + 1]
 *   W, b        HOST arrays of n_layers DEVICE pointers: W[l] float [dims[l+1]][dims[l]], b[l] float [dims[l+1]]
 *   obs         DEVICE [n][ld_obs] float       mean_out, action_out DEVICE [n][A]    logp_out DEVICE [n] or NULL
 *   cuda_stream cudaStream_t the work is enqueued on
 * Limits: n <= IM_NOALLOC_MAX_BATCH and hidden widths <= IM_NOALLOC_MAX_WIDTH; beyond them the call
 * returns IM_ERR_UNSUPPORTED and does nothing.
 * The first call on each device looks up the array's device address.  The look-up itself requests no
 * memory, but under CUDA's lazy module loading it can be the moment the driver loads this library's
 * device code on that GPU and backs the array, which may take a while: make the first call at
 * start-up, off the latency-critical path, outside any stream capture, with the device that will
 * run it current.  Later calls only launch kernels.
 * All calls on a device share the one array: it keeps whatever the last call left (nothing in it
 * needs clearing, every value read is written first by the same call), and two calls whose work
 * overlaps on the GPU (for example on different streams) race on it.  Run them on one stream. */
#define IM_NOALLOC_MAX_BATCH  1024
#define IM_NOALLOC_MAX_WIDTH  1024
#define IM_NOALLOC_SCRATCH_BYTES (2u * IM_NOALLOC_MAX_BATCH * IM_NOALLOC_MAX_WIDTH * 4u)   /* 8 MiB */
im_status im_policy_forward_noalloc(int32_t n_layers, const int32_t *dims, const float *const *W,
                                    const float *const *b, float sigma, uint64_t seed, uint32_t env_id_base,
                                    uint32_t step, int32_t n, const float *obs, int32_t ld_obs,
                                    float *mean_out, float *action_out, float *logp_out, void *cuda_stream);

#if defined(__GNUC__)
#pragma GCC visibility pop
#endif
#ifdef __cplusplus
}
#endif
#endif /* IM_H_ */
