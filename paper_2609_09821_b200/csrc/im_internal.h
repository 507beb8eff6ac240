// Host-side definitions shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>
#include <mutex>
#include <vector>

#include "../../include/im.h"

namespace im {

extern std::atomic<uint64_t> g_launches;   // kernels enqueued by this library

// Per-clip metadata, one 16-byte record so a thread fetches it with one load.
struct ClipMeta {
    int32_t K;        // keyframes
    float fps;
    float dur;        // (K-1)/fps, fp32 division
    int32_t start;    // first row of the clip in the packed keyframe table
};

// One link of a kinematic chain as the env kernel reads it from shared memory (two 16-byte words).
struct ChainLink {
    float off[3];        // origin of the body in its parent's frame
    float mass_frac;     // m_b / sum m
    int32_t b;           // body index
    int32_t flags;       // LINK_OWN: this chain scores the body and writes its observation entries; LINK_EE: end effector
    int32_t pad[2];
};
constexpr int LINK_OWN = 1, LINK_EE = 2;
constexpr int IM_MAX_LINKS = 288;          // sum of chain lengths for any tree of up to 32 bodies (<= 16 x 17)

// Per-clip record of looped playback (im_clips_set_cyclic): the root displacement of one cycle and the flag.
struct ClipLoop {
    float sx, sy, sz;
    int32_t on;
};

// Skeleton as the kernels see it (passed by value inside the kernel parameters).
// Kinematic chains: one root-to-leaf path per leaf.  A body shared by several paths is owned by the first of
// them; within a path the owned bodies are a suffix starting at chain_first_own.  The links of all chains lie
// in one device array, chain c at [link_start[c], link_start[c] + chain_len[c]).
struct SkelDev {
    int32_t J;
    uint32_t ee_mask;
    int32_t n_chains;
    int32_t n_links;
    uint8_t chain_len[IM_MAX_BODIES];
    uint8_t chain_first_own[IM_MAX_BODIES];
    uint16_t link_start[IM_MAX_BODIES];
};

// One-time kernel set-up (shared-memory opt-in, SM count) is per device: run `fn` once for the current device.
constexpr int kMaxDevices = 64;
struct DeviceOnce {
    std::mutex m;
    bool done[kMaxDevices] = {};
    template <typename F> cudaError_t run(F fn)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(m);
        if (done[dev]) return cudaSuccess;
        e = fn();
        done[dev] = e == cudaSuccess;
        return e;
    }
};
// Number of SMs of the current device (cached per device).
int device_sm_count();

struct EnvKernelParams {
    SkelDev sk;
    // clip library
    const float4 *frames;     // [rows][2+2J] float4, see clip_table_kernel
    const float4 *links;      // [n_links][2]: the chains' ChainLink records
    const ClipMeta *meta;     // [C]
    int32_t C;
    int32_t n_rows;           // keyframes of all clips together (rows of `frames`)
    // configuration
    int32_t N;
    uint32_t env_id_base;
    float dt;
    uint32_t seed_lo, seed_hi;
    im_reward_config reward;
    int32_t ld_obs;
    int32_t write_back;
    int32_t grace_steps;
    float reset_noise_std;
    int32_t n_bins;                          // adaptive initialisation: phase bins per clip (0: uniform draw)
    const unsigned long long *reset_cdf;     // [C * n_bins] exclusive upper thresholds in [0, 2^32]
    uint32_t *stat_starts, *stat_failures;   // [C * n_bins]
    // extended observation (0 / null: the 24J+1 layout)
    int32_t n_future;                        // reference frames ahead whose end-effector targets are observed (>= 1)
    int32_t act_dim;                         // previous-action entries
    const float *prev_action;                // [N][ld_action]
    int32_t ld_action;
    unsigned long long *summary;             // [4] training summaries (null: none)
    const ClipLoop *loops;                   // [C] looped clips (null: no clip of the library loops)
    int32_t *cycle;                          // per-env cycle count on a looped clip
    uint32_t step;
    // per-env state
    int32_t *clip_id;
    float *t;
    int32_t *ep_len;
    // per-step I/O
    float *pos, *quat, *lin, *ang;
    long long stride;                        // component rows: floats between two rows
    int32_t aos;                             // non-zero: simulator records read in place, described by the two arrays below
    long long aos_env_stride[4];             // pos, quat, linvel, angvel: floats between two envs
    int32_t aos_body_stride[4];              //                            floats between two bodies
    float *obs;
    uint16_t *obs_bf16;       // optional bf16 copy of the observation rows (same row stride), or null
    float *reward_out;
    uint8_t *flags_out;
    float *terms_out;
    uint32_t *status;
};

}  // namespace im

struct im_skeleton {
    im::SkelDev dev;
    int32_t n_ee;
    im::ChainLink links[im::IM_MAX_LINKS];
};

struct im_clips {
    int32_t C, J;
    int64_t rows;
    float4 *d_frames;
    im::ClipMeta *d_meta;
    std::vector<im::ClipMeta> meta;
    std::vector<im::ClipLoop> loops;       // root displacement per cycle; `on` set by im_clips_set_cyclic
    im::ClipLoop *d_loops;
    bool any_loop;
    float min_dur;
    int device;
};

constexpr int kHostChunks = 4;             // env ranges the host-buffer step uploads and launches separately

struct im_env {
    const im_skeleton *skel;
    const im_clips *clips;
    im_env_config cfg;
    cudaStream_t stream;
    int32_t *d_clip_id;
    float *d_t;
    int32_t *d_ep_len;
    uint32_t *d_status;
    int32_t *d_cycle;      // cycles completed on a looped clip
    float4 *d_links;       // the skeleton's chain links on the env's device
    int D;                 // observation width: 24J + 1 plus the extension columns
    size_t smem_bytes;
    uint16_t *d_obs_bf16;  // attached policy's bf16 input rows (null when detached)
    int32_t n_bins;        // adaptive initialisation (0: off)
    unsigned long long *d_reset_cdf;
    uint32_t *d_stat_starts, *d_stat_failures;
    int32_t n_future, act_dim, ld_action;   // extended observation (im_env_set_obs_extension); D is the extended width
    const float *prev_action;
    unsigned long long *d_summary;          // caller-owned accumulator of im_env_set_summary (null: none)
    // staging for the *_host entry points (allocated on first use)
    float *d_aos_sim;      // component rows gathered from array-of-structures inputs (allocated on first use)
    float *d_sim, *d_obs, *d_reward, *d_mean, *d_action;
    uint8_t *d_flags;
    int staged_A;
    cudaStream_t h2d_stream, d2h_stream;   // copies of the host-buffer step run beside the kernels
    cudaEvent_t ev_h2d[4], ev_policy;      // one upload event per env range of the host-buffer step
};

// Launchers implemented in the kernel translation units.
namespace im {
size_t env_kernel_smem_bytes(int J, int n_chains, int n_links, int extra_cols);
// clip table rows from the caller's keyframes (device copies of the host arrays); last[r] marks a clip's final frame
cudaError_t launch_clip_table(const float *root_pos, const float *local_quat, const uint8_t *last, int64_t rows, int J,
                              float4 *frames, cudaStream_t stream);
inline int clip_row_stride(int J) { return 2 + 2 * J; }
cudaError_t env_kernel_prepare(size_t smem);
cudaError_t launch_env_kernel(const EnvKernelParams &p, bool reset_all, size_t smem, cudaStream_t stream);
cudaError_t launch_debug_math(int op, int n, const float *in, float *out, cudaStream_t stream);
// simulator-native (array of structures) body states <-> component rows [13 J][stride]
cudaError_t aos_adapter_prepare();
// reset-bin weights from the failure counts (rollout.cu); n <= 12288 entries
cudaError_t launch_adapt_reset_cdf(uint32_t *starts, uint32_t *failures, int n, float floor_weight, int clear,
                                   unsigned long long *cdf, cudaStream_t stream);
cudaError_t launch_aos_gather(const im_body_state_aos &sim, int J, int N, float *soa, long long stride, cudaStream_t stream);
cudaError_t launch_aos_scatter_reset(const im_body_state_aos &sim, int J, int N, const float *soa, long long stride,
                                     const uint8_t *flags, cudaStream_t stream);
}  // namespace im
