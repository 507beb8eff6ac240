// C-ABI entry points: validation, uploads, handle management, kernel launches.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "im_internal.h"
#include "mlp.h"

namespace im {
std::atomic<uint64_t> g_launches{0};

int device_sm_count()
{
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        int cc_major = 0;
        cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (cc_major != 10) n = -1;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n > 0 ? n : 0;
}
}

using namespace im;

#define IM_CUDA(call)                                  \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return IM_ERR_CUDA;    \
    } while (0)

extern "C" {

const char *im_status_string(im_status s)
{
    switch (s) {
    case IM_OK: return "ok";
    case IM_ERR_INVALID_ARG: return "invalid argument";
    case IM_ERR_BAD_TOPOLOGY: return "bad skeleton topology";
    case IM_ERR_BAD_QUAT: return "keyframe quaternion is not a finite unit quaternion";
    case IM_ERR_ALLOC: return "allocation failed";
    case IM_ERR_CUDA: return "CUDA call failed";
    case IM_ERR_UNSUPPORTED: return "unsupported configuration";
    default: return "unknown status";
    }
}

uint64_t im_launch_count(void) { return g_launches.load(); }

/* ------------------------------------------------------------------ skeleton */
im_status im_create_skeleton(int32_t J, const int32_t *parents, const float *offsets, const float *masses,
                             const int32_t *ee_ids, int32_t n_ee, im_skeleton **out)
{
    if (!out || !parents || !offsets) return IM_ERR_INVALID_ARG;
    if (J < 1 || J > IM_MAX_BODIES || parents[0] != -1) return IM_ERR_BAD_TOPOLOGY;
    for (int j = 1; j < J; ++j)
        if (parents[j] < 0 || parents[j] >= j) return IM_ERR_BAD_TOPOLOGY;
    if (ee_ids && n_ee > 0) {
        if (n_ee > J) return IM_ERR_INVALID_ARG;
        for (int i = 0; i < n_ee; ++i)
            if (ee_ids[i] < 0 || ee_ids[i] >= J) return IM_ERR_INVALID_ARG;
    }
    double msum = 0.0;
    for (int j = 0; j < J; ++j) {
        const double m = masses ? (double)masses[j] : 1.0;
        if (!(m > 0.0) || !std::isfinite(m)) return IM_ERR_INVALID_ARG;
        for (int c = 0; c < 3; ++c)
            if (!std::isfinite(offsets[3 * j + c])) return IM_ERR_INVALID_ARG;
        msum += m;
    }
    im_skeleton *s = new (std::nothrow) im_skeleton();
    if (!s) return IM_ERR_ALLOC;
    std::memset(s, 0, sizeof(*s));
    SkelDev &d = s->dev;
    d.J = J;
    // one root-to-leaf path per leaf; a shared body belongs to the first path that contains it
    uint8_t chain[IM_MAX_BODIES][IM_MAX_BODIES];
    {
        bool has_child[IM_MAX_BODIES] = {false}, owned[IM_MAX_BODIES] = {false};
        for (int j = 1; j < J; ++j) has_child[parents[j]] = true;
        for (int leaf = 0; leaf < J; ++leaf) {
            if (has_child[leaf]) continue;
            const int c = d.n_chains++;
            int depth = 0;
            for (int a = leaf; a > 0; a = parents[a]) ++depth;
            d.chain_len[c] = (uint8_t)(depth + 1);
            int a = leaf;
            for (int k = depth; k >= 0; --k) { chain[c][k] = (uint8_t)a; a = a > 0 ? parents[a] : 0; }
            int first = 0;
            while (first <= depth && owned[chain[c][first]]) ++first;
            d.chain_first_own[c] = (uint8_t)first;
            for (int k = first; k <= depth; ++k) owned[chain[c][k]] = true;
        }
    }
    if (ee_ids && n_ee > 0) {
        for (int i = 0; i < n_ee; ++i) d.ee_mask |= 1u << ee_ids[i];
    } else {
        uint32_t has_child = 0;
        for (int j = 1; j < J; ++j) has_child |= 1u << parents[j];
        d.ee_mask = ~has_child & (J == 32 ? 0xffffffffu : ((1u << J) - 1u));
    }
    s->n_ee = __builtin_popcount(d.ee_mask);
    // the chains' links in the order the env kernel walks them
    for (int c = 0; c < d.n_chains; ++c) {
        d.link_start[c] = (uint16_t)d.n_links;
        for (int k = 0; k < d.chain_len[c]; ++k) {
            const int b = chain[c][k];
            ChainLink &L = s->links[d.n_links++];
            for (int i = 0; i < 3; ++i) L.off[i] = b == 0 ? 0.0f : offsets[3 * b + i];
            L.mass_frac = (float)((masses ? (double)masses[b] : 1.0) / msum);
            L.b = b;
            L.flags = (k >= d.chain_first_own[c] ? LINK_OWN : 0) | (((d.ee_mask >> b) & 1u) ? LINK_EE : 0);
        }
    }
    *out = s;
    return IM_OK;
}

void im_destroy_skeleton(im_skeleton *s) { delete s; }

/* ------------------------------------------------------------------ clips */
im_status im_load_clips(const im_skeleton *skel, int32_t C, const int32_t *n_frames, const float *fps,
                        const float *root_pos, const float *local_quat, im_clips **out)
{
    if (!skel || !out || !n_frames || !fps || !root_pos || !local_quat || C < 1) return IM_ERR_INVALID_ARG;
    const int J = skel->dev.J;
    int64_t rows = 0;
    for (int c = 0; c < C; ++c) {
        if (n_frames[c] < 2 || !(fps[c] > 0.0f) || !std::isfinite(fps[c])) return IM_ERR_INVALID_ARG;
        rows += n_frames[c];
    }
    if (rows > 0x7fffffff) return IM_ERR_INVALID_ARG;
    for (int64_t i = 0; i < rows * J; ++i) {
        const float *q = local_quat + 4 * i;
        const double n2 = (double)q[0] * q[0] + (double)q[1] * q[1] + (double)q[2] * q[2] + (double)q[3] * q[3];
        if (!std::isfinite(n2) || std::fabs(std::sqrt(n2) - 1.0) > 1e-3) return IM_ERR_BAD_QUAT;
    }
    for (int64_t i = 0; i < rows * 3; ++i)
        if (!std::isfinite(root_pos[i])) return IM_ERR_INVALID_ARG;

    im_clips *cl = new (std::nothrow) im_clips();
    if (!cl) return IM_ERR_ALLOC;
    cl->C = C; cl->J = J; cl->rows = rows; cl->d_frames = nullptr; cl->d_meta = nullptr; cl->d_loops = nullptr;
    cl->any_loop = false;
    cl->meta.resize(C);
    cl->loops.resize(C);
    cl->min_dur = INFINITY;
    int32_t start = 0;
    for (int c = 0; c < C; ++c) {
        cl->meta[c] = {n_frames[c], fps[c], (float)(n_frames[c] - 1) / fps[c], start};
        cl->min_dur = std::fmin(cl->min_dur, cl->meta[c].dur);
        const float *p0 = root_pos + 3 * (int64_t)start, *p1 = root_pos + 3 * ((int64_t)start + n_frames[c] - 1);
        cl->loops[c] = {(float)((double)p1[0] - p0[0]), (float)((double)p1[1] - p0[1]), (float)((double)p1[2] - p0[2]), 0};
        start += n_frames[c];
    }
    // The table rows (see clip_table_kernel) are built on the device from copies of the caller's arrays.
    std::vector<uint8_t> last((size_t)rows, 0);
    for (int c = 0; c < C; ++c) last[(size_t)cl->meta[c].start + n_frames[c] - 1] = 1;
    const size_t RS = (size_t)clip_row_stride(J);
    float *d_root = nullptr, *d_quat = nullptr;
    uint8_t *d_last = nullptr;
    cudaGetDevice(&cl->device);
    // (one extra row of zeros so that the last frame's "next" reads stay inside the buffers)
    const size_t root_b = (size_t)(rows + 1) * 3 * sizeof(float), quat_b = (size_t)(rows + 1) * J * 4 * sizeof(float);
    bool ok = cudaMalloc(&cl->d_frames, (size_t)rows * RS * sizeof(float4)) == cudaSuccess &&
              cudaMalloc(&cl->d_meta, C * sizeof(ClipMeta)) == cudaSuccess && cudaMalloc(&cl->d_loops, C * sizeof(ClipLoop)) == cudaSuccess &&
              cudaMalloc(&d_root, root_b) == cudaSuccess &&
              cudaMalloc(&d_quat, quat_b) == cudaSuccess && cudaMalloc(&d_last, (size_t)rows) == cudaSuccess;
    im_status st = ok ? IM_OK : IM_ERR_ALLOC;
    if (ok) {
        ok = cudaMemset(d_root, 0, root_b) == cudaSuccess && cudaMemset(d_quat, 0, quat_b) == cudaSuccess &&
             cudaMemcpy(d_root, root_pos, (size_t)rows * 3 * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(d_quat, local_quat, (size_t)rows * J * 4 * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(d_last, last.data(), (size_t)rows, cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(cl->d_meta, cl->meta.data(), C * sizeof(ClipMeta), cudaMemcpyHostToDevice) == cudaSuccess &&
             cudaMemcpy(cl->d_loops, cl->loops.data(), C * sizeof(ClipLoop), cudaMemcpyHostToDevice) == cudaSuccess &&
             launch_clip_table(d_root, d_quat, d_last, rows, J, cl->d_frames, nullptr) == cudaSuccess &&
             cudaDeviceSynchronize() == cudaSuccess;
        if (!ok) st = IM_ERR_CUDA;
    }
    cudaFree(d_root); cudaFree(d_quat); cudaFree(d_last);
    if (st != IM_OK) {
        im_destroy_clips(cl);
        return st;
    }
    *out = cl;
    return IM_OK;
}

void im_destroy_clips(im_clips *c)
{
    if (!c) return;
    cudaFree(c->d_frames);
    cudaFree(c->d_meta);
    cudaFree(c->d_loops);
    delete c;
}

im_status im_clips_set_cyclic(im_clips *c, const uint8_t *flags)
{
    if (!c) return IM_ERR_INVALID_ARG;
    c->any_loop = false;
    for (int i = 0; i < c->C; ++i) {
        c->loops[i].on = flags && flags[i] ? 1 : 0;
        c->any_loop = c->any_loop || c->loops[i].on;
    }
    IM_CUDA(cudaDeviceSynchronize());           // steps in flight keep the flags they were launched with
    IM_CUDA(cudaMemcpy(c->d_loops, c->loops.data(), c->C * sizeof(ClipLoop), cudaMemcpyHostToDevice));
    return IM_OK;
}

/* ------------------------------------------------------------------ env */
static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

im_status im_env_create(const im_skeleton *skel, const im_clips *clips, const im_env_config *cfg,
                        void *cuda_stream, im_env **out)
{
    if (!skel || !clips || !cfg || !out) return IM_ERR_INVALID_ARG;
    const int J = skel->dev.J, D = 24 * J + 1;
    if (clips->J != J || cfg->n_envs < 1) return IM_ERR_INVALID_ARG;
    if (cfg->ld_obs < D || (cfg->ld_obs & 3)) return IM_ERR_INVALID_ARG;
    if (!(cfg->dt > 0.0f) || !(cfg->dt <= clips->min_dur)) return IM_ERR_INVALID_ARG;
    if (cfg->reward.mode != 0 && cfg->reward.mode != 1) return IM_ERR_INVALID_ARG;
    for (int k = 0; k < IM_N_TERMS; ++k)
        if (!std::isfinite(cfg->reward.w[k]) || !std::isfinite(cfg->reward.a[k]) || cfg->reward.w[k] < 0.0f)
            return IM_ERR_INVALID_ARG;
    if (std::isnan(cfg->reward.h_min) || std::isnan(cfg->reward.r_min)) return IM_ERR_INVALID_ARG;
    if (cfg->grace_steps < 0 || !(cfg->reset_noise_std >= 0.0f) || !std::isfinite(cfg->reset_noise_std))
        return IM_ERR_INVALID_ARG;

    im_env *e = new (std::nothrow) im_env();
    if (!e) return IM_ERR_ALLOC;
    std::memset(e, 0, sizeof(*e));
    e->skel = skel; e->clips = clips; e->cfg = *cfg; e->stream = (cudaStream_t)cuda_stream; e->D = D;
    e->smem_bytes = env_kernel_smem_bytes(J, skel->dev.n_chains, skel->dev.n_links, 0);
    e->n_future = 1;
    int dev = 0, max_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if ((int)e->smem_bytes > max_smem) { delete e; return IM_ERR_UNSUPPORTED; }
    // opt in to the device maximum once: environments of different sizes share the kernels
    if (env_kernel_prepare((size_t)max_smem) != cudaSuccess) { delete e; return IM_ERR_CUDA; }
    const size_t n = (size_t)cfg->n_envs;
    if (cudaMalloc(&e->d_clip_id, n * 4) != cudaSuccess || cudaMalloc(&e->d_t, n * 4) != cudaSuccess ||
        cudaMalloc(&e->d_ep_len, n * 4) != cudaSuccess || cudaMalloc(&e->d_status, 4) != cudaSuccess ||
        cudaMalloc(&e->d_cycle, n * 4) != cudaSuccess ||
        cudaMalloc(&e->d_links, (size_t)skel->dev.n_links * sizeof(ChainLink)) != cudaSuccess) {
        im_env_destroy(e);
        return IM_ERR_ALLOC;
    }
    if (cudaMemcpy(e->d_links, skel->links, (size_t)skel->dev.n_links * sizeof(ChainLink), cudaMemcpyHostToDevice) != cudaSuccess) {
        im_env_destroy(e);
        return IM_ERR_CUDA;
    }
    cudaMemsetAsync(e->d_clip_id, 0, n * 4, e->stream);
    cudaMemsetAsync(e->d_t, 0, n * 4, e->stream);
    cudaMemsetAsync(e->d_ep_len, 0, n * 4, e->stream);
    cudaMemsetAsync(e->d_cycle, 0, n * 4, e->stream);
    cudaMemsetAsync(e->d_status, 0, 4, e->stream);
    *out = e;
    return IM_OK;
}

void im_env_destroy(im_env *e)
{
    if (!e) return;
    cudaFree(e->d_clip_id); cudaFree(e->d_t); cudaFree(e->d_ep_len); cudaFree(e->d_status); cudaFree(e->d_links); cudaFree(e->d_cycle);
    cudaFree(e->d_sim); cudaFree(e->d_obs); cudaFree(e->d_reward); cudaFree(e->d_mean);
    cudaFree(e->d_action); cudaFree(e->d_flags);
    cudaFree(e->d_reset_cdf); cudaFree(e->d_stat_starts); cudaFree(e->d_stat_failures);
    cudaFree(e->d_aos_sim);
    if (e->h2d_stream) cudaStreamDestroy(e->h2d_stream);
    if (e->d2h_stream) cudaStreamDestroy(e->d2h_stream);
    for (int c = 0; c < kHostChunks; ++c)
        if (e->ev_h2d[c]) cudaEventDestroy(e->ev_h2d[c]);
    if (e->ev_policy) cudaEventDestroy(e->ev_policy);
    delete e;
}

static void fill_params(const im_env *e, uint32_t step, EnvKernelParams &p)
{
    std::memset(&p, 0, sizeof(p));
    p.sk = e->skel->dev;
    p.frames = e->clips->d_frames;
    p.links = e->d_links;
    p.meta = e->clips->d_meta;
    p.C = e->clips->C;
    p.n_rows = (int32_t)e->clips->rows;
    p.N = e->cfg.n_envs;
    p.env_id_base = e->cfg.env_id_base;
    p.dt = e->cfg.dt;
    p.seed_lo = (uint32_t)e->cfg.seed;
    p.seed_hi = (uint32_t)(e->cfg.seed >> 32);
    p.reward = e->cfg.reward;
    p.ld_obs = e->cfg.ld_obs;
    p.write_back = e->cfg.write_back_reset;
    p.grace_steps = e->cfg.grace_steps;
    p.reset_noise_std = e->cfg.reset_noise_std;
    p.n_bins = e->n_bins;
    p.reset_cdf = e->d_reset_cdf;
    p.stat_starts = e->d_stat_starts;
    p.stat_failures = e->d_stat_failures;
    p.n_future = e->n_future;
    p.act_dim = e->act_dim;
    p.prev_action = e->prev_action;
    p.ld_action = e->ld_action;
    p.summary = e->d_summary;
    p.loops = e->clips->any_loop ? e->clips->d_loops : nullptr;
    p.cycle = e->d_cycle;
    p.step = step;
    p.clip_id = e->d_clip_id;
    p.t = e->d_t;
    p.ep_len = e->d_ep_len;
    p.status = e->d_status;
    p.obs_bf16 = e->d_obs_bf16;
}

im_status im_env_reset_all(im_env *e, uint32_t step, float *obs_out)
{
    if (!e || !aligned16(obs_out)) return IM_ERR_INVALID_ARG;
    if (!obs_out && !e->d_obs_bf16) return IM_ERR_INVALID_ARG;      // no fp32 rows only with an attached policy's bf16 rows
    EnvKernelParams p;
    fill_params(e, step, p);
    p.obs = obs_out;
    IM_CUDA(launch_env_kernel(p, true, e->smem_bytes, e->stream));
    return IM_OK;
}

im_status im_env_step(im_env *e, uint32_t step, const im_body_state *sim, float *obs_out, float *reward_out,
                      uint8_t *flags_out, float *terms_out)
{
    if (!e || !sim || !reward_out || !flags_out) return IM_ERR_INVALID_ARG;
    if (!obs_out && !e->d_obs_bf16) return IM_ERR_INVALID_ARG;      // no fp32 rows only with an attached policy's bf16 rows
    if (!sim->pos || !sim->quat || !sim->linvel || !sim->angvel || sim->comp_stride < e->cfg.n_envs)
        return IM_ERR_INVALID_ARG;
    if (!aligned16(obs_out) || !aligned16(sim->pos) || !aligned16(sim->quat) || !aligned16(sim->linvel) ||
        !aligned16(sim->angvel) || (sim->comp_stride & 3))
        return IM_ERR_INVALID_ARG;
    if (sim->comp_stride * 4 * (int64_t)e->skel->dev.J >= (int64_t)1 << 31) return IM_ERR_UNSUPPORTED;   // the kernel indexes with 32 bits
    EnvKernelParams p;
    fill_params(e, step, p);
    p.pos = sim->pos; p.quat = sim->quat; p.lin = sim->linvel; p.ang = sim->angvel;
    p.stride = sim->comp_stride;
    p.obs = obs_out; p.reward_out = reward_out; p.flags_out = flags_out; p.terms_out = terms_out;
    IM_CUDA(launch_env_kernel(p, false, e->smem_bytes, e->stream));
    return IM_OK;
}

// The env step on envs [first, first + count) only (count a multiple of the kernel's 32-env tile unless
// it reaches the end): every per-env pointer is advanced, the Philox env ids follow.
static im_status env_step_range(im_env *e, uint32_t step, const im_body_state *sim, float *obs_out, float *reward_out,
                                uint8_t *flags_out, int first, int count)
{
    EnvKernelParams p;
    fill_params(e, step, p);
    p.N = count;
    p.env_id_base += (uint32_t)first;
    p.clip_id += first; p.t += first; p.ep_len += first; p.cycle += first;
    p.pos = sim->pos + first; p.quat = sim->quat + first; p.lin = sim->linvel + first; p.ang = sim->angvel + first;
    p.stride = sim->comp_stride;
    p.obs = obs_out + (size_t)first * e->cfg.ld_obs;
    if (p.obs_bf16) p.obs_bf16 += (size_t)first * e->cfg.ld_obs;
    p.reward_out = reward_out + first; p.flags_out = flags_out + first; p.terms_out = nullptr;
    if (p.prev_action) p.prev_action += (size_t)first * p.ld_action;
    IM_CUDA(launch_env_kernel(p, false, e->smem_bytes, e->stream));
    return IM_OK;
}

im_status im_env_step_aos(im_env *e, uint32_t step, const im_body_state_aos *sim, float *obs_out, float *reward_out,
                          uint8_t *flags_out, float *terms_out)
{
    if (!e || !sim || !reward_out || !flags_out || !aligned16(obs_out)) return IM_ERR_INVALID_ARG;
    if (!obs_out && !e->d_obs_bf16) return IM_ERR_INVALID_ARG;
    const int J = e->skel->dev.J;
    const im_aos_array *arr[4] = {&sim->pos, &sim->quat, &sim->linvel, &sim->angvel};
    for (int i = 0; i < 4; ++i) {
        const int comps = i == 1 ? 4 : 3;
        if (!arr[i]->base || arr[i]->body_stride < comps ||
            arr[i]->env_stride < (int64_t)(J - 1) * arr[i]->body_stride + comps)
            return IM_ERR_INVALID_ARG;
    }
    if (e->d_aos_sim) {
        // staging was asked for (im_env_set_aos_staging): one gather kernel turns the records into component rows,
        // the env kernel then streams those; reset envs are scattered back
        const int N = e->cfg.n_envs;
        const int64_t stride = ((int64_t)N + 3) / 4 * 4;
        IM_CUDA(launch_aos_gather(*sim, J, N, e->d_aos_sim, stride, e->stream));
        im_body_state rows = {e->d_aos_sim, e->d_aos_sim + 3 * J * stride, e->d_aos_sim + 7 * J * stride,
                              e->d_aos_sim + 10 * J * stride, stride};
        const im_status s = im_env_step(e, step, &rows, obs_out, reward_out, flags_out, terms_out);
        if (s != IM_OK) return s;
        if (e->cfg.write_back_reset)
            IM_CUDA(launch_aos_scatter_reset(*sim, J, N, e->d_aos_sim, stride, flags_out, e->stream));
        return IM_OK;
    }
    // the env kernel reads (and, for reset envs with write_back_reset, writes) the simulator's records where they are
    EnvKernelParams p;
    fill_params(e, step, p);
    p.pos = sim->pos.base; p.quat = sim->quat.base; p.lin = sim->linvel.base; p.ang = sim->angvel.base;
    p.aos = 1;
    for (int i = 0; i < 4; ++i) { p.aos_env_stride[i] = arr[i]->env_stride; p.aos_body_stride[i] = arr[i]->body_stride; }
    p.obs = obs_out; p.reward_out = reward_out; p.flags_out = flags_out; p.terms_out = terms_out;
    IM_CUDA(launch_env_kernel(p, false, e->smem_bytes, e->stream));
    return IM_OK;
}

im_status im_env_set_aos_staging(im_env *e, int32_t on)
{
    if (!e) return IM_ERR_INVALID_ARG;
    if (!on) {
        IM_CUDA(cudaStreamSynchronize(e->stream));
        cudaFree(e->d_aos_sim);
        e->d_aos_sim = nullptr;
        return IM_OK;
    }
    if (e->d_aos_sim) return IM_OK;
    const int64_t stride = ((int64_t)e->cfg.n_envs + 3) / 4 * 4;
    if (aos_adapter_prepare() != cudaSuccess) return IM_ERR_CUDA;
    if (cudaMalloc(&e->d_aos_sim, (size_t)13 * e->skel->dev.J * stride * sizeof(float)) != cudaSuccess) return IM_ERR_ALLOC;
    return IM_OK;
}

im_status im_env_attach_policy(im_env *e, im_policy *p)
{
    if (!e) return IM_ERR_INVALID_ARG;
    if (!p) { e->d_obs_bf16 = nullptr; return IM_OK; }
    if (!p->tensor_path) return IM_ERR_UNSUPPORTED;
    int32_t ld = 0;
    void *buf = tc_policy_input(p, &ld);
    if (ld != e->cfg.ld_obs || p->cfg.dims[0] != e->D || p->cfg.max_batch < e->cfg.n_envs || p->stream != e->stream)
        return IM_ERR_INVALID_ARG;
    e->d_obs_bf16 = static_cast<uint16_t *>(buf);
    return IM_OK;
}

im_status im_env_get_state(im_env *e, int32_t *clip_id, float *t, int32_t *ep_len)
{
    if (!e) return IM_ERR_INVALID_ARG;
    const size_t b = (size_t)e->cfg.n_envs * 4;
    if (clip_id) IM_CUDA(cudaMemcpyAsync(clip_id, e->d_clip_id, b, cudaMemcpyDeviceToDevice, e->stream));
    if (t) IM_CUDA(cudaMemcpyAsync(t, e->d_t, b, cudaMemcpyDeviceToDevice, e->stream));
    if (ep_len) IM_CUDA(cudaMemcpyAsync(ep_len, e->d_ep_len, b, cudaMemcpyDeviceToDevice, e->stream));
    return IM_OK;
}

im_status im_env_get_cycles(im_env *e, int32_t *cycle)
{
    if (!e || !cycle) return IM_ERR_INVALID_ARG;
    IM_CUDA(cudaMemcpyAsync(cycle, e->d_cycle, (size_t)e->cfg.n_envs * 4, cudaMemcpyDeviceToDevice, e->stream));
    return IM_OK;
}

im_status im_env_set_cycles(im_env *e, const int32_t *cycle)
{
    if (!e || !cycle) return IM_ERR_INVALID_ARG;
    IM_CUDA(cudaMemcpyAsync(e->d_cycle, cycle, (size_t)e->cfg.n_envs * 4, cudaMemcpyDeviceToDevice, e->stream));
    return IM_OK;
}

im_status im_env_set_state(im_env *e, const int32_t *clip_id, const float *t, const int32_t *ep_len)
{
    if (!e) return IM_ERR_INVALID_ARG;
    const size_t b = (size_t)e->cfg.n_envs * 4;
    if (clip_id) IM_CUDA(cudaMemcpyAsync(e->d_clip_id, clip_id, b, cudaMemcpyDeviceToDevice, e->stream));
    if (t) IM_CUDA(cudaMemcpyAsync(e->d_t, t, b, cudaMemcpyDeviceToDevice, e->stream));
    if (ep_len) IM_CUDA(cudaMemcpyAsync(e->d_ep_len, ep_len, b, cudaMemcpyDeviceToDevice, e->stream));
    return IM_OK;
}

/* ------------------------------------------------------------------ policy */
im_status im_load_policy(const im_policy_config *cfg, const void *const *W, const float *const *b,
                         void *cuda_stream, im_policy **out)
{
    if (!cfg || !W || !b || !out) return IM_ERR_INVALID_ARG;
    const int nl = cfg->n_layers;
    if (nl < 1 || nl > IM_MAX_LAYERS || cfg->max_batch < 1) return IM_ERR_INVALID_ARG;
    if (cfg->dtype != 0 && cfg->dtype != 1) return IM_ERR_INVALID_ARG;
    if (!(cfg->sigma > 0.0f) || !std::isfinite(cfg->sigma)) return IM_ERR_INVALID_ARG;
    int max_hidden = 1;
    for (int l = 0; l <= nl; ++l) {
        if (cfg->dims[l] < 1) return IM_ERR_INVALID_ARG;
        if (l > 0 && l < nl) max_hidden = cfg->dims[l] > max_hidden ? cfg->dims[l] : max_hidden;
    }
    for (int l = 0; l < nl; ++l)
        if (!W[l] || !b[l]) return IM_ERR_INVALID_ARG;

    im_policy *p = new (std::nothrow) im_policy();
    if (!p) return IM_ERR_ALLOC;
    std::memset(p, 0, sizeof(*p));
    p->cfg = *cfg; p->stream = (cudaStream_t)cuda_stream; p->nl = nl;
    p->tensor_path = cfg->dtype == 1 && cfg->impl != 1;
    if (cudaMalloc(&p->d_status, 4) != cudaSuccess) { im_destroy_policy(p); return IM_ERR_ALLOC; }
    cudaMemsetAsync(p->d_status, 0, 4, p->stream);
    if (p->tensor_path) {
        const im_status s = tc_policy_create(p, W, b);
        if (s != IM_OK) { im_destroy_policy(p); return s; }
        *out = p;
        return IM_OK;
    }
    const size_t esz = cfg->dtype == 1 ? 2 : 4;
    for (int l = 0; l < nl; ++l) {
        const size_t wn = (size_t)cfg->dims[l] * cfg->dims[l + 1];
        if (cudaMalloc(&p->d_W[l], wn * esz) != cudaSuccess ||
            cudaMalloc(&p->d_b[l], (size_t)cfg->dims[l + 1] * 4) != cudaSuccess) {
            im_destroy_policy(p);
            return IM_ERR_ALLOC;
        }
        if (cudaMemcpy(p->d_W[l], W[l], wn * esz, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(p->d_b[l], b[l], (size_t)cfg->dims[l + 1] * 4, cudaMemcpyHostToDevice) != cudaSuccess) {
            im_destroy_policy(p);
            return IM_ERR_CUDA;
        }
    }
    p->act_ld = max_hidden;
    for (int i = 0; i < 2; ++i)
        if (cudaMalloc(&p->d_act[i], (size_t)cfg->max_batch * max_hidden * 4) != cudaSuccess) {
            im_destroy_policy(p);
            return IM_ERR_ALLOC;
        }
    *out = p;
    return IM_OK;
}

void im_destroy_policy(im_policy *p)
{
    if (!p) return;
    if (p->tc) tc_policy_destroy(p);
    for (int l = 0; l < IM_MAX_LAYERS; ++l) { cudaFree(p->d_W[l]); cudaFree(p->d_b[l]); }
    cudaFree(p->d_act[0]); cudaFree(p->d_act[1]); cudaFree(p->d_status); cudaFree(p->d_log_std);
    delete p;
}

im_status im_policy_layer_buffers(im_policy *p, int32_t layer, void **W, int32_t *ld, float **bias)
{
    if (!p || !W || !ld || !bias || layer < 0 || layer >= p->nl) return IM_ERR_INVALID_ARG;
    if (p->tensor_path) {
        tc_policy_layer(p, layer, W, ld, bias);
    } else {
        *W = p->d_W[layer];
        *ld = p->cfg.dims[layer];
        *bias = p->d_b[layer];
    }
    return IM_OK;
}

im_status im_policy_set_log_std(im_policy *p, const float *log_std)
{
    if (!p) return IM_ERR_INVALID_ARG;
    const size_t bytes = (size_t)p->cfg.dims[p->nl] * sizeof(float);
    if (!log_std) {                                     // back to the scalar sigma of the configuration
        IM_CUDA(cudaStreamSynchronize(p->stream));      // kernels in flight may still read the array
        cudaFree(p->d_log_std);
        p->d_log_std = nullptr;
        return IM_OK;
    }
    if (!p->d_log_std && cudaMalloc(&p->d_log_std, bytes) != cudaSuccess) return IM_ERR_ALLOC;
    IM_CUDA(cudaMemcpyAsync(p->d_log_std, log_std, bytes, cudaMemcpyDeviceToDevice, p->stream));
    return IM_OK;
}

im_status im_policy_forward(im_policy *p, uint32_t step, int32_t n, const float *obs, int32_t ld_obs,
                            float *mean_out, float *action_out, float *logp_out)
{
    if (!p || !obs || !mean_out || (!action_out && logp_out)) return IM_ERR_INVALID_ARG;
    if (n < 1 || n > p->cfg.max_batch || ld_obs < p->cfg.dims[0] || (ld_obs & 3) || !aligned16(obs))
        return IM_ERR_INVALID_ARG;
    if (p->tensor_path) {
        if (!aligned16(mean_out) || !aligned16(action_out)) return IM_ERR_INVALID_ARG;
        return tc_policy_forward(p, step, n, obs, ld_obs, mean_out, action_out, logp_out);
    }
    const float *in = obs;
    int ld_in = ld_obs;
    const int A = p->cfg.dims[p->nl];
    for (int l = 0; l < p->nl; ++l) {
        const bool last = l == p->nl - 1;
        float *outp = last ? mean_out : p->d_act[l & 1];
        const int ldc = last ? A : p->act_ld;
        IM_CUDA(launch_linear_simt(in, ld_in, p->d_W[l], p->cfg.dtype == 1, p->d_b[l], outp, ldc, n,
                                   p->cfg.dims[l + 1], p->cfg.dims[l], !last, p->stream));
        in = outp;
        ld_in = ldc;
    }
    if (action_out)
        IM_CUDA(launch_sample(mean_out, action_out, logp_out, n, A, p->cfg.sigma, p->d_log_std, p->cfg.seed, step,
                              p->cfg.env_id_base, p->stream));
    return IM_OK;
}

im_status im_policy_forward_staged(im_policy *p, uint32_t step, int32_t n, float *mean_out, float *action_out,
                                   float *logp_out)
{
    if (!p || !mean_out || !action_out) return IM_ERR_INVALID_ARG;
    if (!p->tensor_path) return IM_ERR_UNSUPPORTED;
    if (n < 1 || n > p->cfg.max_batch || !aligned16(mean_out) || !aligned16(action_out)) return IM_ERR_INVALID_ARG;
    return tc_policy_forward(p, step, n, nullptr, 0, mean_out, action_out, logp_out);
}

/* ------------------------------------------------------------------ adaptive episode initialisation */
im_status im_env_set_obs_extension(im_env *e, int32_t n_future, int32_t act_dim, const float *prev_action, int32_t ld_action)
{
    if (!e || n_future < 1 || n_future > 16 || act_dim < 0 || act_dim > 1024) return IM_ERR_INVALID_ARG;
    if (act_dim > 0 && (!prev_action || ld_action < act_dim)) return IM_ERR_INVALID_ARG;
    const int J = e->skel->dev.J;
    const int extra = (n_future - 1) * 9 * e->skel->n_ee + act_dim;
    const int D = 24 * J + 1 + extra;
    if (e->cfg.ld_obs < D) return IM_ERR_INVALID_ARG;
    const size_t smem = env_kernel_smem_bytes(J, e->skel->dev.n_chains, e->skel->dev.n_links, extra);
    int dev = 0, max_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if ((int64_t)smem > (int64_t)max_smem) return IM_ERR_UNSUPPORTED;
    e->n_future = n_future; e->act_dim = act_dim; e->prev_action = act_dim > 0 ? prev_action : nullptr;
    e->ld_action = act_dim > 0 ? ld_action : 0;
    if (D != e->D) e->d_obs_bf16 = nullptr;            // a policy attached for another width no longer fits
    e->D = D;
    e->smem_bytes = smem;
    return IM_OK;
}

im_status im_env_set_summary(im_env *e, uint64_t *acc)
{
    if (!e || (reinterpret_cast<uintptr_t>(acc) & 7u)) return IM_ERR_INVALID_ARG;
    e->d_summary = reinterpret_cast<unsigned long long *>(acc);
    return IM_OK;
}

im_status im_env_set_reset_bins(im_env *e, int32_t n_bins, const float *weights)
{
    if (!e || n_bins < 0 || (n_bins > 0 && !weights)) return IM_ERR_INVALID_ARG;
    const int64_t n = (int64_t)e->clips->C * n_bins;
    if (n > (1 << 26)) return IM_ERR_INVALID_ARG;
    std::vector<unsigned long long> T;
    try {
        T.resize((size_t)n);
    } catch (const std::bad_alloc &) {
        return IM_ERR_ALLOC;
    }
    if (n_bins > 0) {
        // T_i = floor(2^32 (w_0 + .. + w_i) / total), sums in order in fp64, last entry 2^32
        double total = 0.0, cum = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            if (!(weights[i] >= 0.0f) || std::isinf(weights[i])) return IM_ERR_INVALID_ARG;
            total += (double)weights[i];
        }
        if (!(total > 0.0)) return IM_ERR_INVALID_ARG;
        for (int64_t i = 0; i < n; ++i) {
            cum += (double)weights[i];
            T[(size_t)i] = (unsigned long long)std::floor(cum / total * 4294967296.0);
        }
        T[(size_t)n - 1] = 4294967296ull;
    }
    if (n_bins != e->n_bins) {
        // kernels enqueued earlier may still read the old tables
        IM_CUDA(cudaStreamSynchronize(e->stream));
        cudaFree(e->d_reset_cdf); cudaFree(e->d_stat_starts); cudaFree(e->d_stat_failures);
        e->d_reset_cdf = nullptr; e->d_stat_starts = e->d_stat_failures = nullptr;
        e->n_bins = 0;
        if (n_bins > 0) {
            if (cudaMalloc(&e->d_reset_cdf, (size_t)n * 8) != cudaSuccess ||
                cudaMalloc(&e->d_stat_starts, (size_t)n * 4) != cudaSuccess ||
                cudaMalloc(&e->d_stat_failures, (size_t)n * 4) != cudaSuccess) {
                cudaFree(e->d_reset_cdf); cudaFree(e->d_stat_starts); cudaFree(e->d_stat_failures);
                e->d_reset_cdf = nullptr; e->d_stat_starts = e->d_stat_failures = nullptr;
                return IM_ERR_ALLOC;
            }
            e->n_bins = n_bins;
            IM_CUDA(cudaMemsetAsync(e->d_stat_starts, 0, (size_t)n * 4, e->stream));
            IM_CUDA(cudaMemsetAsync(e->d_stat_failures, 0, (size_t)n * 4, e->stream));
        }
    }
    if (n_bins > 0) {
        IM_CUDA(cudaMemcpyAsync(e->d_reset_cdf, T.data(), (size_t)n * 8, cudaMemcpyHostToDevice, e->stream));
        IM_CUDA(cudaStreamSynchronize(e->stream));      // T is a local
    }
    return IM_OK;
}

im_status im_env_adapt_reset_bins(im_env *e, float floor_weight, int32_t clear)
{
    if (!e || !(floor_weight > 0.0f) || std::isinf(floor_weight)) return IM_ERR_INVALID_ARG;
    if (e->n_bins <= 0) return IM_ERR_UNSUPPORTED;
    const int64_t n = (int64_t)e->clips->C * e->n_bins;
    if (n > 12288) return IM_ERR_UNSUPPORTED;
    IM_CUDA(launch_adapt_reset_cdf(e->d_stat_starts, e->d_stat_failures, (int)n, floor_weight, clear, e->d_reset_cdf, e->stream));
    return IM_OK;
}

im_status im_env_get_reset_stats(im_env *e, uint32_t *starts, uint32_t *failures, int32_t clear)
{
    if (!e) return IM_ERR_INVALID_ARG;
    if (e->n_bins <= 0) return IM_ERR_UNSUPPORTED;
    const size_t bytes = (size_t)e->clips->C * e->n_bins * 4;
    if (starts) IM_CUDA(cudaMemcpyAsync(starts, e->d_stat_starts, bytes, cudaMemcpyDeviceToDevice, e->stream));
    if (failures) IM_CUDA(cudaMemcpyAsync(failures, e->d_stat_failures, bytes, cudaMemcpyDeviceToDevice, e->stream));
    if (clear) {
        IM_CUDA(cudaMemsetAsync(e->d_stat_starts, 0, bytes, e->stream));
        IM_CUDA(cudaMemsetAsync(e->d_stat_failures, 0, bytes, e->stream));
    }
    return IM_OK;
}

/* ------------------------------------------------------------------ value head */
im_status im_value_forward(im_policy *critic, int32_t n, const float *obs, int32_t ld_obs, float *value_out)
{
    return im_policy_forward(critic, 0u, n, obs, ld_obs, value_out, nullptr, nullptr);
}

im_status im_value_forward_staged(im_policy *critic, im_policy *src, int32_t n, float *value_out)
{
    if (!critic || !value_out) return IM_ERR_INVALID_ARG;
    if (!critic->tensor_path || (src && !src->tensor_path)) return IM_ERR_UNSUPPORTED;
    if (n < 1 || n > critic->cfg.max_batch || !aligned16(value_out)) return IM_ERR_INVALID_ARG;
    if (src && src->stream != critic->stream) return IM_ERR_INVALID_ARG;
    return tc_policy_forward(critic, 0u, n, nullptr, 0, value_out, nullptr, nullptr, src);
}

/* ------------------------------------------------------------------ host-buffer step */
static im_status ensure_staging(im_env *e, int A)
{
    const size_t n = (size_t)e->cfg.n_envs, J = (size_t)e->skel->dev.J;
    if (!e->d_sim) {
        if (cudaMalloc(&e->d_sim, 13 * J * n * 4) != cudaSuccess ||
            cudaMalloc(&e->d_obs, n * (size_t)e->cfg.ld_obs * 4) != cudaSuccess ||
            cudaMalloc(&e->d_reward, n * 4) != cudaSuccess || cudaMalloc(&e->d_flags, n) != cudaSuccess)
            return IM_ERR_ALLOC;
        if (cudaStreamCreateWithFlags(&e->h2d_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&e->d2h_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&e->ev_policy, cudaEventDisableTiming) != cudaSuccess)
            return IM_ERR_CUDA;
        for (int c = 0; c < kHostChunks; ++c)
            if (cudaEventCreateWithFlags(&e->ev_h2d[c], cudaEventDisableTiming) != cudaSuccess) return IM_ERR_CUDA;
    }
    if (A > e->staged_A) {
        cudaFree(e->d_mean); cudaFree(e->d_action);
        e->d_mean = e->d_action = nullptr;
        if (cudaMalloc(&e->d_mean, n * (size_t)A * 4) != cudaSuccess ||
            cudaMalloc(&e->d_action, n * (size_t)A * 4) != cudaSuccess)
            return IM_ERR_ALLOC;
        e->staged_A = A;
    }
    return IM_OK;
}

im_status im_env_reset_all_host(im_env *e, uint32_t step)
{
    if (!e) return IM_ERR_INVALID_ARG;
    const im_status s = ensure_staging(e, 0);
    if (s != IM_OK) return s;
    return im_env_reset_all(e, step, e->d_obs);
}

im_status im_step_host(im_env *e, im_policy *p, uint32_t step, const float *sim_host, float *action_host,
                       float *reward_host, uint8_t *flags_host)
{
    if (!e || !p || !sim_host || !action_host || !reward_host || !flags_host) return IM_ERR_INVALID_ARG;
    if (p->stream != e->stream || p->cfg.max_batch < e->cfg.n_envs || p->cfg.dims[0] != e->D) return IM_ERR_INVALID_ARG;
    if (e->act_dim > 0) return IM_ERR_UNSUPPORTED;     // the caller-owned previous-action buffer belongs to the device path
    const int A = p->cfg.dims[p->nl];
    if (!e->d_obs) return IM_ERR_INVALID_ARG;          // im_env_reset_all_host has not run
    im_status s = ensure_staging(e, A);
    if (s != IM_OK) return s;
    const size_t n = (size_t)e->cfg.n_envs, J = (size_t)e->skel->dev.J;
    // The body states are needed by the env step only: their upload runs on a copy stream beside
    // the policy forward, and the actions travel back beside the env step (PCIe is full duplex).
    // The previous call waited for all three streams, so the staging buffers are free.
    // The upload is cut into env ranges (columns of the [13 J][N] array) so that the env kernel of a range
    // starts as soon as its columns have arrived and only the last range's kernel is not hidden by the copy.
    // (measured: four ranges are 2 % faster at 65536 envs but 6 % slower at 16384 and 27 % slower at 4096, where the
    // extra launches and copies cost more than the hidden kernel time)
    const int chunks = (n >= 49152 && n % (4 * 32) == 0) ? kHostChunks : 1;
    const size_t nc = n / chunks;
    for (int c = 0; c < chunks; ++c) {
        IM_CUDA(cudaMemcpy2DAsync(e->d_sim + c * nc, n * 4, sim_host + c * nc, n * 4, nc * 4, 13 * J, cudaMemcpyHostToDevice,
                                  e->h2d_stream));
        IM_CUDA(cudaEventRecord(e->ev_h2d[c], e->h2d_stream));
    }
    int32_t ld_in = 0;
    if (e->d_obs_bf16 && p->tensor_path && e->d_obs_bf16 == tc_policy_input(p, &ld_in))
        s = im_policy_forward_staged(p, step, (int32_t)n, e->d_mean, e->d_action, nullptr);
    else
        s = im_policy_forward(p, step, (int32_t)n, e->d_obs, e->cfg.ld_obs, e->d_mean, e->d_action, nullptr);
    if (s != IM_OK) return s;
    IM_CUDA(cudaEventRecord(e->ev_policy, e->stream));
    IM_CUDA(cudaStreamWaitEvent(e->d2h_stream, e->ev_policy, 0));
    IM_CUDA(cudaMemcpyAsync(action_host, e->d_action, n * (size_t)A * 4, cudaMemcpyDeviceToHost, e->d2h_stream));
    im_body_state sim = {e->d_sim, e->d_sim + 3 * J * n, e->d_sim + 7 * J * n, e->d_sim + 10 * J * n, (int64_t)n};
    for (int c = 0; c < chunks; ++c) {
        IM_CUDA(cudaStreamWaitEvent(e->stream, e->ev_h2d[c], 0));
        s = env_step_range(e, step, &sim, e->d_obs, e->d_reward, e->d_flags, (int)(c * nc), (int)nc);
        if (s != IM_OK) return s;
    }
    IM_CUDA(cudaMemcpyAsync(reward_host, e->d_reward, n * 4, cudaMemcpyDeviceToHost, e->stream));
    IM_CUDA(cudaMemcpyAsync(flags_host, e->d_flags, n, cudaMemcpyDeviceToHost, e->stream));
    IM_CUDA(cudaStreamSynchronize(e->stream));
    IM_CUDA(cudaStreamSynchronize(e->d2h_stream));
    return IM_OK;
}

im_status im_debug_set_wait(uint64_t limit_ns, int32_t skip_loads)
{
    if (limit_ns == 0) return IM_ERR_INVALID_ARG;
    IM_CUDA(cudaDeviceSynchronize());                   // kernels in flight keep the setting they started with
    IM_CUDA(tc_set_wait_debug(limit_ns, skip_loads != 0));
    IM_CUDA(ppo_set_wait_debug(limit_ns, skip_loads != 0));
    return IM_OK;
}

im_status im_debug_math(int32_t op, int32_t n, const float *in, float *out, void *cuda_stream)
{
    if ((op != IM_DEBUG_ANGLE_SQ && op != IM_DEBUG_SLERP) || n < 1 || !in || !out) return IM_ERR_INVALID_ARG;
    IM_CUDA(launch_debug_math(op, n, in, out, (cudaStream_t)cuda_stream));
    return IM_OK;
}

im_status im_poll_device_status(im_env *e, im_policy *p, uint32_t *out)
{
    if (!out || (!e && !p) || (e && p)) return IM_ERR_INVALID_ARG;
    cudaStream_t st = e ? e->stream : p->stream;
    const uint32_t *src = e ? e->d_status : p->d_status;
    IM_CUDA(cudaMemcpyAsync(out, src, 4, cudaMemcpyDeviceToHost, st));
    IM_CUDA(cudaStreamSynchronize(st));
    return IM_OK;
}

}  // extern "C"
