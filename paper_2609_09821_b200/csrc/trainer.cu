// The update phase behind the C ABI (the paper's `update_policy(storage)`, Figure 2): an MLP trainer
// handle (fp32 master weights, Adam state, bf16 working copies, activation and gradient buffers, the
// buffer plan and the row-slice choice of the dW products) and a PPO updater handle that sequences one
// minibatch update of an actor and a critic, or all epochs and minibatches of a collected rollout.
// Host code only: every arithmetic step is one of the library's kernels, reached through the same entry
// points a caller could use one by one.
#include <cmath>
#include <cstring>
#include <new>

#include "im_internal.h"
#include "mlp.h"

namespace {

int pad64(int x) { return (x + 63) / 64 * 64; }
int pad128(int x) { return (x + 127) / 128 * 128; }

// Device array of n elements, zeroed on `st` (the stream everything else of the handle runs on) unless told otherwise.
template <typename T> bool dev_alloc(T **p, size_t n, cudaStream_t st, bool zero = true)
{
    if (cudaMalloc(p, n * sizeof(T)) != cudaSuccess) { *p = nullptr; return false; }
    return !zero || cudaMemsetAsync(*p, 0, n * sizeof(T), st) == cudaSuccess;
}

}  // namespace

struct im_trainer {
    int nl, Mb, t, max_split;
    int dims[IM_MAX_LAYERS + 1], Kp[IM_MAX_LAYERS], Np[IM_MAX_LAYERS];
    cudaStream_t stream;
    float *W[IM_MAX_LAYERS], *b[IM_MAX_LAYERS], *mW[IM_MAX_LAYERS], *vW[IM_MAX_LAYERS], *mb[IM_MAX_LAYERS], *vb[IM_MAX_LAYERS];
    float *dW[IM_MAX_LAYERS], *db[IM_MAX_LAYERS];
    uint16_t *Wb[IM_MAX_LAYERS], *WbT[IM_MAX_LAYERS];      // bf16 [Np][Kp] and its transpose [Kp][Np]
    uint16_t *H[IM_MAX_LAYERS];                            // H[0]: input rows [Mb][Kp0]; H[l]: activations [Mb][Np[l-1]]
    uint16_t *dZ[IM_MAX_LAYERS];                           // gradient at layer l's pre-activation [Mb][Np[l]]
    float *out;                                            // [Mb][dims[nl]]
    uint16_t *dWs;                                         // partial dW products of one layer, all row slices
    float *colsum_ws, *col_partial;
    size_t colsum_ws_bytes;
    int ld_partial;
    uint32_t *status;
};

struct im_ppo_updater {
    im_trainer *actor, *critic;
    im_ppo_update_config cfg;
    int A, Mb, t;
    float *log_std, *log_std_old, *m_ls, *v_ls, *d_log_std, *lr, *scale, *moments, *summary, *d_mean, *d_value;
    void *ws;
    float *g_action, *g_mean_old, *g_logp_old, *g_advantage, *g_value_old, *g_returns;   // gathered minibatch (shuffled updates)
    int g_rows;
};

extern "C" {

/* Row slices of the dW product of a layer with Np (padded) outputs and Kp (padded) inputs on M rows.  dW contracts
 * over the batch -- a long sum feeding few output tiles -- so the rows are cut into S slices that run as one launch.
 * S is the power of two (slices of whole 128-row blocks) with the least modelled time: waves of tiles on 148 SMs
 * times rows per slice (5 ns per row and wave, measured on a 1024 x 1024 layer), plus the pass that adds the S
 * partial products (1 ps per element).  any_rows: ignore the divisibility rule (an upper bound for sizing). */
int32_t im_trainer_dw_slices(int32_t Np, int32_t Kp, int64_t M, int32_t max_split, int32_t any_rows)
{
    const int npb = pad128(Np);
    const long long tiles = (long long)(npb / 128) * ((Kp + 255) / 256 > 1 ? (Kp + 255) / 256 : 1);
    int best = 1;
    double best_cost = -1.0;
    for (int S = 1; S <= max_split && (any_rows || M % (128LL * S) == 0); S *= 2) {
        const long long waves = (tiles * S + 147) / 148;
        const double cost = 5e-9 * (double)M * (double)waves / S + 1e-12 * (double)S * npb * Kp;
        if (best_cost < 0.0 || cost < best_cost * (1.0 - 1e-9)) { best = S; best_cost = cost; }
    }
    return best;
}

void im_trainer_destroy(im_trainer *tr)
{
    if (!tr) return;
    for (int l = 0; l < IM_MAX_LAYERS; ++l) {
        cudaFree(tr->W[l]); cudaFree(tr->b[l]); cudaFree(tr->mW[l]); cudaFree(tr->vW[l]); cudaFree(tr->mb[l]); cudaFree(tr->vb[l]);
        cudaFree(tr->dW[l]); cudaFree(tr->db[l]); cudaFree(tr->Wb[l]); cudaFree(tr->WbT[l]); cudaFree(tr->H[l]); cudaFree(tr->dZ[l]);
    }
    cudaFree(tr->out); cudaFree(tr->dWs); cudaFree(tr->colsum_ws); cudaFree(tr->col_partial); cudaFree(tr->status);
    delete tr;
}

im_status im_trainer_create(int32_t n_layers, const int32_t *dims, const float *const *W, const float *const *b,
                            int32_t max_rows, void *cuda_stream, im_trainer **out)
{
    if (!dims || !W || !b || !out || n_layers < 2 || n_layers > IM_MAX_LAYERS) return IM_ERR_INVALID_ARG;
    if (max_rows < 64 || (max_rows & 63)) return IM_ERR_INVALID_ARG;
    for (int l = 0; l <= n_layers; ++l)
        if (dims[l] < 1) return IM_ERR_INVALID_ARG;
    for (int l = 1; l < n_layers; ++l)
        if (dims[l] & 63) return IM_ERR_UNSUPPORTED;                 // hidden widths are whole 64-column tiles
    if (dims[n_layers] > 80) return IM_ERR_UNSUPPORTED;              // the fp32-output head kernel
    for (int l = 0; l < n_layers; ++l)
        if (!W[l] || !b[l]) return IM_ERR_INVALID_ARG;
    if (im::device_sm_count() <= 0) return IM_ERR_UNSUPPORTED;
    im_trainer *tr = new (std::nothrow) im_trainer();
    if (!tr) return IM_ERR_ALLOC;
    std::memset(tr, 0, sizeof(*tr));
    tr->nl = n_layers; tr->Mb = max_rows; tr->max_split = 64; tr->stream = (cudaStream_t)cuda_stream;
    cudaStream_t st = tr->stream;
    for (int l = 0; l <= n_layers; ++l) tr->dims[l] = dims[l];
    int maxNp = 0;
    size_t need = 0;
    bool ok = true;
    for (int l = 0; l < n_layers && ok; ++l) {
        const int N = dims[l + 1], K = dims[l], Np = pad64(N), Kp = pad64(K);
        tr->Np[l] = Np; tr->Kp[l] = Kp;
        maxNp = Np > maxNp ? Np : maxNp;
        const size_t wn = (size_t)N * K;
        ok = dev_alloc(&tr->W[l], wn, st, false) && dev_alloc(&tr->b[l], (size_t)Np, st) && dev_alloc(&tr->mW[l], wn, st) &&
             dev_alloc(&tr->vW[l], wn, st) && dev_alloc(&tr->mb[l], (size_t)N, st) && dev_alloc(&tr->vb[l], (size_t)N, st) &&
             dev_alloc(&tr->dW[l], wn, st) && dev_alloc(&tr->db[l], (size_t)N, st) && dev_alloc(&tr->Wb[l], (size_t)Np * Kp, st) &&
             dev_alloc(&tr->WbT[l], (size_t)Kp * Np, st) && dev_alloc(&tr->H[l], (size_t)max_rows * Kp, st) &&
             dev_alloc(&tr->dZ[l], (size_t)max_rows * Np, st);
        // partial dW products: room for the most slices the model can choose (more rows never favour fewer slices)
        const size_t s_max = (size_t)im_trainer_dw_slices(Np, Kp, max_rows, tr->max_split, 1);
        const size_t n = s_max * pad128(Np) * Kp;
        need = n > need ? n : need;
    }
    const size_t slices256 = ((size_t)max_rows + 255) / 256;
    tr->colsum_ws_bytes = slices256 * (size_t)(maxNp > 80 ? maxNp : 80) * sizeof(float);
    tr->ld_partial = maxNp;
    ok = ok && dev_alloc(&tr->out, (size_t)max_rows * dims[n_layers], st) && dev_alloc(&tr->dWs, need, st) &&
         dev_alloc(&tr->colsum_ws, tr->colsum_ws_bytes / sizeof(float), st, false) &&
         dev_alloc(&tr->col_partial, (size_t)(max_rows / 32) * maxNp, st, false) && dev_alloc(&tr->status, 1, st);
    if (!ok) { im_trainer_destroy(tr); return IM_ERR_ALLOC; }
    // weights: fp32 masters as given; bf16 working copies (rounded on the device, zero padded) and their transposes
    for (int l = 0; l < n_layers; ++l) {
        const int N = dims[l + 1], K = dims[l];
        if (cudaMemcpyAsync(tr->W[l], W[l], (size_t)N * K * sizeof(float), cudaMemcpyHostToDevice, tr->stream) != cudaSuccess ||
            cudaMemcpyAsync(tr->b[l], b[l], (size_t)N * sizeof(float), cudaMemcpyHostToDevice, tr->stream) != cudaSuccess) {
            im_trainer_destroy(tr);
            return IM_ERR_CUDA;
        }
        im_status s = im_f32_to_bf16_padded(tr->W[l], K, N, K, tr->Wb[l], tr->Kp[l], tr->stream);
        if (s == IM_OK) s = im_transpose_bf16(tr->Wb[l], tr->Kp[l], tr->Np[l], tr->Kp[l], tr->WbT[l], tr->Np[l], tr->stream);
        if (s != IM_OK) { im_trainer_destroy(tr); return s; }
    }
    if (cudaStreamSynchronize(tr->stream) != cudaSuccess) { im_trainer_destroy(tr); return IM_ERR_CUDA; }   // W, b are the caller's
    *out = tr;
    return IM_OK;
}

im_status im_trainer_tensor(im_trainer *tr, int32_t which, int32_t layer, void **ptr, int64_t *rows, int64_t *cols,
                            int64_t *ld, int32_t *dtype)
{
    if (!tr || !ptr || !rows || !cols || !ld || !dtype) return IM_ERR_INVALID_ARG;
    const bool per_layer = which != IM_TRAINER_OUT && which != IM_TRAINER_STATUS;
    if (per_layer && (layer < 0 || layer >= tr->nl)) return IM_ERR_INVALID_ARG;
    const int l = per_layer ? layer : 0;
    const int64_t N = tr->dims[l + 1], K = tr->dims[l], Np = tr->Np[l], Kp = tr->Kp[l];
    *dtype = IM_DTYPE_F32;
    switch (which) {
    case IM_TRAINER_W: *ptr = tr->W[l]; *rows = N; *cols = K; *ld = K; break;
    case IM_TRAINER_B: *ptr = tr->b[l]; *rows = 1; *cols = N; *ld = Np; break;
    case IM_TRAINER_W_BF16: *ptr = tr->Wb[l]; *rows = Np; *cols = Kp; *ld = Kp; *dtype = IM_DTYPE_BF16; break;
    case IM_TRAINER_WT_BF16: *ptr = tr->WbT[l]; *rows = Kp; *cols = Np; *ld = Np; *dtype = IM_DTYPE_BF16; break;
    case IM_TRAINER_M_W: *ptr = tr->mW[l]; *rows = N; *cols = K; *ld = K; break;
    case IM_TRAINER_V_W: *ptr = tr->vW[l]; *rows = N; *cols = K; *ld = K; break;
    case IM_TRAINER_M_B: *ptr = tr->mb[l]; *rows = 1; *cols = N; *ld = N; break;
    case IM_TRAINER_V_B: *ptr = tr->vb[l]; *rows = 1; *cols = N; *ld = N; break;
    case IM_TRAINER_DW: *ptr = tr->dW[l]; *rows = N; *cols = K; *ld = K; break;
    case IM_TRAINER_DB: *ptr = tr->db[l]; *rows = 1; *cols = N; *ld = N; break;
    case IM_TRAINER_H: *ptr = tr->H[l]; *rows = tr->Mb; *cols = Kp; *ld = Kp; *dtype = IM_DTYPE_BF16; break;
    case IM_TRAINER_OUT: *ptr = tr->out; *rows = tr->Mb; *cols = tr->dims[tr->nl]; *ld = tr->dims[tr->nl]; break;
    case IM_TRAINER_STATUS: *ptr = tr->status; *rows = 1; *cols = 1; *ld = 1; *dtype = IM_DTYPE_U32; break;
    default: return IM_ERR_INVALID_ARG;
    }
    return IM_OK;
}

im_status im_trainer_set_step_count(im_trainer *tr, int32_t t)
{
    if (!tr || t < 0) return IM_ERR_INVALID_ARG;
    tr->t = t;
    return IM_OK;
}

im_status im_trainer_forward(im_trainer *tr, int32_t M)
{
    if (!tr || M < 1 || M > tr->Mb) return IM_ERR_INVALID_ARG;
    const int L = tr->nl - 1;
    for (int l = 0; l < L; ++l) {
        const im_status s = im_gemm_bf16(tr->H[l], tr->Kp[l], tr->Wb[l], tr->Kp[l], tr->H[l + 1], tr->Np[l], M, tr->Np[l],
                                         tr->Kp[l], tr->b[l], 1, tr->status, tr->stream);
        if (s != IM_OK) return s;
    }
    return im_gemm_bf16_f32out(tr->H[L], tr->Kp[L], tr->Wb[L], tr->Kp[L], tr->out, M, tr->dims[tr->nl], tr->Kp[L], tr->b[L],
                               tr->status, tr->stream);
}

im_status im_trainer_backward(im_trainer *tr, const float *d_out, int32_t M)
{
    if (!tr || !d_out || M < 64 || (M & 63) || M > tr->Mb) return IM_ERR_INVALID_ARG;
    const int L = tr->nl - 1, A = tr->dims[tr->nl];
    im_status s = im_f32_to_bf16_padded(d_out, A, M, A, tr->dZ[L], tr->Np[L], tr->stream);
    if (s == IM_OK) s = im_colsum_f32(d_out, A, M, A, tr->db[L], tr->colsum_ws, tr->colsum_ws_bytes, tr->stream);
    for (int l = L; l >= 0 && s == IM_OK; --l) {
        const int N = tr->dims[l + 1], K = tr->dims[l], Np = tr->Np[l], Kp = tr->Kp[l];
        // dW = dZ^T H over S row slices in one launch (both operands read as they lie, M/N-major tensor-core
        // operands: no transposed copies); the S partial products are added afterwards
        const int Npb = pad128(Np);
        const int S = im_trainer_dw_slices(Np, Kp, M, tr->max_split, 0);
        s = im_gemm_bf16_tn(tr->dZ[l], Np, tr->H[l], Kp, tr->dWs, Kp, M, Np, Kp, S, Npb, tr->status, tr->stream);
        if (s == IM_OK) s = im_sum_slices_bf16_to_f32(tr->dWs, (int64_t)Npb * Kp, Kp, S, N, K, tr->dW[l], tr->stream);
        if (l > 0 && s == IM_OK) {
            // dH = (H > 0) * (dZ W); the product's epilogue applies the ReLU mask and leaves the column sums of every
            // 32-row block, which add up to the bias gradient of the layer below
            s = im_gemm_bf16_dgrad(tr->dZ[l], Np, tr->WbT[l], Np, tr->dZ[l - 1], Kp, M, Kp, Np, tr->H[l], Kp, tr->col_partial,
                                   tr->ld_partial, tr->status, tr->stream);
            if (s == IM_OK)
                s = im_colsum_f32(tr->col_partial, tr->ld_partial, M / 32, K, tr->db[l - 1], tr->colsum_ws, tr->colsum_ws_bytes,
                                  tr->stream);
        }
    }
    return s;
}

im_status im_trainer_step(im_trainer *tr, const im_adam_config *adam, const float *lr, const float *grad_scale)
{
    if (!tr || !adam || !lr) return IM_ERR_INVALID_ARG;
    tr->t += 1;
    for (int l = 0; l < tr->nl; ++l) {
        const int N = tr->dims[l + 1], K = tr->dims[l];
        im_status s = im_adam_step(adam, tr->t, (int64_t)N * K, tr->W[l], tr->dW[l], tr->mW[l], tr->vW[l], lr, grad_scale,
                                   tr->Wb[l], K, tr->Kp[l], tr->stream);
        if (s == IM_OK) s = im_adam_step(adam, tr->t, N, tr->b[l], tr->db[l], tr->mb[l], tr->vb[l], lr, grad_scale, nullptr, 0, 0, tr->stream);
        if (s == IM_OK) s = im_transpose_bf16(tr->Wb[l], tr->Kp[l], tr->Np[l], tr->Kp[l], tr->WbT[l], tr->Np[l], tr->stream);
        if (s != IM_OK) return s;
    }
    return IM_OK;
}

im_status im_trainer_push_to_policy(im_trainer *tr, im_policy *p)
{
    if (!tr || !p || p->nl != tr->nl || p->stream != tr->stream) return IM_ERR_INVALID_ARG;
    for (int l = 0; l <= tr->nl; ++l)
        if (p->cfg.dims[l] != tr->dims[l]) return IM_ERR_INVALID_ARG;
    for (int l = 0; l < tr->nl; ++l) {
        void *w = nullptr;
        int32_t ld = 0;
        float *bias = nullptr;
        im_status s = im_policy_layer_buffers(p, l, &w, &ld, &bias);
        if (s != IM_OK) return s;
        const int N = tr->dims[l + 1], K = tr->dims[l];
        if (p->tensor_path || p->cfg.dtype == 1) {
            s = im_f32_to_bf16_padded(tr->W[l], K, N, K, static_cast<uint16_t *>(w), ld, tr->stream);
        } else {
            s = cudaMemcpy2DAsync(w, (size_t)ld * 4, tr->W[l], (size_t)K * 4, (size_t)K * 4, N, cudaMemcpyDeviceToDevice, tr->stream) ==
                        cudaSuccess ? IM_OK : IM_ERR_CUDA;
        }
        if (s == IM_OK) s = im_copy_f32(bias, tr->b[l], N, tr->stream);
        if (s != IM_OK) return s;
    }
    return IM_OK;
}

/* ------------------------------------------------------------------ PPO updater */
void im_ppo_updater_destroy(im_ppo_updater *u)
{
    if (!u) return;
    cudaFree(u->log_std); cudaFree(u->log_std_old); cudaFree(u->m_ls); cudaFree(u->v_ls); cudaFree(u->d_log_std); cudaFree(u->lr);
    cudaFree(u->scale); cudaFree(u->moments); cudaFree(u->summary); cudaFree(u->d_mean); cudaFree(u->d_value); cudaFree(u->ws);
    cudaFree(u->g_action); cudaFree(u->g_mean_old); cudaFree(u->g_logp_old); cudaFree(u->g_advantage); cudaFree(u->g_value_old);
    cudaFree(u->g_returns);
    delete u;
}

im_status im_ppo_updater_create(im_trainer *actor, im_trainer *critic, const float *log_std, const im_ppo_update_config *cfg,
                                im_ppo_updater **out)
{
    if (!actor || !critic || !log_std || !cfg || !out) return IM_ERR_INVALID_ARG;
    if (actor->stream != critic->stream || critic->dims[critic->nl] != 1 || actor->Mb != critic->Mb) return IM_ERR_INVALID_ARG;
    if (!(cfg->lr > 0.0f) || !(cfg->clip > 0.0f) || !(cfg->max_grad_norm > 0.0f) || !(cfg->lr_min <= cfg->lr_max)) return IM_ERR_INVALID_ARG;
    im_ppo_updater *u = new (std::nothrow) im_ppo_updater();
    if (!u) return IM_ERR_ALLOC;
    std::memset(u, 0, sizeof(*u));
    u->actor = actor; u->critic = critic; u->cfg = *cfg; u->A = actor->dims[actor->nl]; u->Mb = actor->Mb;
    const size_t A = (size_t)u->A;
    cudaStream_t st = actor->stream;
    bool ok = dev_alloc(&u->log_std, A, st) && dev_alloc(&u->log_std_old, A, st) && dev_alloc(&u->m_ls, A, st) && dev_alloc(&u->v_ls, A, st) &&
              dev_alloc(&u->d_log_std, A, st) && dev_alloc(&u->lr, 1, st) && dev_alloc(&u->scale, 2, st) && dev_alloc(&u->moments, 2, st) &&
              dev_alloc(&u->summary, 6, st) && dev_alloc(&u->d_mean, (size_t)u->Mb * A, st) && dev_alloc(&u->d_value, (size_t)u->Mb, st) &&
              cudaMalloc(&u->ws, im_ppo_workspace_bytes()) == cudaSuccess;
    if (!ok) { im_ppo_updater_destroy(u); return IM_ERR_ALLOC; }
    if (cudaMemcpyAsync(u->log_std, log_std, A * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(u->log_std_old, log_std, A * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(u->lr, &cfg->lr, 4, cudaMemcpyHostToDevice, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
        im_ppo_updater_destroy(u);
        return IM_ERR_CUDA;
    }
    *out = u;
    return IM_OK;
}

im_status im_ppo_updater_tensor(im_ppo_updater *u, int32_t which, float **ptr, int64_t *n)
{
    if (!u || !ptr || !n) return IM_ERR_INVALID_ARG;
    switch (which) {
    case IM_PPO_LOG_STD: *ptr = u->log_std; *n = u->A; break;
    case IM_PPO_LOG_STD_OLD: *ptr = u->log_std_old; *n = u->A; break;
    case IM_PPO_M_LOG_STD: *ptr = u->m_ls; *n = u->A; break;
    case IM_PPO_V_LOG_STD: *ptr = u->v_ls; *n = u->A; break;
    case IM_PPO_LR: *ptr = u->lr; *n = 1; break;
    case IM_PPO_GRAD_SCALE: *ptr = u->scale; *n = 2; break;
    case IM_PPO_SUMMARY: *ptr = u->summary; *n = 6; break;
    default: return IM_ERR_INVALID_ARG;
    }
    return IM_OK;
}

im_status im_ppo_updater_set_step_count(im_ppo_updater *u, int32_t t)
{
    if (!u || t < 0) return IM_ERR_INVALID_ARG;
    u->t = t;
    return IM_OK;
}

im_status im_ppo_update(im_ppo_updater *u, int32_t M, const im_ppo_minibatch *mb)
{
    if (!u || !mb || M < 64 || (M & 63) || M > u->Mb) return IM_ERR_INVALID_ARG;
    if (!mb->action || !mb->mean_old || !mb->logp_old || !mb->advantage || !mb->returns) return IM_ERR_INVALID_ARG;
    if (u->cfg.clip_value_loss && !mb->value_old) return IM_ERR_INVALID_ARG;
    im_trainer *a = u->actor, *c = u->critic;
    cudaStream_t st = a->stream;
    im_status s = im_trainer_forward(a, M);
    if (s == IM_OK) s = im_trainer_forward(c, M);
    if (s != IM_OK) return s;
    const float *mom = nullptr;
    if (u->cfg.normalize_advantage) {
        s = im_moments(mb->advantage, M, u->moments, u->ws, st);
        if (s != IM_OK) return s;
        mom = u->moments;
    }
    const im_ppo_config pc = {u->cfg.clip, u->cfg.value_coef, u->cfg.entropy_coef, u->cfg.clip_value_loss};
    const im_ppo_batch pb = {a->out, u->log_std, mb->action, mb->logp_old, mb->mean_old,
                             mb->log_std_old ? mb->log_std_old : u->log_std_old, mb->advantage, mom, c->out, mb->value_old, mb->returns};
    s = im_ppo_loss(&pc, M, u->A, &pb, u->d_mean, u->d_log_std, u->d_value, u->summary, u->ws, st);
    if (s == IM_OK) s = im_trainer_backward(a, u->d_mean, M);
    if (s == IM_OK) s = im_trainer_backward(c, u->d_value, M);
    if (s != IM_OK) return s;
    // global-norm clip over every gradient tensor of both nets and the log-std
    const float *grads[4 * IM_MAX_LAYERS + 1];
    int64_t sizes[4 * IM_MAX_LAYERS + 1];
    int n = 0;
    for (im_trainer *t : {a, c}) {
        for (int l = 0; l < t->nl; ++l) { grads[n] = t->dW[l]; sizes[n++] = (int64_t)t->dims[l + 1] * t->dims[l]; }
        for (int l = 0; l < t->nl; ++l) { grads[n] = t->db[l]; sizes[n++] = t->dims[l + 1]; }
    }
    grads[n] = u->d_log_std; sizes[n++] = u->A;
    s = im_grad_scale(n, grads, sizes, u->cfg.max_grad_norm, u->scale, u->ws, st);
    if (s == IM_OK) s = im_trainer_step(a, &u->cfg.adam, u->lr, u->scale);
    if (s == IM_OK) s = im_trainer_step(c, &u->cfg.adam, u->lr, u->scale);
    u->t += 1;
    if (s == IM_OK) s = im_adam_step(&u->cfg.adam, u->t, u->A, u->log_std, u->d_log_std, u->m_ls, u->v_ls, u->lr, u->scale, nullptr, 0, 0, st);
    if (s == IM_OK) s = im_adaptive_lr(u->lr, u->summary + 4, u->cfg.kl_target, u->cfg.lr_min, u->cfg.lr_max, st);
    return s;
}

im_status im_ppo_update_rollout(im_ppo_updater *u, const im_rollout_view *v, int32_t epochs, int32_t n_minibatches,
                                const int32_t *perm)
{
    if (!u || !v || epochs < 1 || n_minibatches < 1) return IM_ERR_INVALID_ARG;
    if (!v->obs || !v->action || !v->mean || !v->logp || !v->advantage || !v->returns || !v->value) return IM_ERR_INVALID_ARG;
    const int64_t total = (int64_t)v->T * v->N;
    if (v->T < 1 || v->N < 1 || v->A != u->A || total % n_minibatches) return IM_ERR_INVALID_ARG;
    const int64_t M64 = total / n_minibatches;
    if (M64 % 64 || M64 > u->Mb) return IM_ERR_INVALID_ARG;
    const int M = (int)M64, A = u->A, D = u->actor->dims[0];
    if (u->critic->dims[0] != D || v->ld_obs < D) return IM_ERR_INVALID_ARG;
    cudaStream_t st = u->actor->stream;
    if (perm && u->g_rows < M) {
        // (first shuffled update of this size: buffers for the gathered minibatch)
        cudaFree(u->g_action); cudaFree(u->g_mean_old); cudaFree(u->g_logp_old); cudaFree(u->g_advantage); cudaFree(u->g_value_old);
        cudaFree(u->g_returns);
        u->g_rows = 0;
        if (!dev_alloc(&u->g_action, (size_t)M * A, st, false) || !dev_alloc(&u->g_mean_old, (size_t)M * A, st, false) ||
            !dev_alloc(&u->g_logp_old, (size_t)M, st, false) || !dev_alloc(&u->g_advantage, (size_t)M, st, false) ||
            !dev_alloc(&u->g_value_old, (size_t)M, st, false) || !dev_alloc(&u->g_returns, (size_t)M, st, false))
            return IM_ERR_ALLOC;
        u->g_rows = M;
    }
    for (int ep = 0; ep < epochs; ++ep) {
        for (int k = 0; k < n_minibatches; ++k) {
            const int64_t r0 = (int64_t)k * M;
            im_ppo_minibatch mb;
            im_status s = IM_OK;
            if (!perm) {
                // contiguous block: the observations are converted into both nets' input rows, the rest is read in place
                for (im_trainer *t : {u->actor, u->critic})
                    if (s == IM_OK) s = im_f32_to_bf16_padded(v->obs + r0 * v->ld_obs, v->ld_obs, M, D, t->H[0], t->Kp[0], st);
                mb = {v->action + r0 * A, v->mean + r0 * A, nullptr, v->logp + r0, v->advantage + r0, v->value + r0, v->returns + r0};
            } else {
                const int32_t *idx = perm + (int64_t)ep * total + r0;
                for (im_trainer *t : {u->actor, u->critic})
                    if (s == IM_OK) s = im_gather_rows_f32(v->obs, v->ld_obs, idx, total, M, D, t->H[0], t->Kp[0], 1, u->actor->status, st);
                const struct { const float *src; int cols; float *dst; } g[6] = {
                    {v->action, A, u->g_action}, {v->mean, A, u->g_mean_old}, {v->logp, 1, u->g_logp_old},
                    {v->advantage, 1, u->g_advantage}, {v->value, 1, u->g_value_old}, {v->returns, 1, u->g_returns}};
                for (const auto &x : g)
                    if (s == IM_OK) s = im_gather_rows_f32(x.src, x.cols, idx, total, M, x.cols, x.dst, x.cols, 0, u->actor->status, st);
                mb = {u->g_action, u->g_mean_old, nullptr, u->g_logp_old, u->g_advantage, u->g_value_old, u->g_returns};
            }
            if (s == IM_OK) s = im_ppo_update(u, M, &mb);
            if (s != IM_OK) return s;
        }
    }
    return IM_OK;
}

}  // extern "C"
