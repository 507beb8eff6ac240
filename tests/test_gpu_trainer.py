"""GPU parity of the training-side path (forward with kept activations, backward pass, Adam step) of
one MLP against the CPU oracle, through the C ABI.

Tolerance of the gradients: the oracle takes the kernels' operand precision (bf16 activations, output
gradients and dH, exact sums, dW rounded to bf16); what is left is fp32 accumulation order, the rare
bf16 rounding flip of a hidden activation (fp32 versus exact accumulation) and what it does to a ReLU
mask.  Bound used: |g - o| <= 2e-2 (|o| + rms of the tensor), the policy-mean bar of the forward path.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import trainer as T
from paper_2609_09821_b200 import workloads as W

pytestmark = pytest.mark.gpu


def close(got, want, tol, what):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    lim = tol * (np.abs(want) + np.sqrt(np.mean(want ** 2)))
    bad = np.abs(got - want) > lim
    assert not bad.any(), "%s: %d of %d outside %.0e, worst %.3e" % (what, bad.sum(), bad.size, tol,
                                                                      (np.abs(got - want) / (lim / tol + 1e-300)).max())


def test_building_blocks_against_plain_definitions():
    g = torch.Generator(device="cuda").manual_seed(1)
    x = torch.randn((300, 200), device="cuda", generator=g).to(torch.bfloat16)
    out = torch.zeros((200, 304), dtype=torch.bfloat16, device="cuda")
    B.transpose_bf16(x, out[:, :300])
    assert torch.equal(out[:, :300], x.t())
    f = torch.randn((70, 69), device="cuda", generator=g)
    p = torch.full((70, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    B.f32_to_bf16_padded(f, p)
    assert torch.equal(p[:, :69], f.to(torch.bfloat16)) and (p[:, 69:] == 0).all()
    q = torch.full((70, 124), 7.0, dtype=torch.bfloat16, device="cuda")       # row stride not a multiple of 8: scalar kernel
    B.f32_to_bf16_padded(f, q)
    assert torch.equal(q[:, :69], f.to(torch.bfloat16)) and (q[:, 69:] == 0).all()
    wide = torch.randn((3001, 577), device="cuda", generator=g)
    pw = torch.full((3001, 640), 7.0, dtype=torch.bfloat16, device="cuda")
    B.f32_to_bf16_padded(wide, pw)
    assert torch.equal(pw[:, :577], wide.to(torch.bfloat16)) and (pw[:, 577:] == 0).all()
    big = torch.randn((5000, 300), device="cuda", generator=g)
    ws = torch.empty(20 * 300, device="cuda")
    cs = torch.empty(300, device="cuda")
    B.colsum(big, cs, ws)
    np.testing.assert_allclose(cs.cpu().numpy(), big.double().sum(0).cpu().numpy(), rtol=1e-5, atol=1e-4)
    with pytest.raises(B.ImError):
        B.colsum(big, cs, ws[:300])                       # workspace too small for twenty slices


@pytest.mark.parametrize("M,N,K,relu", [(200, 64, 64, True), (1000, 256, 192, False), (4096, 1024, 640, True),
                                         (130, 128, 1024, False)])
def test_generic_gemm_against_exact_products(M, N, K, relu):
    """bf16 operands, exact products summed in fp64, bf16 output: the kernel may differ by the fp32
    accumulation and one bf16 rounding."""
    g = np.random.default_rng(M + N)
    a = W.round_to_bf16(g.standard_normal((M, K)).astype(np.float32))[0]
    b = W.round_to_bf16((g.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))[0]
    bias = g.standard_normal(N).astype(np.float32)
    want = a.astype(np.float64) @ b.astype(np.float64).T + bias
    if relu:
        want = np.maximum(want, 0.0)
    A_, B_ = torch.from_numpy(a).cuda().to(torch.bfloat16), torch.from_numpy(b).cuda().to(torch.bfloat16)
    C_ = torch.full((M, N), 9.0, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gemm_bf16(A_, B_, C_, torch.from_numpy(bias).cuda(), relu, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = C_.float().cpu().numpy()
    assert np.abs(got - want).max() <= 2.0 ** -8 * np.abs(want).max() + 1e-3
    close(got, want, 1e-2, "gemm")


@pytest.mark.parametrize("dims,M", [((361, 128, 64, 28), 256), ((577, 256, 128, 69), 640), ((361, 64, 1), 128),
                                    ((577, 256, 128, 69), 1024)])       # the last one splits every dW product in four
def test_forward_backward_and_step_match_oracle(dims, M):
    pw = W.make_policy_weights(dims, "bf16", 11)
    g = np.random.default_rng(12)
    obs = g.standard_normal((M, dims[0])).astype(np.float32)
    d_out = (g.standard_normal((M, dims[-1])) / M).astype(np.float32)
    tr = T.MlpTrainer(dims, pw["W"], pw["b"], max_rows=M + 64)
    rows = tr.input_rows(M)
    rows.zero_()
    rows[:, :dims[0]] = torch.from_numpy(obs).cuda().to(torch.bfloat16)
    out = tr.forward(M)
    want = O.policy_forward(dims, pw["W"], pw["b"], 1.0, 0, 0, obs.astype(np.float64), bf16_operands=True)["mean"]
    close(out.cpu().numpy(), want, 2e-2, "training forward")
    tr.backward(torch.from_numpy(d_out).cuda(), M)
    torch.cuda.synchronize()
    assert tr.device_status() == 0
    dW, db = O.mlp_backward(dims, pw["W"], pw["b"], obs.astype(np.float64), d_out.astype(np.float64), bf16_operands=True)
    for l in range(len(dims) - 1):
        close(tr.dW[l].cpu().numpy(), dW[l], 2e-2, "dW[%d]" % l)
        close(tr.db[l].cpu().numpy(), db[l], 2e-2, "db[%d]" % l)
    # optimiser step from the kernel's own gradients: new fp32 weights, bf16 copies and transposes
    grads = [x.cpu().numpy().copy() for x in tr.grads()]
    ws, sc = B.ppo_workspace(), torch.empty(2, device="cuda")
    B.grad_scale(tr.grads(), 1e-3, sc, ws)
    lr = torch.tensor([5e-4], device="cuda")
    W0 = [w.cpu().numpy().copy() for w in tr.W]
    b0 = [x.cpu().numpy().copy() for x in tr.b]
    tr.step(lr, sc)
    torch.cuda.synchronize()
    scale = O.grad_scale(grads, 1e-3)
    np.testing.assert_allclose(sc[0].item(), scale, rtol=1e-5)
    assert scale < 1.0
    f = lambda x: float(np.float32(x))
    for l in range(len(dims) - 1):
        N, K = dims[l + 1], dims[l]
        w, m, v = W0[l].copy(), np.zeros_like(W0[l]), np.zeros_like(W0[l])
        O.adam_step(w, grads[l], m, v, f(5e-4), 1, f(0.9), f(0.999), f(1e-8), f(sc[0].item()))
        np.testing.assert_allclose(tr.W[l].cpu().numpy(), w, rtol=2e-6, atol=2e-9)
        assert torch.equal(tr.Wb[l][:N, :K], tr.W[l].to(torch.bfloat16))
        assert torch.equal(tr.WbT[l], tr.Wb[l].t())
        assert (tr.Wb[l][N:] == 0).all() and (tr.Wb[l][:, K:] == 0).all()
        bb, m, v = b0[l][:N].copy(), np.zeros(N, np.float32), np.zeros(N, np.float32)
        O.adam_step(bb, grads[len(dims) - 1 + l], m, v, f(5e-4), 1, f(0.9), f(0.999), f(1e-8), f(sc[0].item()))
        np.testing.assert_allclose(tr.b[l][:N].cpu().numpy(), bb, rtol=2e-6, atol=2e-9)
    # the updated net runs: a second forward differs from the first
    out2 = tr.forward(M).clone()
    torch.cuda.synchronize()
    assert not torch.equal(out2, torch.from_numpy(want.astype(np.float32)).cuda())


def test_ppo_update_matches_the_oracle_pipeline_and_improves_the_objective():
    """One whole minibatch update (both nets, loss, clip, Adam, learning rate) against the same
    pipeline assembled from oracle functions; then a few more updates on the same minibatch must
    lower the loss (the update does what an optimiser step is for)."""
    from tests.test_gpu_trainer import close as _close
    A, D, M = 28, 361, 512
    adims, cdims = (D, 128, 64, A), (D, 128, 64, 1)
    aw, cw = W.make_policy_weights(adims, "bf16", 21), W.make_policy_weights(cdims, "bf16", 22)
    g = np.random.default_rng(23)
    obs = g.standard_normal((M, D)).astype(np.float32)
    actor, critic = T.MlpTrainer(adims, aw["W"], aw["b"], M), T.MlpTrainer(cdims, cw["W"], cw["b"], M)
    log_std0 = np.full(A, -1.0, np.float32)
    up = T.PpoUpdater(actor, critic, torch.from_numpy(log_std0), lr=5e-4, clip=0.2, value_coef=2.0, entropy_coef=2.5e-4,
                      max_grad_norm=1.0, kl_target=0.008)
    for tr in (actor, critic):
        rows = tr.input_rows(M)
        rows.zero_()
        rows[:, :D] = torch.from_numpy(obs).cuda().to(torch.bfloat16)
    # behaviour data: the current nets' outputs are the "old" policy, actions sampled around them
    mean_old = O.policy_forward(adims, aw["W"], aw["b"], 1.0, 0, 0, obs.astype(np.float64), bf16_operands=True)["mean"]
    value_old = O.policy_forward(cdims, cw["W"], cw["b"], 1.0, 0, 0, obs.astype(np.float64), bf16_operands=True)["mean"][:, 0]
    z = g.standard_normal((M, A))
    action = (mean_old + np.exp(-1.0) * z).astype(np.float32)
    logp_old = (-0.5 * (z ** 2).sum(1) - A * (-1.0) - 0.5 * A * np.log(2 * np.pi)).astype(np.float32)
    batch_np = dict(action=action, mean_old=mean_old.astype(np.float32), log_std_old=log_std0, logp_old=logp_old,
                    advantage=(g.standard_normal(M) * 2 + 0.5).astype(np.float32), value_old=value_old.astype(np.float32),
                    returns=(value_old + g.standard_normal(M)).astype(np.float32))
    batch = {k: torch.from_numpy(v).cuda() for k, v in batch_np.items()}
    up.update(M, batch)
    torch.cuda.synchronize()
    assert actor.device_status() == 0 and critic.device_status() == 0
    # oracle pipeline on the same inputs
    am, ar = O.moments(batch_np["advantage"])
    ob = dict(batch_np, mean=mean_old.astype(np.float32), log_std=log_std0, value=value_old.astype(np.float32))
    loss = O.ppo_loss(ob, 0.2, 2.0, 2.5e-4, True, am, ar)
    s = up.summary.cpu().numpy()
    np.testing.assert_allclose(s[:4], loss["summary"][:4], rtol=2e-2, atol=2e-3)       # bf16 nets: forward differs by ~1e-2
    dWa, dba = O.mlp_backward(adims, aw["W"], aw["b"], obs.astype(np.float64), loss["d_mean"], bf16_operands=True)
    for l in range(3):
        _close(actor.dW[l].cpu().numpy(), dWa[l], 5e-2, "actor dW[%d] through the whole pipeline" % l)
    assert 0.0 < up.scale[0].item() <= 1.0 and up.scale[1].item() > 0.0
    assert up.lr.item() == pytest.approx(5e-4 * 1.5, rel=1e-5)          # KL of the first update is ~0: the rate goes up
    first = float(s[0])
    for _ in range(8):
        up.update(M, batch)
    torch.cuda.synchronize()
    assert float(up.summary[0].item()) < first
    assert np.isfinite(up.log_std.cpu().numpy()).all()


def test_whole_training_iteration_runs_from_one_cuda_graph():
    """Rollout (policy forward, critic, env step into storage), GAE and the PPO update epochs enqueued
    back to back with no host read in between; the same sequence captured in one CUDA graph and
    replayed from the same starting state reproduces every number bit for bit."""
    from paper_2609_09821_b200 import rollout as R
    wl = W.WORKLOADS["cfg3_16384_lib32"]
    skel, lib, pol = W.build_scene(wl)
    n, Tn, A, D = 256, 4, wl.act_dim, wl.obs_dim
    ld = B.padded_ld(D)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        gs = B.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
        gc = B.Clips(gs, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
        env = B.Env(gs, gc, B.make_env_config(n, wl.dt, 0, W.REWARD_MULT, W.ROOT_HEIGHT, ld), stream=stream)
        cdims = tuple(wl.mlp_dims[:-1]) + (1,)
        cw = W.make_policy_weights(cdims, "bf16", 5)
        actor_t = T.MlpTrainer(wl.mlp_dims, pol["W"], pol["b"], 256, stream=stream)
        critic_t = T.MlpTrainer(cdims, cw["W"], cw["b"], 256, stream=stream)
        upd = T.PpoUpdater(actor_t, critic_t, torch.full((A,), -2.0), lr=5e-4)
        actor = B.Policy(wl.mlp_dims, pol["W_bf16"], pol["b"], "bf16", 0.1, 0, n, stream=stream)
        critic = B.Policy(cdims, cw["W_bf16"], cw["b"], "bf16", 1.0, 0, n, stream=stream)
        actor.set_log_std(upd.log_std)
        st = R.RolloutStorage(Tn, n, A, ld, keep_obs=True)
        env.reset_all(st.obs_row(0), 0)
        c, t, _ = env.get_state()
        sims = {s: W.synth_sim_state_torch(skel, lib, c.long(), t.double() + wl.dt * s, s, wl) for s in range(1, Tn + 1)}
        state0 = [x.clone() for x in env.get_state()]
        obs0 = st.obs_row(0).clone()
        probe_mean, probe_act = torch.empty((n, A), device="cuda"), torch.empty((n, A), device="cuda")
        before_mean = torch.empty((n, A), device="cuda")
        actor.forward(99, st.obs_row(0), before_mean, probe_act)

        def iteration():
            R.collect(env, actor, critic, st, lambda s: sims[s], 1, 0.99, 0.95)
            T.update_from_storage(upd, st, epochs=2, n_minibatches=4)
            actor_t.push_to_policy(actor)                          # the next rollout acts with the trained nets
            critic_t.push_to_policy(critic)
            actor.set_log_std(upd.log_std)
            actor.forward(99, st.obs_row(0), probe_mean, probe_act)

        def snapshot():
            return [x.clone() for x in (st.advantage, st.returns, st.reward, upd.summary, upd.lr, upd.log_std,
                                        actor_t.W[0], actor_t.W[-1], critic_t.W[1], actor_t.mW[0], probe_mean)]

        def restore(tr0):
            env.set_state(*state0)
            st.obs_row(0).copy_(obs0)
            for tr, saved in zip((actor_t, critic_t), tr0):
                for dst, src in zip(tr.W + tr.b + tr.mW + tr.vW + tr.mb + tr.vb + tr.Wb + tr.WbT, saved):
                    dst.copy_(src)
                tr.set_step_count(0)
            upd.set_step_count(0)
            upd.lr.fill_(5e-4); upd.log_std.fill_(-2.0); upd.m_ls.zero_(); upd.v_ls.zero_()
            actor_t.push_to_policy(actor); critic_t.push_to_policy(critic); actor.set_log_std(upd.log_std)

        saved = [[x.clone() for x in tr.W + tr.b + tr.mW + tr.vW + tr.mb + tr.vb + tr.Wb + tr.WbT] for tr in (actor_t, critic_t)]
        iteration()
        stream.synchronize()
        eager = snapshot()
        assert all(torch.isfinite(x).all() for x in eager)
        assert not torch.equal(eager[6], saved[0][0])             # the actor's first layer moved
        assert not torch.equal(eager[10], before_mean)            # and the rollout policy acts differently now
        # the pushed weights are the trainer's: the policy's means equal the trainer's own forward
        rows = actor_t.input_rows(n)
        B.f32_to_bf16_padded(st.obs_row(0)[:, :D], rows, stream)
        assert torch.equal(actor_t.forward(n), eager[10])
        restore(saved)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            iteration()
        restore(saved)                                             # capture itself does not run anything
        graph.replay()
        stream.synchronize()
        for a, b in zip(eager, snapshot()):
            assert torch.equal(a, b)
        assert env.device_status() == 0 and actor_t.device_status() == 0 and critic_t.device_status() == 0


@pytest.mark.parametrize("R,Mo,No,slices", [(128, 64, 64, 1), (256, 128, 128, 2), (1024, 200, 256, 4), (512, 69, 512, 2),
                                             (2048, 1024, 640, 4), (512, 128, 320, 2),
                                             (8192, 1024, 1024, 8), (16384, 512, 640, 16), (4096, 1024, 512, 8)])
def test_transposed_product_reads_both_operands_in_place(R, Mo, No, slices):
    """A^T B of two row-major bf16 matrices on the tensor cores (operands M/N-major), per row slice; the last
    three shapes have enough 256 x 256 tiles for the CTA-pair kernel (one of them with a ragged last tile)."""
    g = np.random.default_rng(R + Mo)
    a = W.round_to_bf16(g.standard_normal((R, Mo)).astype(np.float32))[0]
    b = W.round_to_bf16((g.standard_normal((R, No)) / 8).astype(np.float32))[0]
    lda = (Mo + 7) // 8 * 8
    A_ = torch.zeros((R, lda), dtype=torch.bfloat16, device="cuda")
    A_[:, :Mo] = torch.from_numpy(a).cuda().to(torch.bfloat16)
    B_ = torch.from_numpy(b).cuda().to(torch.bfloat16)
    pitch = (Mo + 127) // 128 * 128
    C_ = torch.full((slices * pitch, No), 5.0, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gemm_bf16_tn(A_[:, :Mo], B_, C_, slices, pitch, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    Rs = R // slices
    got = C_.float().cpu().numpy().reshape(slices, pitch, No)
    for s in range(slices):
        want = a[s * Rs:(s + 1) * Rs].astype(np.float64).T @ b[s * Rs:(s + 1) * Rs].astype(np.float64)
        assert np.abs(got[s, :Mo] - want).max() <= 2.0 ** -8 * np.abs(want).max() + 1e-3, "slice %d" % s


def test_row_gather_is_exact_and_flags_bad_indices():
    g = torch.Generator().manual_seed(3)
    x = torch.randn((5000, 361), generator=g).cuda()
    v = torch.randn(5000, generator=g).cuda()
    idx = torch.randperm(5000, generator=g)[:1234].to(torch.int32).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((1234, 361), 7.0, device="cuda")
    B.gather_rows(x, idx, out, status)
    assert torch.equal(out, x[idx.long()])
    out1 = torch.empty(1234, device="cuda")
    B.gather_rows(v, idx, out1, status)
    assert torch.equal(out1, v[idx.long()])
    ob = torch.full((1234, 384), 7.0, dtype=torch.bfloat16, device="cuda")
    B.gather_rows(x, idx, ob, status)
    assert torch.equal(ob[:, :361], x[idx.long()].to(torch.bfloat16)) and not ob[:, 361:].any()
    assert int(status.item()) == 0
    bad = idx.clone(); bad[5] = 5000; bad[9] = -1
    B.gather_rows(x, bad, out, status)
    assert int(status.item()) != 0                                   # clamped and reported, nothing read out of range
    assert torch.equal(out[5], x[4999]) and torch.equal(out[9], x[0]) and torch.equal(out[10], x[idx[10].long()])


def test_shuffled_minibatches_equal_contiguous_ones_on_permuted_data():
    """update_from_storage with a permutation visits sample perm[k] where the contiguous path visits
    sample k: run on the permutation and on explicitly permuted arrays, the two leave the same bits."""
    from types import SimpleNamespace
    dims, cdims, Tn, n = (61, 128, 64, 12), (61, 128, 64, 1), 4, 128
    A, D, total = dims[-1], dims[0], Tn * n
    ld = B.padded_ld(D)
    g = torch.Generator().manual_seed(11)
    rnd = lambda *sh: torch.randn(*sh, generator=g).cuda()
    base = SimpleNamespace(T=Tn, N=n, A=A, keep_obs=True, ld_obs=ld, obs=rnd(Tn + 1, n, ld), action=rnd(Tn, n, A),
                           mean=rnd(Tn, n, A) * 0.1, logp=rnd(Tn, n) - 5.0, advantage=rnd(Tn, n), returns=rnd(Tn, n),
                           value=rnd(Tn + 1, n))
    perm = torch.stack([torch.randperm(total, generator=g) for _ in range(2)]).to(torch.int32).cuda()

    def fresh():
        aw, cw = W.make_policy_weights(dims, "bf16", 2), W.make_policy_weights(cdims, "bf16", 3)
        return T.PpoUpdater(T.MlpTrainer(dims, aw["W"], aw["b"], 256), T.MlpTrainer(cdims, cw["W"], cw["b"], 256),
                            torch.full((A,), -1.0), lr=1e-3)

    up1 = fresh()
    T.update_from_storage(up1, base, epochs=2, n_minibatches=2, perm=perm)
    up2 = fresh()
    for ep in range(2):
        p = perm[ep].long()
        take = lambda x, *tail: x.reshape(total, *tail)[p].reshape(Tn, n, *tail).contiguous()
        obs = base.obs.clone(); obs[:Tn] = take(base.obs[:Tn], ld)
        val = base.value.clone(); val[:Tn] = take(base.value[:Tn])
        shuffled = SimpleNamespace(T=Tn, N=n, A=A, keep_obs=True, ld_obs=ld, obs=obs, action=take(base.action, A),
                                   mean=take(base.mean, A), logp=take(base.logp), advantage=take(base.advantage),
                                   returns=take(base.returns), value=val)
        T.update_from_storage(up2, shuffled, epochs=1, n_minibatches=2)
    torch.cuda.synchronize()
    for a, b in zip(up1.actor.W + up1.critic.W + [up1.log_std, up1.lr, up1.summary],
                    up2.actor.W + up2.critic.W + [up2.log_std, up2.lr, up2.summary]):
        assert torch.equal(a, b)
    assert up1.actor.device_status() == 0
    with pytest.raises(ValueError):
        T.update_from_storage(up1, base, epochs=2, n_minibatches=2, perm=perm.long())


@pytest.mark.parametrize("M,N,K", [(64, 64, 64), (320, 128, 192), (1024, 256, 128), (37888 + 64, 512, 1024), (40000 - 32, 1024, 512)])
def test_dgrad_product_masks_and_sums_in_its_epilogue(M, N, K):
    """im_gemm_bf16_dgrad against the three separate steps it replaces, in exact arithmetic: small integer
    operands make every product and sum exact, so the fused output and its 32-row column sums must
    equal dZ @ Wt^T masked by H > 0 bit for bit (single-CTA and CTA-pair kernels, ragged last tiles)."""
    g = torch.Generator().manual_seed(M + N)
    dz = torch.randint(-2, 3, (M, K), generator=g).to(torch.bfloat16).cuda()
    wt = torch.randint(-2, 3, (N, K), generator=g).to(torch.bfloat16).cuda()
    h = torch.randint(-1, 3, (M, N), generator=g).clamp(min=0).to(torch.bfloat16).cuda()
    h[0, :] = 0; h[:, 1] = 0; h[3, 5] = -0.0
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    want = (dz.float() @ wt.float().T) * (h > 0)
    for use_mask, use_sum in ((True, True), (True, False), (False, True)):
        out = torch.full((M, N), 7.0, dtype=torch.bfloat16, device="cuda")
        part = torch.full((M // 32, N + 2), 7.0, device="cuda")
        B.gemm_bf16_dgrad(dz, wt, out, h if use_mask else None, part if use_sum else None, status)
        ref = want if use_mask else dz.float() @ wt.float().T
        assert torch.equal(out.float(), ref.to(torch.bfloat16).float())
        if use_sum:
            assert torch.equal(part[:, :N], ref.view(M // 32, 32, N).sum(1))
            assert (part[:, N:] == 7.0).all()
        else:
            assert (part == 7.0).all()
    assert int(status.item()) == 0


def test_whole_ppo_update_through_the_raw_c_abi():
    """One PPO minibatch update driven by lib.im_* calls alone (no Python wrapper classes in between): trainers
    and updater created, input rows filled, im_ppo_update enqueued, gradients and the loss summary read back
    through im_trainer_tensor / im_ppo_updater_tensor and compared with the pipeline assembled from oracle
    functions, as test_ppo_update_matches_the_oracle_pipeline_and_improves_the_objective does through the wrappers."""
    import ctypes as C
    lib = B.load()
    A, D, M = 28, 361, 256
    adims, cdims = (D, 128, 64, A), (D, 128, 64, 1)
    aw, cw = W.make_policy_weights(adims, "bf16", 31), W.make_policy_weights(cdims, "bf16", 32)
    g = np.random.default_rng(33)
    obs = g.standard_normal((M, D)).astype(np.float32)
    stream = torch.cuda.current_stream().cuda_stream

    def create(dims, w):
        nl = len(dims) - 1
        Wc = [np.ascontiguousarray(x, np.float32) for x in w["W"]]
        bc = [np.ascontiguousarray(x, np.float32) for x in w["b"]]
        Wp = (C.c_void_p * nl)(*[x.ctypes.data for x in Wc])
        bp = (C.c_void_p * nl)(*[x.ctypes.data for x in bc])
        d = np.asarray(dims, np.int32)
        h = C.c_void_p()
        assert lib.im_trainer_create(nl, d.ctypes.data, C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p), M, stream, C.byref(h)) == 0
        return h

    def tensor(h, which, layer):
        ptr, rows, cols, ld, dt = C.c_void_p(), C.c_int64(), C.c_int64(), C.c_int64(), C.c_int32()
        assert lib.im_trainer_tensor(h, which, layer, C.byref(ptr), C.byref(rows), C.byref(cols), C.byref(ld), C.byref(dt)) == 0
        vector = which in (1, 6, 7, 9, 12)
        shape = (cols.value,) if vector else (rows.value, cols.value)
        return B.device_tensor(ptr.value, shape, {0: "f32", 1: "bf16", 2: "u32"}[dt.value], None if vector else ld.value)

    actor, critic = create(adims, aw), create(cdims, cw)
    log_std0 = np.full(A, -1.0, np.float32)
    cfg = B.PpoUpdateConfig(5e-4, 0.2, 2.0, 2.5e-4, 1, 1.0, 0.008, 1e-5, 1e-2, 1, B.AdamConfig(0.9, 0.999, 1e-8))
    upd = C.c_void_p()
    assert lib.im_ppo_updater_create(actor, critic, log_std0.ctypes.data, C.byref(cfg), C.byref(upd)) == 0
    for h in (actor, critic):
        rows = tensor(h, 10, 0)                                   # IM_TRAINER_H of layer 0: the input rows
        rows.zero_()
        rows[:M, :D] = torch.from_numpy(obs).cuda().to(torch.bfloat16)
    mean_old = O.policy_forward(adims, aw["W"], aw["b"], 1.0, 0, 0, obs.astype(np.float64), bf16_operands=True)["mean"]
    value_old = O.policy_forward(cdims, cw["W"], cw["b"], 1.0, 0, 0, obs.astype(np.float64), bf16_operands=True)["mean"][:, 0]
    z = g.standard_normal((M, A))
    batch_np = dict(action=(mean_old + np.exp(-1.0) * z).astype(np.float32), mean_old=mean_old.astype(np.float32),
                    logp_old=(-0.5 * (z ** 2).sum(1) + A - 0.5 * A * np.log(2 * np.pi)).astype(np.float32),
                    advantage=(g.standard_normal(M) * 2 + 0.5).astype(np.float32), value_old=value_old.astype(np.float32),
                    returns=(value_old + g.standard_normal(M)).astype(np.float32))
    dev = {k: torch.from_numpy(v).cuda() for k, v in batch_np.items()}
    mb = B.PpoMinibatch(dev["action"].data_ptr(), dev["mean_old"].data_ptr(), None, dev["logp_old"].data_ptr(),
                        dev["advantage"].data_ptr(), dev["value_old"].data_ptr(), dev["returns"].data_ptr())
    assert lib.im_ppo_update(upd, M, C.byref(mb)) == 0
    assert lib.im_ppo_update(upd, M + 1, C.byref(mb)) == -1                    # rows not a multiple of 64
    torch.cuda.synchronize()
    assert int(tensor(actor, 12, 0).item()) == 0 and int(tensor(critic, 12, 0).item()) == 0
    am, ar = O.moments(batch_np["advantage"])
    ob = dict(batch_np, mean=mean_old.astype(np.float32), log_std=log_std0, log_std_old=log_std0, value=value_old.astype(np.float32))
    loss = O.ppo_loss(ob, 0.2, 2.0, 2.5e-4, True, am, ar)
    ptr, n = C.c_void_p(), C.c_int64()
    assert lib.im_ppo_updater_tensor(upd, 6, C.byref(ptr), C.byref(n)) == 0 and n.value == 6     # IM_PPO_SUMMARY
    summary = B.device_tensor(ptr.value, (6,), "f32").cpu().numpy()
    np.testing.assert_allclose(summary[:4], loss["summary"][:4], rtol=2e-2, atol=2e-3)
    dWa, dba = O.mlp_backward(adims, aw["W"], aw["b"], obs.astype(np.float64), loss["d_mean"], bf16_operands=True)
    dWc, dbc = O.mlp_backward(cdims, cw["W"], cw["b"], obs.astype(np.float64), loss["d_value"][:, None], bf16_operands=True)
    for l in range(3):
        close(tensor(actor, 8, l).cpu().numpy(), dWa[l], 5e-2, "actor dW[%d]" % l)                 # IM_TRAINER_DW
        close(tensor(actor, 9, l).cpu().numpy(), dba[l], 5e-2, "actor db[%d]" % l)                 # IM_TRAINER_DB
        close(tensor(critic, 8, l).cpu().numpy(), dWc[l], 5e-2, "critic dW[%d]" % l)
    # the step moved the weights and the bf16 copies follow the fp32 masters
    for l in range(3):
        w, wb = tensor(actor, 0, l), tensor(actor, 2, l)
        assert not torch.equal(w.cpu(), torch.from_numpy(np.ascontiguousarray(aw["W"][l], np.float32)))
        assert torch.equal(wb[:adims[l + 1], :adims[l]], w.to(torch.bfloat16))
    lib.im_ppo_updater_destroy(upd)
    lib.im_trainer_destroy(actor)
    lib.im_trainer_destroy(critic)
