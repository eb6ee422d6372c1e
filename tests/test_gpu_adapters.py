"""The adapter-side entry points on the GPU against their oracle: the KV-layout writer is a bit-exact gather, the
action post-processing float32 arithmetic (one fused multiply-add per element: 1e-6 relative)."""
import numpy as np
import pytest
import torch

from oracle import adapter_oracle as A
from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,L,B,p_max,Hkv,dh", [(torch.bfloat16, 3, 5, 70, 1, 256), (torch.float32, 2, 4, 33, 2, 24),
                                                      (torch.bfloat16, 18, 8, 968, 1, 256)])
def test_kv_layout_writer_is_a_bit_exact_ragged_gather(dtype, L, B, p_max, Hkv, dh):
    g = torch.Generator().manual_seed(7)
    k = torch.randn(L, B, p_max, Hkv, dh, generator=g).to(dtype)
    v = torch.randn(L, B, p_max, Hkv, dh, generator=g).to(dtype)
    lens = synth.make_ragged_lengths(41, B, 0, p_max)
    lens[0], lens[-1] = 0, p_max                                    # an empty request and a full one
    as_bits = (lambda t: t.view(torch.int16).numpy()) if dtype == torch.bfloat16 else (lambda t: t.numpy())
    ref, cu_ref = A.pack_prefix_kv(as_bits(k), as_bits(v), lens)
    total = int(cu_ref[-1])
    out, cu, status = binding.pack_prefix_kv(k.cuda(), v.cuda(), torch.from_numpy(lens).cuda(), kv_tokens=total + 3)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert cu.cpu().numpy().tolist() == cu_ref.tolist()
    got = as_bits(out.cpu())
    assert np.array_equal(got[:, :, :total], ref)
    assert not got[:, :, total:].any()                              # rows past the last request stay untouched


def test_kv_layout_writer_feeds_the_denoising_call():
    """Packed by the writer, the prefix KV gives the same actions as the host-side packing of the synthetic inputs."""
    from tests.helpers import small_bf16_config
    cfg = small_bf16_config("pi0", max_batch=3, max_prefix_len=90)
    W = synth.make_weights(cfg, 24, std=0.05)
    lens = np.array([90, 0, 37], dtype=np.int32)
    kvs = [synth.make_prefix_kv(cfg, 24, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    padded = torch.zeros(cfg.n_layers, 2, 3, 90, cfg.n_kv_heads, cfg.head_dim, dtype=torch.bfloat16)
    for b, kv in enumerate(kvs):
        padded[:, :, b, : kv.shape[2]] = kv
    out, cu_d, status = binding.pack_prefix_kv(padded[:, 0].contiguous().cuda(), padded[:, 1].contiguous().cuda(),
                                               torch.from_numpy(lens).cuda(), kv_tokens=int(cu[-1]))
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(out.cpu(), packed)
    states = torch.stack([synth.make_state(cfg, 24, b) for b in range(3)]).cuda()
    noise = torch.stack([synth.make_noise(cfg, 24, b) for b in range(3)]).cuda()
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        a = ex.denoise_batched(out, cu_d, states, noise, 3).clone()
        b2 = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), states, noise, 3).clone()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0 and torch.equal(a, b2)


def test_kv_layout_writer_reports_bad_lengths_on_the_device():
    k = torch.zeros(1, 2, 8, 1, 64, dtype=torch.bfloat16).cuda()
    for lens in ([3, 9], [-1, 2]):
        out, cu, status = binding.pack_prefix_kv(k, k, torch.tensor(lens, dtype=torch.int32).cuda(), kv_tokens=16)
        torch.cuda.synchronize()
        assert int(status.item()) == binding.ERR_INVALID_ARG and not out.any()
    out, cu, status = binding.pack_prefix_kv(k, k, torch.tensor([8, 8], dtype=torch.int32).cuda(), kv_tokens=15)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.ERR_INVALID_ARG            # does not fit the output buffer
    with pytest.raises(binding.PhyaiError):
        binding.pack_prefix_kv(torch.zeros(1, 1, 4, 1, 4, dtype=torch.bfloat16).cuda(),   # 8-byte rows
                               torch.zeros(1, 1, 4, 1, 4, dtype=torch.bfloat16).cuda(), torch.tensor([1], dtype=torch.int32).cuda())


def test_action_postprocessing_matches_oracle():
    g = torch.Generator().manual_seed(9)
    x = torch.randn(6, 50, 32, generator=g) * 1.3
    q01, q99 = -torch.rand(32, generator=g) * 3 - 0.1, torch.rand(32, generator=g) * 3 + 0.1
    for kw in (dict(), dict(out_horizon=32, out_dim=14), dict(clip=None)):
        ref = A.postprocess_actions(x.numpy(), q01.numpy(), q99.numpy(), **kw)
        got = binding.postprocess_actions(x.cuda(), q01.cuda(), q99.cuda(), **kw).cpu().numpy()
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=1e-6, atol=1e-6)
    got = binding.postprocess_actions(x.cuda(), None, None, clip=(-1.0, 1.0)).cpu().numpy()
    np.testing.assert_allclose(got, np.clip(x.numpy(), -1, 1), rtol=0, atol=1e-7)


def test_frontend_worker_pads_the_local_batch_to_its_fixed_shape():
    """One rank: three requests into a fixed local batch of four.  The padded slot runs as a request with an empty
    prefix, its output is dropped; every real request matches the oracle."""
    from oracle import expert_oracle as O
    from paper_2608_03682_b200.frontend import DPFrontend, ExpertWorker
    from tests.helpers import BAR, rel_err, small_bf16_config
    cfg = small_bf16_config("pi0", max_batch=4, max_prefix_len=120)
    W = synth.make_weights(cfg, 25, std=0.05)
    reqs = [dict(prefix_kv=synth.make_prefix_kv(cfg, 25, p, b), state=synth.make_state(cfg, 25, b),
                 noise=synth.make_noise(cfg, 25, b), n_steps=3) for b, p in enumerate([120, 0, 57])]
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        fe = DPFrontend(ExpertWorker(ex, cfg, 3), local_batch=4, window_ms=5.0)
        ids = [fe.submit(r) for r in reqs]
        out = fe.serve_round(timeout_ms=500.0)
        assert sorted(out) == ids and fe.serve_round(timeout_ms=10.0) == {}
        fe.close()
    Wf = O.Weights(W)
    for rid, r in zip(ids, reqs):
        ref = O.denoise(cfg, Wf, r["prefix_kv"], r["prefix_kv"].shape[2], r["state"], r["noise"], 3)
        assert rel_err(out[rid], ref) <= BAR["bf16"], (rid, rel_err(out[rid], ref))


def test_two_workers_prepare_the_next_chunk_while_the_first_is_in_flight():
    """launch / collect: two handles on two streams, both batches enqueued before either is collected (the RTC
    schedule: the next chunk is prepared during the current execution window); results equal the blocking calls."""
    from paper_2608_03682_b200.frontend import ExpertWorker
    from tests.helpers import small_bf16_config
    cfg = small_bf16_config("pi0", max_batch=2, max_prefix_len=120)
    W = synth.make_weights(cfg, 26, std=0.05)
    mk = lambda b, p: dict(prefix_kv=synth.make_prefix_kv(cfg, 26, p, b), state=synth.make_state(cfg, 26, b),
                           noise=synth.make_noise(cfg, 26, b), n_steps=3)
    batch_a, batch_b = [mk(0, 120), mk(1, 33)], [mk(2, 77), None]
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex_a, binding.Expert(cfg, binding.weights_to_device(W)) as ex_b:
        wa, wb = ExpertWorker(ex_a, cfg, 3), ExpertWorker(ex_b, cfg, 3)
        pa = wa.launch(batch_a)
        pb = wb.launch(batch_b)                      # enqueued while the first batch is still running
        out_b, out_a = wb.collect(pb), wa.collect(pa)
        ref_a, ref_b = wa(batch_a), wb(batch_b)
    for got, ref in zip(out_a + out_b[:1], ref_a + ref_b[:1]):
        assert np.array_equal(got, ref)


# ------------------------------------------------------------------ feature-handoff head: request-local K / V projections
@pytest.mark.parametrize("tokens,feat_dim,n_kv,dh,layers", [(300, 512, 2, 128, 3), (37, 1024, 1, 256, 2), (1500, 256, 2, 64, 2)])
def test_feature_projection_matches_oracle(tokens, feat_dim, n_kv, dh, layers):
    cfg = synth.ExpertConfig(n_layers=layers, width=256, mlp_dim=512, n_q_heads=2 * n_kv, n_kv_heads=n_kv, head_dim=dh,
                             state_dim=4, action_dim=4, horizon=4, has_state_token=True, max_prefix_len=tokens, max_batch=1,
                             cond="pi0", dtype="bf16")
    F = synth.make_features(41, tokens, feat_dim)
    wk, wv = synth.make_kv_projections(cfg, 41, feat_dim)
    got = binding.project_features_kv(F.cuda(), [w.cuda() for w in wk], [w.cuda() for w in wv], n_kv, dh, kv_tokens=tokens + 5)
    torch.cuda.synchronize()
    ref = A.project_features_kv(F.double().numpy(), [w.double().numpy() for w in wk], [w.double().numpy() for w in wv], n_kv, dh)
    g = got.double().cpu().numpy()
    assert np.all(g[:, :, tokens:] == 0)                      # rows past `tokens` are left alone
    err = np.abs(g[:, :, :tokens] - ref)
    # bf16 storage of an fp32-accumulated product: half an ulp (2^-9 relative) plus accumulation noise
    assert np.all(err <= np.abs(ref) * 2.0 ** -8 + 1e-4), float(err.max())


@pytest.mark.parametrize("batch", [1, 3])
def test_feature_handoff_head_end_to_end(batch):
    """Projected features as the loop's prefix KV: the device projects and denoises (four steps, 40 x 132 chunk); the
    oracle projects in float64, stores bf16 and denoises.  Reduced depth so that the oracle stays fast."""
    cfg = synth.groot_like_config(max_batch=batch, n_layers=4, max_prefix_len=400)
    W = synth.make_weights(cfg, 42)
    feat_dim = 768
    wk, wv = synth.make_kv_projections(cfg, 42, feat_dim)
    lens = [400, 123, 256][:batch]
    feats = [synth.make_features(42, n, feat_dim, b) for b, n in enumerate(lens)]
    states = torch.stack([synth.make_state(cfg, 42, b) for b in range(batch)])
    noise = torch.stack([synth.make_noise(cfg, 42, b) for b in range(batch)])
    cu = np.zeros(batch + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    kv = binding.project_features_kv(torch.cat(feats).cuda(), [w.cuda() for w in wk], [w.cuda() for w in wv], cfg.n_kv_heads,
                                     cfg.head_dim)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = ex.denoise_batched(kv, torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 4)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        out = out.double().cpu().numpy()
    for b in range(batch):
        kv_ref = A.project_features_kv(feats[b].double().numpy(), [w.double().numpy() for w in wk],
                                       [w.double().numpy() for w in wv], cfg.n_kv_heads, cfg.head_dim)
        kv_ref = torch.from_numpy(kv_ref).to(torch.bfloat16)          # the layout stores bf16
        ref = O.denoise(cfg, W, kv_ref, lens[b], states[b], noise[b], 4)
        err = O.max_rel_err(out[b], ref)
        print(f"feature-handoff head, request {b}: max rel err {err:.2e}")
        assert err <= 2e-2, (b, err)


def test_projector_handle_gives_the_one_shot_result_for_every_token_count():
    cfg = synth.ExpertConfig(n_layers=3, width=256, mlp_dim=512, n_q_heads=4, n_kv_heads=2, head_dim=128, state_dim=4,
                             action_dim=4, horizon=4, has_state_token=True, max_prefix_len=700, max_batch=1, cond="pi0",
                             dtype="bf16")
    wk, wv = synth.make_kv_projections(cfg, 43, 512)
    wk, wv = [w.cuda() for w in wk], [w.cuda() for w in wv]
    with binding.KvProjector(wk, wv, 2, 128, max_tokens=700) as proj:
        for tokens in (700, 1, 64, 333):                      # one handle, shrinking and growing inputs
            F = synth.make_features(43, tokens, 512, request=tokens).cuda()
            a = proj.run(F)
            torch.cuda.synchronize()
            b = binding.project_features_kv(F, wk, wv, 2, 128)
            assert torch.equal(a, b), tokens
        with pytest.raises(binding.PhyaiError):
            proj.run(synth.make_features(43, 701, 512).cuda())
