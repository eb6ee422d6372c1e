"""GPU parity: the CUDA library (through the C ABI) against the float64 oracle on the same seeded
inputs.  Bars: max relative error on the final action chunk <= 1e-4 (fp32), <= 2e-2 (bf16 / e4m3)."""
import numpy as np
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth
from tests.helpers import BAR, elem_rel_err, gpu_single, rel_err, small_bf16_config, w8a8_bar

pytestmark = pytest.mark.gpu


def _inputs(cfg, cfg_id, P, request=0):
    kv = synth.make_prefix_kv(cfg, cfg_id, P, request)
    state = synth.make_state(cfg, cfg_id, request) if cfg.has_state_token else None
    noise = synth.make_noise(cfg, cfg_id, request)
    return kv, state, noise


# ------------------------------------------------------------------------------------------ C1
@pytest.mark.parametrize("use_graph", [True, False])
def test_tiny_fp32_config_matches_oracle(use_graph):
    cfg = synth.tiny_config()
    W = synth.make_weights(cfg, 1)
    kv, state, noise = _inputs(cfg, 1, 64)
    ref = O.denoise(cfg, W, kv, 64, state, noise, 4)
    got = gpu_single(cfg, W, kv, 64, state, noise, 4, use_graph=use_graph)
    assert rel_err(got, ref) <= BAR["f32"], rel_err(got, ref)


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("opts", [dict(), dict(rope_theta=0.0), dict(gelu_exact=True),
                                  dict(suffix_block_causal=True)])
def test_fp32_variants_match_oracle(cond, opts):
    cfg = synth.ExpertConfig(n_layers=2, width=96, mlp_dim=160, n_q_heads=4, n_kv_heads=2, head_dim=24, state_dim=5,
                             action_dim=7, horizon=9, has_state_token=True, max_prefix_len=40, cond=cond,
                             dtype="f32", **opts)
    W = synth.make_weights(cfg, 11, std=0.08)
    for P in (0, 1, 37):
        kv, state, noise = _inputs(cfg, 11, P)
        ref = O.denoise(cfg, W, kv, P, state, noise, 3)
        got = gpu_single(cfg, W, kv, P, state, noise, 3)
        assert rel_err(got, ref) <= BAR["f32"], (P, rel_err(got, ref))


# ------------------------------------------------------------------------------------------ bf16, reduced
@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_small_bf16_expert_matches_oracle(cond, engine):
    cfg = small_bf16_config(cond)
    W = synth.make_weights(cfg, 12, std=0.05)
    for P in (0, 77, 200):
        kv, state, noise = _inputs(cfg, 12, P)
        ref = O.denoise(cfg, W, kv, P, state, noise, 4)
        got = gpu_single(cfg, W, kv, P, state, noise, 4, engine=engine)
        bar = BAR["f32"] if engine == "simt" else BAR["bf16"]
        assert rel_err(got, ref) <= bar, (P, rel_err(got, ref))


@pytest.mark.parametrize("head_dim,n_q,n_kv", [(64, 4, 2), (256, 2, 1)])
def test_small_bf16_other_head_sizes_through_every_batch1_path(head_dim, n_q, n_kv):
    """head_dim 64 takes the fp32 QKV output (no rotary epilogue) into the cluster-merged attention, head_dim 256 the
    rotated bf16 operands (and, by default, the cluster split-K projections with folded norms); each also through
    the general GEMM kernel and through the split attention + merge kernels.  Prefix lengths: empty, shorter than
    one key tile, several tiles."""
    cfg = small_bf16_config("pi0", head_dim=head_dim, n_q_heads=n_q, n_kv_heads=n_kv, max_prefix_len=700)
    W = synth.make_weights(cfg, 18, std=0.05)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for P in (0, 41, 700):
            kv, state, noise = _inputs(cfg, 18, P)
            ref = O.denoise(cfg, W, kv, P, state, noise, 3)
            for opts in ({"use_cluster_attention": 1, "use_cluster_gemm": 1}, {"use_cluster_gemm": 0},
                         {"use_cluster_attention": 0}):
                for k, v in opts.items():
                    ex.set_option(k, v)
                got = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
                assert rel_err(got, ref) <= BAR["bf16"], (P, opts, rel_err(got, ref))


# ------------------------------------------------------------------------------------------ C2 / C3
@pytest.mark.parametrize("name", ["C2", "C3"])
def test_pi_shaped_bf16_batch1_matches_oracle(name):
    """Full-size batch-1 configurations through the default path (captured loop of cluster split-K projections with
    folded norms and cluster-merged attention), through the general GEMM kernel + norm kernels (attention with the
    output projection fused in, then with a separate output projection), and with the split attention + merge
    kernels."""
    wl = synth.WORKLOADS[name]
    cfg = synth.pi0_config() if name == "C2" else synth.pi05_config()
    W = synth.make_weights(cfg, wl["cfg_id"])
    kv, state, noise = _inputs(cfg, wl["cfg_id"], wl["prefix"])
    ref = O.denoise(cfg, W, kv, wl["prefix"], state, noise, wl["n_steps"])
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for label, opts in (("default", {}), ("general GEMM kernel", {"use_cluster_gemm": 0}),
                            ("separate output projection", {"use_fused_oproj": 0}),
                            ("split attention", {"use_fused_oproj": 1, "use_cluster_attention": 0})):
            for k, v in opts.items():
                ex.set_option(k, v)
            got = gpu_single(cfg, W, kv, wl["prefix"], state, noise, wl["n_steps"], expert=ex)
            err = rel_err(got, ref)
            print(f"{name} [{label}]: max rel err {err:.3e}, element-wise (floored) {elem_rel_err(got, ref):.3e}, "
                  f"||ref||inf {np.abs(ref).max():.3f}")
            assert err <= BAR["bf16"], (label, err)


@pytest.mark.parametrize("cond,horizon,block_causal", [("pi0", 50, False), ("pi0", 7, True), ("pi05", 55, False),
                                                       ("pi05", 16, False)])
def test_full_width_two_layer_expert_through_the_fused_attention_projection(cond, horizon, block_causal):
    """Width 1024, 8 heads of 256: the shapes for which the cluster attention kernel also applies the output
    projection.  Two layers keep the oracle fast; prefix lengths cover no prefix at all, key ranges without tiles,
    a ragged last tile and the maximum; suffix lengths cover owners without rows (8 rows), a full 8-row owner
    boundary (16 / 56 rows) and the usual 51.  Each case runs through the cluster split-K projections (default) and
    through the general GEMM kernel with the fused and with the separate output projection."""
    cfg = synth.ExpertConfig(n_layers=2, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256,
                             state_dim=32, action_dim=32, horizon=horizon, has_state_token=(cond == "pi0"),
                             max_prefix_len=968, max_batch=1, cond=cond, dtype="bf16",
                             suffix_block_causal=block_causal)
    W = synth.make_weights(cfg, 21)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for P in (0, 5, 130, 816, 968):
            kv, state, noise = _inputs(cfg, 21, P)
            ref = O.denoise(cfg, W, kv, P, state, noise, 3)
            for cluster_gemm, fused in ((1, 0), (0, 1), (0, 0)):
                ex.set_option("use_cluster_gemm", cluster_gemm)
                ex.set_option("use_fused_oproj", fused)
                got = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
                err = rel_err(got, ref)
                assert err <= BAR["bf16"], (P, cluster_gemm, fused, err)


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("block_causal", [False, True])
def test_full_width_several_short_requests_share_the_single_tile_path(cond, block_causal):
    """Width 1024 with several requests whose suffix tokens together fit one 64-token tile: the cluster kernels, the
    step-boundary kernel (token row -> request, action row) and the cluster attention kernel (two heads per CTA, since
    8 x heads x requests CTAs do not fit) all see more than one request; ragged prefixes including an empty one."""
    if block_causal and cond == "pi05":
        pytest.skip("the block-causal mask concerns the state token, which pi0.5 has not")
    cfg = synth.ExpertConfig(n_layers=2, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256,
                             state_dim=32, action_dim=32, horizon=11, has_state_token=(cond == "pi0"),
                             max_prefix_len=400, max_batch=4, cond=cond, dtype="bf16", suffix_block_causal=block_causal)
    lens = [400, 0, 33, 257]
    W = synth.make_weights(cfg, 24)
    kvs = [synth.make_prefix_kv(cfg, 24, p, b) if p else synth.make_prefix_kv(cfg, 24, 1, b)[:, :, :0] for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 24, b) for b in range(4)]) if cfg.has_state_token else None
    noise = torch.stack([synth.make_noise(cfg, 24, b) for b in range(4)])
    Wf = O.Weights(W)
    refs = [O.denoise(cfg, Wf, kvs[b], lens[b], None if states is None else states[b], noise[b], 3) for b in range(4)]
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for opts in ({}, {"use_state_cache": 1}, {"use_b1_step": 0}, {"b1_attn_hpc": 2}):
            for k, v in opts.items():
                ex.set_option(k, v)
            out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(),
                                     noise.cuda(), 3)
            torch.cuda.synchronize()
            assert ex.poll_status() == 0
            out = out.double().cpu().numpy()
            for b in range(4):
                assert rel_err(out[b], refs[b]) <= BAR["bf16"], (opts, b, rel_err(out[b], refs[b]))
            for k in opts:
                ex.set_option(k, 1 if k == "use_b1_step" else 0)


# ------------------------------------------------------------------------------------------ batched, ragged
def _batched_case(cfg, cfg_id, lens, n_steps, check, engine="auto", std=0.05):
    W = synth.make_weights(cfg, cfg_id, std=std)
    kvs = [synth.make_prefix_kv(cfg, cfg_id, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    B = len(lens)
    states = torch.stack([synth.make_state(cfg, cfg_id, b) for b in range(B)]) if cfg.has_state_token else None
    noise = torch.stack([synth.make_noise(cfg, cfg_id, b) for b in range(B)])
    with binding.Expert(cfg, binding.weights_to_device(W), engine=engine) as ex:
        out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(),
                                 noise.cuda(), n_steps)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        out = out.double().cpu().numpy()
        singles = {}
        for b in check:
            singles[b] = ex.denoise(kvs[b].cuda(), int(lens[b]), None if states is None else states[b].cuda(),
                                    noise[b].cuda(), n_steps).double().cpu().numpy()
        torch.cuda.synchronize()
    bar = BAR["f32"] if (cfg.dtype == "f32" or engine == "simt") else BAR["bf16"]
    Wf = O.Weights(W)
    for b in check:
        ref = O.denoise(cfg, Wf, kvs[b], int(lens[b]), None if states is None else states[b], noise[b], n_steps)
        assert rel_err(out[b], ref) <= bar, (b, rel_err(out[b], ref))
        # the batched call (general GEMM kernel beyond 64 tokens) and the single-request call (cluster split-K
        # kernel) round differently, so they agree with each other only to the same bar as with the oracle
        assert rel_err(out[b], singles[b]) <= bar, (b, rel_err(out[b], singles[b]))
    assert np.isfinite(out).all()


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
def test_small_bf16_ragged_batch_matches_oracle_per_request(cond):
    cfg = small_bf16_config(cond, max_batch=5)
    _batched_case(cfg, 13, [200, 0, 63, 64, 129], 3, check=[0, 1, 2, 3, 4])


def test_small_bf16_large_batch_uses_wide_tiles_and_unsplit_attention():
    cfg = small_bf16_config("pi0", max_batch=300, max_prefix_len=96)
    lens = synth.make_ragged_lengths(14, 300, 10, 96)
    order = np.argsort(lens)
    _batched_case(cfg, 14, lens, 2, check=[0, 299, int(order[0]), int(order[-1])])


@pytest.mark.parametrize("cond,dtype,head_dim,n_q", [("pi0", "bf16", 128, 2), ("pi0", "bf16", 256, 4), ("pi0", "w8e4m3", 128, 2),
                                                     ("pi0", "w8a8e4m3", 256, 4), ("pi05", "bf16", 256, 4), ("pi05", "w4a16", 128, 2)])
def test_persistent_tile_gemm_with_more_tiles_than_sms(cond, dtype, head_dim, n_q):
    """4200 tokens, MLP width 2048: the gate / up projection has 544 output tiles of 128 rows x 256 tokens (the
    q | k | v projection 204 with four heads of 256), so every CTA of the persistent kernel walks several tiles through
    both accumulators and around the stage ring.  Checked against the oracle on four requests and, over the whole
    batch, against the one-tile-per-CTA kernels."""
    cfg = small_bf16_config(cond, max_batch=300, max_prefix_len=96, mlp_dim=2048, head_dim=head_dim, n_q_heads=n_q,
                            dtype=dtype)
    lens = synth.make_ragged_lengths(16, 300, 10, 96)
    W = synth.make_weights(cfg, 16, std=0.05)
    kvs = [synth.make_prefix_kv(cfg, 16, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 16, b) for b in range(300)]) if cfg.has_state_token else None
    noise = torch.stack([synth.make_noise(cfg, 16, b) for b in range(300)])
    args = (packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(), noise.cuda(), 2)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = ex.denoise_batched(*args).double().cpu().numpy()
        assert ex.poll_status() == 0
        ex.set_option("use_persistent_gu", 0)
        ex.set_option("use_persistent_qkv", 0)
        plain = ex.denoise_batched(*args).double().cpu().numpy()
        assert ex.poll_status() == 0
    assert np.isfinite(out).all()
    Wf = O.Weights(W)
    for b in (0, 151, 299, int(np.argmax(lens))):
        st_b = None if states is None else states[b]
        ref = O.denoise(cfg, Wf, kvs[b], int(lens[b]), st_b, noise[b], 2)
        if dtype == "w8a8e4m3":
            bar, _ = w8a8_bar(cfg, Wf, kvs[b], int(lens[b]), st_b, noise[b], 2, ref)
        else:
            bar = BAR["bf16"]
        assert rel_err(out[b], ref) <= bar, (b, rel_err(out[b], ref), bar)
        assert rel_err(plain[b], ref) <= bar, (b, rel_err(plain[b], ref), bar)
    # the two kernels sum the same products in the same k order: they differ by the rounding of the epilogue only
    assert rel_err(out, plain) <= (BAR["bf16"] if dtype != "w8a8e4m3" else 0.15), rel_err(out, plain)


@pytest.mark.parametrize("batch", [5, 9, 20])
def test_tcgen05_attention_with_split_key_ranges_matches_oracle_and_the_unsplit_kernel(batch):
    """Few requests: the tcgen05 attention kernel splits every request's key tiles over up to 8 CTAs per head pair and a
    merge kernel combines the partial results.  Ragged prefixes from 0 (a single key tile: all ranges but one are
    empty) to 200 (four tiles); compared with the oracle per request and with the unsplit kernel."""
    cfg = small_bf16_config("pi0", max_batch=batch, max_prefix_len=200, head_dim=256, n_q_heads=4)
    lens = [0, 200, 63, 64, 129, 1, 65, 199, 128][:batch] + [int(x) for x in synth.make_ragged_lengths(17, max(0, batch - 9), 0, 200)]
    lens = lens[:batch]
    W = synth.make_weights(cfg, 17, std=0.05)
    kvs = [synth.make_prefix_kv(cfg, 17, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 17, b) for b in range(batch)])
    noise = torch.stack([synth.make_noise(cfg, 17, b) for b in range(batch)])
    args = (packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 3)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        n_split = ex.launches_per_call(batch, 3)
        out = ex.denoise_batched(*args).double().cpu().numpy()
        assert ex.poll_status() == 0
        n_split = ex.launches_per_call(batch, 3)
        ex.set_option("use_attn_splits", 0)
        plain = ex.denoise_batched(*args).double().cpu().numpy()
        assert ex.poll_status() == 0
        n_plain = ex.launches_per_call(batch, 3)
    # the split path adds one merge launch per layer and step (3 layers x 3 steps) where it is chosen
    assert n_split == n_plain + (9 if batch * 2 <= 148 // 4 else 0), (n_split, n_plain)
    Wf = O.Weights(W)
    for b in range(min(batch, 9)):
        ref = O.denoise(cfg, Wf, kvs[b], int(lens[b]), states[b], noise[b], 3)
        assert rel_err(out[b], ref) <= BAR["bf16"], (b, lens[b], rel_err(out[b], ref))
    assert rel_err(out, plain) <= BAR["bf16"], rel_err(out, plain)


def test_fp32_ragged_batch_matches_oracle_per_request():
    cfg = synth.ExpertConfig(n_layers=2, width=64, mlp_dim=96, n_q_heads=2, n_kv_heads=2, head_dim=16, state_dim=3,
                             action_dim=4, horizon=6, has_state_token=True, max_prefix_len=30, max_batch=4,
                             cond="pi0", dtype="f32")
    _batched_case(cfg, 15, [30, 0, 7, 19], 3, check=[0, 1, 2, 3], std=0.1)


def test_bad_cu_prefix_lens_is_reported_and_nothing_is_written():
    cfg = small_bf16_config("pi0", max_batch=2)
    W = synth.make_weights(cfg, 13, std=0.05)
    kv = synth.make_prefix_kv(cfg, 13, 50).cuda()
    noise = torch.stack([synth.make_noise(cfg, 13, b) for b in range(2)]).cuda()
    states = torch.stack([synth.make_state(cfg, 13, b) for b in range(2)]).cuda()
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = torch.full_like(noise, 7.0)
        ex.denoise_batched(kv, torch.tensor([0, 40, 30], dtype=torch.int32).cuda(), states, noise, 2, out=out)
        torch.cuda.synchronize()
        assert ex.poll_status() == binding.ERR_INVALID_ARG
        assert bool((out == 7.0).all())
        ex.denoise_batched(kv, torch.tensor([0, 20, 50], dtype=torch.int32).cuda(), states, noise, 2, out=out)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0 and bool(torch.isfinite(out).all())


# ------------------------------------------------------------------------------------------ kernel families
@pytest.mark.parametrize("cond", ["pi0", "pi05"])
def test_cluster_gemm_path_and_general_path_agree_and_are_reproducible(cond):
    """Calls of at most 64 suffix tokens run their projections on the cluster split-K kernel (norms folded in);
    the same requests through the general GEMM kernel + norm kernels (option use_cluster_gemm = 0) must match the
    oracle too, and both must give the same bits run to run (partial sums are added in a fixed order)."""
    cfg = small_bf16_config(cond, max_batch=4)
    W = synth.make_weights(cfg, 16, std=0.05)
    lens = [150, 0, 64, 33]
    kvs = [synth.make_prefix_kv(cfg, 16, p, b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 16, b) for b in range(4)]) if cfg.has_state_token else None
    noise = torch.stack([synth.make_noise(cfg, 16, b) for b in range(4)])
    Wf = O.Weights(W)
    refs = [O.denoise(cfg, Wf, kvs[b], lens[b], None if states is None else states[b], noise[b], 3) for b in range(4)]
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        args = (packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(), noise.cuda(), 3)
        outs = {}
        for mode in (1, 0):
            ex.set_option("use_cluster_gemm", mode)
            a = ex.denoise_batched(*args).clone()
            b2 = ex.denoise_batched(*args).clone()
            torch.cuda.synchronize()
            assert ex.poll_status() == 0
            assert torch.equal(a, b2)
            outs[mode] = a.double().cpu().numpy()
        for b in range(4):
            for mode in (1, 0):
                assert rel_err(outs[mode][b], refs[b]) <= BAR["bf16"], (mode, b, rel_err(outs[mode][b], refs[b]))


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
def test_small_e4m3_expert_decoded_in_the_kernel_matches_oracle_and_the_expanded_weights(cond):
    """e4m3 weights on the cluster split-K path are streamed as bytes and decoded to bf16 inside the kernel; the decode
    is exact, so the result must equal, bit for bit, the one obtained from the bf16 images made at create time."""
    cfg = small_bf16_config(cond, dtype="w8e4m3", max_prefix_len=300)
    W = synth.make_weights(cfg, 22, std=0.05)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for P in (0, 130, 300):
            kv, state, noise = _inputs(cfg, 22, P)
            ref = O.denoise(cfg, W, kv, P, state, noise, 3)
            outs = []
            for mode in (1, 0):
                ex.set_option("use_w8_inkernel", mode)
                got = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
                assert rel_err(got, ref) <= BAR["w8e4m3"], (P, mode, rel_err(got, ref))
                outs.append(got)
            assert np.array_equal(outs[0], outs[1]), P


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
def test_small_w8a8_expert_matches_oracle_single_and_batched(cond):
    """W8A8: per-token e4m3 activations and e4m3 weights on the FP8 tensor path (general kernels at every batch size);
    the oracle applies the same quantization rule ahead of the seven large projections."""
    cfg = small_bf16_config(cond, dtype="w8a8e4m3", max_prefix_len=300, max_batch=5)
    W = synth.make_weights(cfg, 23, std=0.05)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for P in (0, 1, 130, 300):
            kv, state, noise = _inputs(cfg, 23, P)
            ref = O.denoise(cfg, W, kv, P, state, noise, 3)
            got = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
            bar, d_q = w8a8_bar(cfg, W, kv, P, state, noise, 3, ref)
            print(f"w8a8 {cond} P={P}: {rel_err(got, ref):.2e} (quantization noise of the mode {d_q:.2e}, bar {bar:.2e})")
            assert rel_err(got, ref) <= bar, (P, rel_err(got, ref), bar)
        lens = [300, 0, 17, 129, 64]
        kvs = [synth.make_prefix_kv(cfg, 23, p, b) if p else synth.make_prefix_kv(cfg, 23, 1, b)[:, :, :0] for b, p in enumerate(lens)]
        packed, cu = synth.pack_prefix_kv(kvs)
        states = torch.stack([synth.make_state(cfg, 23, b) for b in range(5)]) if cfg.has_state_token else None
        noise = torch.stack([synth.make_noise(cfg, 23, b) for b in range(5)])
        out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(),
                                 noise.cuda(), 3)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        out = out.double().cpu().numpy()
        for b in range(5):
            ref = O.denoise(cfg, W, kvs[b], lens[b], None if states is None else states[b], noise[b], 3)
            bar, d_q = w8a8_bar(cfg, W, kvs[b], lens[b], None if states is None else states[b], noise[b], 3, ref)
            print(f"w8a8 {cond} batched request {b}: {rel_err(out[b], ref):.2e} (noise {d_q:.2e}, bar {bar:.2e})")
            assert rel_err(out[b], ref) <= bar, (b, rel_err(out[b], ref), bar)


@pytest.mark.parametrize("cond", ["pi0", "pi05"])
@pytest.mark.parametrize("engine", ["auto", "simt"])
def test_small_w4a16_expert_matches_oracle_single_and_batched(cond, engine):
    """W4A16: the seven large matrices as 4-bit integers (two output channels per byte) with per-channel scales;
    single requests (cluster split-K kernels), a ragged batch (general kernels) and the CUDA-core engine."""
    cfg = small_bf16_config(cond, dtype="w4a16", max_prefix_len=300, max_batch=5)
    W = synth.make_weights(cfg, 25, std=0.05)
    bar = BAR["f32"] if engine == "simt" else BAR["w4a16"]
    with binding.Expert(cfg, binding.weights_to_device(W), engine=engine) as ex:
        for P in (0, 130, 300):
            kv, state, noise = _inputs(cfg, 25, P)
            ref = O.denoise(cfg, W, kv, P, state, noise, 3)
            got = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
            assert rel_err(got, ref) <= bar, (P, rel_err(got, ref))
            if engine == "auto":
                # the cluster path streams the 4-bit codes and decodes them in the kernel (exactly): bit-equal to the
                # run on the bf16 images made at create
                ex.set_option("use_w8_inkernel", 0)
                again = gpu_single(cfg, W, kv, P, state, noise, 3, expert=ex)
                ex.set_option("use_w8_inkernel", 1)
                assert np.array_equal(got, again), P
        lens = [300, 0, 17, 129, 64]
        kvs = [synth.make_prefix_kv(cfg, 25, p, b) if p else synth.make_prefix_kv(cfg, 25, 1, b)[:, :, :0] for b, p in enumerate(lens)]
        packed, cu = synth.pack_prefix_kv(kvs)
        states = torch.stack([synth.make_state(cfg, 25, b) for b in range(5)]) if cfg.has_state_token else None
        noise = torch.stack([synth.make_noise(cfg, 25, b) for b in range(5)])
        out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), None if states is None else states.cuda(),
                                 noise.cuda(), 3)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        out = out.double().cpu().numpy()
        for b in range(5):
            ref = O.denoise(cfg, W, kvs[b], lens[b], None if states is None else states[b], noise[b], 3)
            assert rel_err(out[b], ref) <= bar, (b, rel_err(out[b], ref))


def test_single_request_after_a_ragged_batch_with_many_heads():
    """16 query heads of 256 select the request-per-CTA tcgen05 attention kernel even for one request; it walks the
    requests in an order that the batched call writes.  A single-request call on the same handle must reset it."""
    cfg = small_bf16_config("pi0", head_dim=256, n_q_heads=16, n_kv_heads=2, max_batch=3, max_prefix_len=150)
    W = synth.make_weights(cfg, 19, std=0.05)
    lens = [20, 150, 77]
    kvs = [synth.make_prefix_kv(cfg, 19, p, b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 19, b) for b in range(3)])
    noise = torch.stack([synth.make_noise(cfg, 19, b) for b in range(3)])
    Wf = O.Weights(W)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        out = ex.denoise_batched(packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 2)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        batched = out.double().cpu().numpy()
        single = gpu_single(cfg, W, kvs[2], lens[2], states[2], noise[2], 2, expert=ex)
    for b in range(3):
        ref = O.denoise(cfg, Wf, kvs[b], lens[b], states[b], noise[b], 2)
        assert rel_err(batched[b], ref) <= BAR["bf16"], (b, rel_err(batched[b], ref))
    ref = O.denoise(cfg, Wf, kvs[2], lens[2], states[2], noise[2], 2)
    assert rel_err(single, ref) <= BAR["bf16"], rel_err(single, ref)


def test_large_batch_tcgen05_attention_matches_oracle_and_the_mma_sync_kernel():
    """head_dim 256 and >= 100 head-pair CTAs select the tcgen05 attention kernel; ragged prefixes with
    empty, sub-tile, exact-tile and multi-tile lengths."""
    cfg = small_bf16_config("pi0", head_dim=256, max_batch=104, max_prefix_len=200)
    lens = synth.make_ragged_lengths(17, 104, 0, 200)
    lens[:6] = [0, 1, 63, 64, 65, 200]
    W = synth.make_weights(cfg, 17, std=0.05)
    kvs = [synth.make_prefix_kv(cfg, 17, int(p), b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 17, b) for b in range(104)])
    noise = torch.stack([synth.make_noise(cfg, 17, b) for b in range(104)])
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        args = (packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 2)
        tc = ex.denoise_batched(*args).double().cpu().numpy()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        ex.set_option("use_tc_attention", 0)
        legacy = ex.denoise_batched(*args).double().cpu().numpy()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
    assert np.isfinite(tc).all()
    Wf = O.Weights(W)
    for b in (0, 1, 2, 3, 4, 5, 50, 103):
        ref = O.denoise(cfg, Wf, kvs[b], int(lens[b]), states[b], noise[b], 2)
        assert rel_err(tc[b], ref) <= BAR["bf16"], (b, rel_err(tc[b], ref))
        assert rel_err(legacy[b], ref) <= BAR["bf16"], (b, rel_err(legacy[b], ref))



# ------------------------------------------------------------------------------------------ state-token caching
@pytest.mark.parametrize("shape", ["small", "full_width"])
def test_block_causal_state_token_is_cached_once_per_call(shape):
    """With the block-causal suffix mask the state token's per-layer key and value do not depend on x or t; single-tile
    calls compute them once per call (a pass over the state tokens alone) and run the loop on the action tokens.
    Same mathematics as the masked network: compared with the oracle, and with the uncached GPU path."""
    if shape == "small":
        cfg = small_bf16_config("pi0", suffix_block_causal=True, max_batch=3, max_prefix_len=300)
        cases, n = [[300], [0], [41, 0, 222]], 4
    else:
        cfg = synth.ExpertConfig(n_layers=2, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256,
                                 state_dim=32, action_dim=32, horizon=50, has_state_token=True, max_prefix_len=968,
                                 max_batch=1, cond="pi0", dtype="bf16", suffix_block_causal=True)
        cases, n = [[816], [968], [5]], 3
    W = synth.make_weights(cfg, 23, std=0.05 if shape == "small" else 0.02)
    Wf = O.Weights(W)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        for lens in cases:
            B = len(lens)
            kvs = [synth.make_prefix_kv(cfg, 23, p, b) for b, p in enumerate(lens)]
            packed, cu = synth.pack_prefix_kv(kvs)
            states = torch.stack([synth.make_state(cfg, 23, b) for b in range(B)])
            noise = torch.stack([synth.make_noise(cfg, 23, b) for b in range(B)])
            args = (packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), n)
            outs = {}
            for cached in (1, 0):
                ex.set_option("use_state_cache", cached)
                outs[cached] = ex.denoise_batched(*args).double().cpu().numpy()
                torch.cuda.synchronize()
                assert ex.poll_status() == 0
            assert ex.launches_per_call(B, n) > 0
            for b in range(B):
                ref = O.denoise(cfg, Wf, kvs[b], lens[b], states[b], noise[b], n)
                for cached in (1, 0):
                    assert rel_err(outs[cached][b], ref) <= BAR["bf16"], (lens, b, cached, rel_err(outs[cached][b], ref))
            assert rel_err(outs[1], outs[0]) <= BAR["bf16"]
