"""A device-side wait that gives up: with the iteration bound of the kernels' waits lowered to 1, a pipeline wait
(a weight or activation copy that has not landed at the first poll) expires, the status word reports TIMEOUT, the
kernels still run to their end (nothing hangs, nothing is left in flight), and after the bound is restored the same
handle gives the correct result again.  Nothing here faults or hangs the device: the waited-for data does arrive."""
import pytest
import torch

from oracle import expert_oracle as O
from paper_2608_03682_b200 import binding, synth
from tests.helpers import BAR, rel_err, small_bf16_config

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cluster_gemm", [1, 0])
@pytest.mark.parametrize("batch", [1, 40, 80])   # 80 requests = 1120 tokens: the persistent 256-token-tile kernels
def test_expired_wait_is_reported_and_the_handle_recovers(cluster_gemm, batch):
    cfg = small_bf16_config("pi0", max_batch=batch, max_prefix_len=150)
    W = synth.make_weights(cfg, 31, std=0.05)
    lens = [150 - (7 * b) % 90 for b in range(batch)]
    kvs = [synth.make_prefix_kv(cfg, 31, p, b) for b, p in enumerate(lens)]
    packed, cu = synth.pack_prefix_kv(kvs)
    states = torch.stack([synth.make_state(cfg, 31, b) for b in range(batch)])
    noise = torch.stack([synth.make_noise(cfg, 31, b) for b in range(batch)])
    args = (packed.cuda(), torch.from_numpy(cu).cuda(), states.cuda(), noise.cuda(), 3)
    ref0 = O.denoise(cfg, W, kvs[0], lens[0], states[0], noise[0], 3)
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        ex.set_option("use_cluster_gemm", cluster_gemm)
        good = ex.denoise_batched(*args).clone()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        assert rel_err(good[0].double().cpu().numpy(), ref0) <= BAR["bf16"]

        ex.set_option("wait_limit", 1)
        out = torch.full_like(noise, 7.0).cuda()
        ex.denoise_batched(*args, out=out)
        torch.cuda.synchronize()                      # returns: every wait is bounded
        assert ex.poll_status() == binding.ERR_TIMEOUT
        assert ex.poll_status() == 0                  # reading the status word clears it
        # the result of a timed-out call is invalid by contract (stores after the give-up are suppressed, earlier
        # ones are not undone); it is only required to be there, i.e. the call ran to its end

        ex.set_option("wait_limit", 1 << 22)
        again = ex.denoise_batched(*args).clone()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        # (beyond 64 tokens the split-K residual adds are atomic, so two runs agree to rounding, not to the bit)
        assert rel_err(again[0].double().cpu().numpy(), ref0) <= BAR["bf16"]
        assert rel_err(again.double().cpu().numpy(), good.double().cpu().numpy()) <= BAR["bf16"]


@pytest.mark.parametrize("cond,dtype", [("pi0", "bf16"), ("pi05", "bf16"), ("pi0", "w8e4m3"), ("pi0", "w4a16")])
def test_expired_waits_in_the_full_width_single_tile_kernels(cond, dtype):
    """Width 1024: the step-boundary cluster kernel, the one-head-per-CTA attention kernel with its bulk-copied Q tile
    and the stage-by-stage weight decode all have waits of their own; lowered to one poll they give up (the data
    still arrives), the call returns with TIMEOUT, and the handle is good again afterwards."""
    cfg = synth.ExpertConfig(n_layers=2, width=1024, mlp_dim=4096, n_q_heads=8, n_kv_heads=1, head_dim=256, state_dim=32,
                             action_dim=32, horizon=50, has_state_token=(cond == "pi0"), max_prefix_len=300, max_batch=1,
                             cond=cond, dtype=dtype)
    W = synth.make_weights(cfg, 32)
    kv = synth.make_prefix_kv(cfg, 32, 300)
    state = synth.make_state(cfg, 32) if cfg.has_state_token else None
    noise = synth.make_noise(cfg, 32)
    ref = O.denoise(cfg, W, kv, 300, state, noise, 3)
    dev = lambda t: None if t is None else t.cuda()
    with binding.Expert(cfg, binding.weights_to_device(W)) as ex:
        good = ex.denoise(dev(kv), 300, dev(state), dev(noise), 3).clone()
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        assert rel_err(good.double().cpu().numpy(), ref) <= BAR["bf16"]
        ex.set_option("wait_limit", 1)
        ex.denoise(dev(kv), 300, dev(state), dev(noise), 3)
        torch.cuda.synchronize()
        assert ex.poll_status() == binding.ERR_TIMEOUT
        ex.set_option("wait_limit", 1 << 22)
        again = ex.denoise(dev(kv), 300, dev(state), dev(noise), 3)
        torch.cuda.synchronize()
        assert ex.poll_status() == 0
        assert torch.equal(again, good)              # the single-tile path is bit-reproducible
