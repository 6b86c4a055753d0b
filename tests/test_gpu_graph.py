"""The compute calls of the path recorded once into a CUDA graph and replayed on new data.

After af_reserve the calls other than af_pack_microbatch allocate nothing and never wait on the
host, so a launch-bound step (small batches: a handful of kernels of a few microseconds each) can
be captured and replayed as one graph launch.  The replay must give what the plain calls give, on
the data that is in the buffers at replay time, and what the oracle gives."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O
from paper_2507_01663_b200 import workloads as wl
from gpu_util import ADV_TOL, GRAD_RTOL, LOGP_TOL, LOSS_RTOL, device, np_of, rel

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2507_01663_b200 import binding as B
    c = B.Context(0)
    yield c
    c.close()


class Step:
    """Device buffers of one micro-batch holding every response of the workload in order, and the
    chain advantage -> log-prob -> loss -> backward, then the same update as one fused call."""

    def __init__(self, ctx, w):
        from paper_2507_01663_b200 import binding as B
        dev = device()
        self.ctx, self.w, self.B = ctx, w, B
        T = w.total_tokens
        self.T = T
        self.H = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
        self.W = wl.gen_weight(w).to(dev)
        self.y = wl.gen_target(w).to(dev)
        self.reward = torch.empty(w.N, device=dev)
        self.old, self.ref = torch.empty(T, device=dev), torch.empty(T, device=dev)
        self.cu = torch.as_tensor(w.tok_offset.astype(np.int32), device=dev)
        self.adv = torch.empty(w.N, device=dev)
        self.logp, self.ent, self.lse, self.g = (torch.empty(T, device=dev) for _ in range(4))
        self.out = B.new_loss_out(dev)
        self.dH = torch.empty(T, w.d, dtype=torch.bfloat16, device=dev)
        self.dW = torch.empty(w.V, w.d, device=dev)
        # outputs of the fused call
        self.logp_f, self.ent_f, self.lse_f, self.g_f = (torch.empty(T, device=dev) for _ in range(4))
        self.out_f = B.new_loss_out(dev)
        self.dH_f = torch.empty_like(self.dH)
        self.dW_f = torch.empty_like(self.dW)

    def load(self, H, reward, old, ref):
        self.H.copy_(H)
        self.reward.copy_(reward)
        self.old.copy_(old)
        self.ref.copy_(ref)

    def poison(self):
        for t in (self.adv, self.logp, self.ent, self.lse, self.g, self.logp_f, self.ent_f, self.lse_f, self.g_f,
                  self.dW, self.dW_f):
            t.fill_(123.0)
        self.dH.fill_(5.0)
        self.dH_f.fill_(5.0)
        self.out.zero_()
        self.out_f.zero_()

    def run(self, scoring_only=False):
        c, w = self.ctx, self.w
        c.grpo_advantage(self.reward, None, w.n_prompts, self.adv)
        c.token_logprob(self.H, self.W, self.y, self.logp, self.ent, self.lse)
        c.policy_loss(self.logp, self.old, self.ref, self.adv, self.cu, self.out, self.g, self.ent,
                      w.clip_eps, w.clip_eps, w.kl_coef)
        if scoring_only:
            return
        c.policy_loss_backward(self.H, self.W, self.y, self.lse, self.g, self.dH, self.dW)
        c.policy_update(self.H, self.W, self.y, self.old, self.ref, self.adv, self.cu, self.out_f, self.logp_f,
                        self.lse_f, self.dH_f, self.dW_f, entropy=self.ent_f, dlogp=self.g_f,
                        clip_lo=w.clip_eps, clip_hi=w.clip_eps, kl_coef=w.kl_coef)

    def results(self):
        torch.cuda.synchronize()
        B = self.B
        return {"adv": self.adv.clone(), "logp": self.logp.clone(), "ent": self.ent.clone(), "lse": self.lse.clone(),
                "g": self.g.clone(), "dH": self.dH.clone(), "dW": self.dW.clone(), "loss": B.read_loss_out(self.out),
                "logp_f": self.logp_f.clone(), "g_f": self.g_f.clone(), "dH_f": self.dH_f.clone(),
                "dW_f": self.dW_f.clone(), "loss_f": B.read_loss_out(self.out_f)}


def same(a, b):
    for k in a:
        if isinstance(a[k], dict):
            assert a[k] == b[k], k
        else:
            assert torch.equal(a[k], b[k]), k


def data_sets(w):
    """Two sets of (hidden, reward, old, ref) for the same sequence table."""
    H = wl.gen_hidden(w)
    lp, _, _ = O.token_logprob_ref(wl.bf16_bits(H), wl.bf16_bits(wl.gen_weight(w)), wl.gen_target(w).numpy())
    T = w.total_tokens
    first = (H, wl.gen_reward(w), torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_OLD, T),
             torch.tensor(lp, dtype=torch.float32) + wl.gen_noise(w, wl.S_REF, T))
    H2 = torch.flip(H, dims=[0]).contiguous()
    lp2, _, _ = O.token_logprob_ref(wl.bf16_bits(H2), wl.bf16_bits(wl.gen_weight(w)), wl.gen_target(w).numpy())
    second = (H2, 1.0 - wl.gen_reward(w), torch.tensor(lp2, dtype=torch.float32) + wl.gen_noise(w, wl.S_REF, T),
              torch.tensor(lp2, dtype=torch.float32) + wl.gen_noise(w, wl.S_OLD, T))
    return first, second


@pytest.mark.parametrize("name,variant", [("cfg1", 2), ("cfg4_mini", 2), ("cfg4_mini", 1)])
def test_captured_step_replays_on_new_data(ctx, name, variant):
    w = wl.make_workload(name)
    first, second = data_sets(w)
    ctx.set_tuning(0, 256, variant)
    ctx.reserve(w.total_tokens, w.N, w.d, w.V, with_backward=2)
    st = Step(ctx, w)
    st.load(*first)
    st.run()                                    # plain calls
    plain_first = st.results()
    reserved = ctx.workspace_bytes()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        st.run()
    assert ctx.workspace_bytes() == reserved    # nothing was grown while recording

    st.poison()
    graph.replay()
    same(plain_first, st.results())

    st.load(*second)                            # new contents, same buffers
    st.poison()
    graph.replay()
    replay_second = st.results()
    st.poison()
    st.run()
    same(st.results(), replay_second)
    ctx.set_tuning(0, 0)
    assert ctx.check_device_errors() == 0
    assert not torch.equal(plain_first["logp"], replay_second["logp"])

    # and against the oracle, on the second data set
    H2, reward2, old2, ref2 = second
    Wb, yb = wl.bf16_bits(wl.gen_weight(w)), wl.gen_target(w).numpy()
    adv_ref = O.grpo_advantage_ref(np_of(reward2), w.group_id, w.n_prompts)
    assert np.abs(np_of(replay_second["adv"]) - adv_ref).max() <= ADV_TOL
    lp, ent, lse = O.token_logprob_ref(wl.bf16_bits(H2), Wb, yb)
    for key, r in (("logp", lp), ("ent", ent), ("lse", lse), ("logp_f", lp)):
        assert np.abs(np_of(replay_second[key]) - r).max() <= LOGP_TOL, key
    oref = O.policy_loss_ref(np_of(replay_second["logp"]), old2.numpy(), ref2.numpy(), np_of(replay_second["adv"]),
                             w.tok_offset, w.clip_eps, w.clip_eps, w.kl_coef, 0, 1.0, entropy=np_of(replay_second["ent"]))
    for key in ("loss", "pg_loss", "kl_mean"):
        assert rel(replay_second["loss"][key], oref[key]) <= LOSS_RTOL, key
        assert rel(replay_second["loss_f"][key], oref[key]) <= LOSS_RTOL, key
    dH_ref, dW_ref = O.policy_loss_backward_ref(wl.bf16_bits(H2), Wb, yb, np_of(replay_second["lse"]),
                                                np_of(replay_second["g"]))
    nH, nW = np.linalg.norm(dH_ref), np.linalg.norm(dW_ref)
    for kH, kW in (("dH", "dW"), ("dH_f", "dW_f")):
        assert np.linalg.norm(np_of(replay_second[kH].float()) - dH_ref) <= GRAD_RTOL * nH, kH
        assert np.linalg.norm(np_of(replay_second[kW]) - dW_ref) <= GRAD_RTOL * nW, kW


def test_replay_of_a_launch_bound_scoring_step(ctx):
    """At the smallest workload the scoring step (advantage, log-prob, loss) runs for a few tens of
    microseconds on the device and the host's launches take longer than that.  The replay must give
    the plain calls' results bit for bit; the two timings are printed, not asserted (a shared machine can
    disturb either loop; timing belongs to the benchmark)."""
    w = wl.make_workload("cfg1")
    first, _ = data_sets(w)
    ctx.reserve(w.total_tokens, w.N, w.d, w.V, with_backward=2)
    st = Step(ctx, w)
    st.load(*first)
    for _ in range(3):
        st.run(scoring_only=True)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        st.run(scoring_only=True)

    def avg_us(fn, n=50):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / n

    # best of three: a timing comparison should not depend on one disturbed loop
    plain = min(avg_us(lambda: st.run(scoring_only=True)) for _ in range(3))
    replay = min(avg_us(graph.replay) for _ in range(3))
    print(f"cfg1 scoring step: plain calls {plain:.1f} us, graph replay {replay:.1f} us")
    st.run(scoring_only=True)
    torch.cuda.synchronize()
    want = {k: getattr(st, k).clone() for k in ("logp", "ent", "lse", "g", "adv")}
    for k in want:
        getattr(st, k).fill_(3.0)
    graph.replay()
    torch.cuda.synchronize()
    for k, v in want.items():
        assert torch.equal(getattr(st, k), v), k
    assert ctx.check_device_errors() == 0


def test_advantage_by_group_id_is_recordable_right_after_reserve(ctx):
    """The per-group accumulators of the id path belong to what af_reserve sizes: a context that has
    never taken advantages by id records the call without growing its workspace, and the replay on
    new rewards agrees with the oracle and, bit for bit, with the plain call."""
    w = wl.make_workload("cfg5_mini")
    dev = device()
    ctx.reserve(w.total_tokens, w.N, w.d, w.V, with_backward=0)
    reserved = ctx.workspace_bytes()
    order = np.random.default_rng(5).permutation(w.N)
    gid_host = np.asarray(w.group_id, dtype=np.int32)[order]
    gid = torch.as_tensor(gid_host, device=dev)
    reward = torch.empty(w.N, device=dev)
    adv = torch.empty(w.N, device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.grpo_advantage(reward, gid, w.n_prompts, adv)
    assert ctx.workspace_bytes() == reserved
    for flip in (False, True):
        r = wl.gen_reward(w).numpy()[order]
        r = (1.0 - r) if flip else r
        reward.copy_(torch.as_tensor(r))
        adv.fill_(9.0)
        graph.replay()
        torch.cuda.synchronize()
        replayed = adv.clone()
        assert np.abs(np_of(replayed) - O.grpo_advantage_ref(r, gid_host, w.n_prompts)).max() <= ADV_TOL
        adv.fill_(9.0)
        ctx.grpo_advantage(reward, gid, w.n_prompts, adv)
        torch.cuda.synchronize()
        assert torch.equal(adv, replayed)
    assert ctx.check_device_errors() == 0
