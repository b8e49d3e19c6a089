"""Whole-step parity of the CUDA library against the CPU oracle (lock-step, through the C ABI)."""
import pytest
import torch

from oracle.hydra_oracle import HydraOracle
from synth import get_config, make_weights, make_prompts, load_tree, chain_tree
from synth.configs import ModelCfg, HeadCfg
from tests.parity import lockstep

pytestmark = pytest.mark.gpu


def run(model, head, parent, prompts_lens, steps, seed, max_seq, oracle_dtype=torch.float64, weights_device="cpu",
        norm_gain_std=0.0, gemm_mode=0, **kw):
    from paper_2402_05109_b200 import Hydra
    w = make_weights(model, head, seed, device=weights_device, norm_gain_std=norm_gain_std)
    wg = {k: v.cuda() for k, v in w.items()}
    wc = {k: v.cpu() for k, v in w.items()}
    prompts = make_prompts(seed, prompts_lens, model.vocab)
    o = HydraOracle(model, head, parent, wc, max_seq, dtype=oracle_dtype, cache_weights=True)
    g = Hydra(model, head, parent, wg, max_batch=len(prompts), max_seq=max_seq)
    g.set_gemm_mode(gemm_mode)
    try:
        return lockstep(o, g, prompts, steps, seed, **kw), g
    finally:
        g.close()


def test_c1_tiny_fp32_all_steps_accept_exercise():
    cfg = get_config("c1")
    st, _ = run(cfg.model, cfg.head, load_tree(cfg.tree), cfg.prompt_lens, cfg.steps, cfg.seed, cfg.max_seq, kv_layers=(0, 1))
    assert st.steps == 8
    seen = {n for step in st.n_acc for n in step}
    assert seen >= {0, 1, 2, 3}, seen
    assert st.max_logit_err < 1e-3 and st.max_hidden_err < 1e-4      # float path: far inside the tolerances


def test_small_bf16_hydrapp_ragged_batch():
    """bfloat16 / tensor-core path with the prefix layer, 4-layer heads, the 63-node tree and a ragged batch
    whose prompts span several prefill chunks with ragged tails."""
    m = ModelCfg(3, 256, 2, 128, 512, 1024, dtype="bf16")
    h = HeadCfg(4, 4, True)
    st, _ = run(m, h, load_tree("tree63_d4"), [37, 130, 64], 6, 5, 256)
    seen = {n for step in st.n_acc for n in step}
    assert seen >= {0, 1, 2, 3, 4}, seen


@pytest.mark.parametrize("head_dim,kv_planes", [(128, 2), (128, 1), (64, 2)])
def test_prompt_lengths_around_the_prefill_chunk(head_dim, kv_planes):
    """Prompts that end just before, on and just after the 64- and 128-row boundaries of the prompt pass (the bfloat16 path
    walks 128-row causal chunks: two 64-row attention launches at head_dim 128 with two planes, one 128-row launch otherwise):
    the lock-step protocol compares the caches of both layers, the last hidden state and the first steps with the oracle."""
    m = ModelCfg(2, 256, 256 // head_dim, head_dim, 512, 1024, dtype="bf16", kv_planes=kv_planes)
    h = HeadCfg(3, 2, True)
    st, _ = run(m, h, load_tree("tree15_d3"), [127, 128, 129, 64, 65, 191, 256, 1], 2, 31, 320, kv_layers=(0, 1))
    assert st.steps == 2


@pytest.mark.parametrize("dtype,mlp,prefix", [("bf16", 1, False), ("bf16", 3, True), ("fp32", 2, False)])
def test_medusa_mode_heads(dtype, mlp, prefix):
    """Sequentially independent heads (the Medusa baseline): head i sees the hidden state alone, one logits row per
    sequence and level, every parent of a level gets the same children (the oracle's head with head.medusa)."""
    m = ModelCfg(2, 256, 2, 128, 512, 1024, dtype=dtype)
    h = HeadCfg(4, mlp, prefix, medusa=True)
    st, _ = run(m, h, load_tree("tree63_d4"), [37, 70, 9], 4, 13, 192)
    seen = {n for step in st.n_acc for n in step}
    assert st.steps == 4 and seen >= {0, 1, 2, 3}, seen


@pytest.mark.parametrize("kv_planes", [1])
def test_single_plane_cache_option(kv_planes):
    """kv_planes = 1: q and the caches hold one float16 plane (half the cache bytes); small models stay far inside the
    tolerances (the deepest shapes do not: two planes are the default)."""
    m = ModelCfg(3, 256, 2, 128, 512, 1024, dtype="bf16", kv_planes=kv_planes)
    h = HeadCfg(4, 2, True)
    st, _ = run(m, h, load_tree("tree63_d4"), [37, 130], 3, 5, 256)
    assert st.steps == 3 and st.max_hidden_err < 5e-3


@pytest.mark.parametrize("dtype,gemm_mode", [("bf16", 0), ("bf16", 1), ("fp32", 0)])
def test_random_norm_gains_reach_the_right_norms(dtype, gemm_mode):
    """Every RMSNorm gain vector (2 per layer, the final norm, the prefix layer's 2) drawn as 1 + 0.1 N(0,1) from its
    own stream: a kernel that ignored a gain, or read another norm's, would leave the tolerances at once (a 10 %
    per-channel error).  The benchmark shapes use gains of 1, which cannot show this."""
    m = ModelCfg(3, 256, 2, 128, 512, 1024, dtype=dtype)
    h = HeadCfg(4, 2, True)
    st, _ = run(m, h, load_tree("tree63_d4"), [37, 70], 3, 21, 192, norm_gain_std=0.1, gemm_mode=gemm_mode,
                kv_layers=(0, 1, 2))
    assert st.steps == 3


@pytest.mark.parametrize("mode", [1])
def test_small_bf16_other_gemm_modes_and_root_only_tree(mode):
    """mode 1: the SIMT GEMM (reads only the hi plane of the activations)."""
    from paper_2402_05109_b200 import Hydra
    m = ModelCfg(2, 256, 4, 64, 512, 1024, dtype="bf16")
    h = HeadCfg(2, 1, False)
    w = make_weights(m, h, 6)
    prompts = make_prompts(6, [20], m.vocab)
    o = HydraOracle(m, h, [-1], w, 64)
    g = Hydra(m, h, [-1], {k: v.cuda() for k, v in w.items()}, 1, 64)
    g.set_gemm_mode(mode)
    st = lockstep(o, g, prompts, 3, 6, plant=False)
    assert all(n == [0] for n in st.n_acc)
    g.close()


def test_chain_tree_and_capacity_and_state_errors():
    from paper_2402_05109_b200 import Hydra, HydraError
    m = ModelCfg(2, 256, 4, 64, 512, 1024, dtype="fp32")
    h = HeadCfg(3, 1, False)
    w = make_weights(m, h, 7)
    parent = chain_tree(3)
    o = HydraOracle(m, h, parent, w, 48)
    g = Hydra(m, h, parent, {k: v.cuda() for k, v in w.items()}, 1, 48)
    with pytest.raises(HydraError, match="order"):
        g.batch = 1
        g.draft()
    st = lockstep(o, g, make_prompts(7, [30], m.vocab), 3, 7)
    # capacity: the lock-step protocol polled after every phase, so the host's bound equals the real length L0 now;
    # without further polls it grows by K+1 = 4 per step, and a step whose bound + T exceeds max_seq = 48 must be
    # refused before any launch
    L0 = int(g.get_buffer("LEN")[0])
    allowed = 0
    while L0 + allowed * 4 + 4 <= 48:
        allowed += 1
    for _ in range(allowed):
        g.step()
    before = g.launch_count()
    with pytest.raises(HydraError, match="capacity"):
        g.step()
    assert g.launch_count() == before and allowed >= 1
    g.close()


def test_polling_lets_decoding_use_the_whole_cache():
    """The host's length bounds grow by K+1 per step; hydra_poll_status replaces them by the real lengths.  With
    root-only acceptance (random candidates are rejected) a sequence grows by one token per step, so a caller
    that polls must be able to decode until len + T == max_seq, far beyond what the bounds alone allow."""
    from paper_2402_05109_b200 import Hydra, HydraError
    m = ModelCfg(1, 256, 4, 64, 512, 1024, dtype="fp32")
    h = HeadCfg(3, 1, False)
    parent = chain_tree(3)
    T, max_seq, plen = len(parent), 64, 20
    w = make_weights(m, h, 12)
    g = Hydra(m, h, parent, {k: v.cuda() for k, v in w.items()}, 1, max_seq)
    g.prefill(make_prompts(12, [plen], m.vocab))
    never = torch.full((1, T), -1, dtype=torch.int32)
    never[0, 1] = m.vocab - 1                       # planted first candidate: (almost surely) not the base argmax
    g.set_plant(never.cuda())
    n_acc = torch.empty(1, dtype=torch.int32, device="cuda")
    steps, lens = 0, []
    while True:
        try:
            g.step(n_acc)
        except HydraError as e:
            assert "capacity" in str(e)
            break
        g.poll_status()
        steps += 1
        lens.append(int(g.get_buffer("LEN")[0]))
        assert steps < 200
    assert lens[-1] + T > max_seq and lens[-1] <= max_seq          # stopped only when the cache was really full
    assert steps > (max_seq - T - plen) // (h.n_heads + 1) + 2     # more steps than the un-refreshed bounds allow
    g.close()


def test_out_of_range_token_sets_status_word():
    from paper_2402_05109_b200 import Hydra, HydraError
    m = ModelCfg(1, 256, 4, 64, 512, 1024, dtype="fp32")
    h = HeadCfg(1, 1, False)
    w = make_weights(m, h, 8)
    g = Hydra(m, h, [-1, 0], {k: v.cuda() for k, v in w.items()}, 1, 32)
    g.prefill(make_prompts(8, [5], m.vocab))
    g.draft()
    bad = torch.tensor([[3, 5000]], dtype=torch.int32).cuda()
    g.verify(bad)
    with pytest.raises(HydraError, match="index"):
        g.poll_status()
    g.poll_status()                     # cleared by the poll
    g.close()


def test_step_graph_replay_matches_kernel_by_kernel_launches():
    """hydra_step on a non-default stream replays a captured CUDA graph from the second step on; the emitted
    tokens must equal those of a context that launches kernel by kernel (default stream)."""
    from paper_2402_05109_b200 import Hydra
    m = ModelCfg(2, 256, 2, 128, 512, 1024, dtype="bf16")
    h = HeadCfg(4, 2, True)
    parent = load_tree("tree63_d4")
    w = {k: v.cuda() for k, v in make_weights(m, h, 9).items()}
    prompts = make_prompts(9, [40, 75], m.vocab)
    outs = []
    for use_stream in (False, True):
        g = Hydra(m, h, parent, w, 2, 704)
        stream = torch.cuda.Stream() if use_stream else torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            g.prefill(prompts)
            n_acc = torch.empty(2, dtype=torch.int32, device="cuda")
            out = torch.empty(2, 5, dtype=torch.int32, device="cuda")
            seq = []
            for s in range(100):                      # long enough for the attention grid to grow (re-capture)
                g.step(n_acc, out)
                seq.append(out.clone())
            g.poll_status()
            stream.synchronize()
        outs.append(torch.stack(seq).cpu())
        assert g.launch_count() > 100 * 50
        g.close()
    assert torch.equal(outs[0], outs[1])
