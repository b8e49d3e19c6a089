"""Lock-step parity of the CUDA library against the CPU oracle at the five benchmark shapes, full model sizes.

The oracle computes in float32 on the bfloat16-rounded weights (widened once, on the GPU, so that the CPU side
does no conversions).  It is slow by design, so every shape runs prefill plus a few decode steps; the planted
lengths cycle so that different accepted lengths occur.  c5's prompts are shortened to 128 tokens per sequence
for the compared run (the weights and the batch are at full shape); the timing runs use the full prompts.
"""
import gc
import time

import pytest
import torch

from oracle.hydra_oracle import HydraOracle
from synth import get_config, make_tensor, weight_names, make_prompts, load_tree
from tests.parity import lockstep

pytestmark = pytest.mark.gpu


def weights_both(cfg):
    """Weights on the GPU (storage dtype) and the same values as float32 CPU tensors for the oracle."""
    wg, wc = {}, {}
    for name in weight_names(cfg.model, cfg.head):
        t = make_tensor(cfg.model, cfg.head, cfg.seed, name, device="cuda")
        wg[name] = t
        wc[name] = t.float().cpu()
    return wg, wc


def run_cfg(cfg, wg, wc, prompt_lens, steps, max_seq, **kw):
    from paper_2402_05109_b200 import Hydra
    parent = load_tree(cfg.tree)
    prompts = make_prompts(cfg.seed, prompt_lens, cfg.model.vocab)
    o = HydraOracle(cfg.model, cfg.head, parent, wc, max_seq, dtype=torch.float32)
    g = Hydra(cfg.model, cfg.head, parent, wg, max_batch=len(prompts), max_seq=max_seq)
    t0 = time.time()
    try:
        st = lockstep(o, g, prompts, steps, cfg.seed, **kw)
    finally:
        g.close()
    print("%s B=%d: %d steps in %.0f s; logits max-abs %.4f, hidden rel-L2 %.4f, head logits %.4f, kv %.4f, forced argmax %d, "
          "under-gap children %d, accepted %s" % (cfg.name, len(prompts), st.steps, time.time() - t0, st.max_logit_err,
                                                  st.max_hidden_err, st.max_head_logit_err, st.max_kv_err, st.forced_amax,
                                                  st.undergap_children, st.n_acc))
    return st


def cleanup():
    gc.collect()
    torch.cuda.empty_cache()


def test_c2_7b_batch1_prompt512():
    cfg = get_config("c2")
    wg, wc = weights_both(cfg)
    st = run_cfg(cfg, wg, wc, cfg.prompt_lens, 5, 512 + 5 * 5 + 64 + 8, kv_layers=(0, 31))
    assert {n for s in st.n_acc for n in s} >= {0, 1, 2, 3, 4}
    del wg, wc
    cleanup()


def test_c3_7b_ragged_batches():
    cfg8 = get_config("c3b8")
    wg, wc = weights_both(cfg8)
    for b in (2, 4, 8):
        lens = cfg8.prompt_lens[:b]
        st = run_cfg(cfg8, wg, wc, lens, 2, max(lens) + 2 * 5 + 64 + 8, kv_layers=(0,))
        assert len({n for s in st.n_acc for n in s}) >= 2          # accepted lengths differ across the batch
    del wg, wc
    cleanup()


def test_c4_13b_long_prompt():
    cfg = get_config("c4")
    wg, wc = weights_both(cfg)
    run_cfg(cfg, wg, wc, cfg.prompt_lens, 2, 2048 + 2 * 5 + 64 + 8, kv_layers=(0, 39))
    del wg, wc
    cleanup()


def test_c5_33b_batch4():
    cfg = get_config("c5")
    wg, wc = weights_both(cfg)
    run_cfg(cfg, wg, wc, [128] * 4, 2, 128 + 2 * 5 + 64 + 8, kv_layers=(0,))
    del wg, wc
    cleanup()
