"""Writes the stored expected values of tests/golden/ from the CPU oracle alone:  python tests/golden/make_golden.py"""
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle.hydra_oracle import HydraOracle  # noqa: E402
from synth import get_config, make_weights, make_prompts, load_tree  # noqa: E402

STEPS = 8


def c1_stream():
    cfg = get_config("c1")
    parent = load_tree(cfg.tree)
    w = make_weights(cfg.model, cfg.head, cfg.seed)
    prompts = make_prompts(cfg.seed, cfg.prompt_lens, cfg.model.vocab)
    o = HydraOracle(cfg.model, cfg.head, parent, w, cfg.max_seq)
    o.prefill(prompts)
    steps = []
    for _ in range(STEPS):
        tok, head_logits = o.draft(return_logits=True)
        amax, logits = o.verify(tok)
        n_acc, path, out_tok = o.accept_compact(tok, amax)
        # smallest gap that decided an integer in this step: between the last kept and the first dropped head logit of
        # any parent, and between the two largest verify logits of any row (a float32 path may differ below ~1e-4)
        gaps = []
        for p, lg in head_logits[0].items():
            srt = lg.sort(descending=True).values
            c = len(o.tree.children[p])
            gaps += [float(srt[i] - srt[i + 1]) for i in range(c)]
        top2 = logits[0].topk(2, dim=-1).values
        gaps += [float(g) for g in (top2[:, 0] - top2[:, 1])]
        steps.append({"tree_tok": [int(t) for t in tok[0]], "amax": [int(a) for a in amax[0]], "n_acc": int(n_acc[0]),
                      "committed": [int(t) for t in out_tok[0][: int(n_acc[0]) + 1]], "min_gap": min(gaps)})
    return {"config": "c1", "steps": steps}


if __name__ == "__main__":
    with open(os.path.join(HERE, "c1_stream.json"), "w") as f:
        json.dump(c1_stream(), f, indent=1)
    print("wrote c1_stream.json")
