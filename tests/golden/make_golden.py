"""Writes the stored expected values under tests/golden/ by calling only the CPU oracle.

The paper prints no worked numeric example of the verification step (its numbers are
end-to-end accuracy and tokens/s on datasets that are not available here), so the stored
values are the oracle's own results on seeded synthetic inputs.  They guard against an
unintended change of the oracle and give the GPU tests a fixed target for the tiny
workload.  Run:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import aj_inputs as gen  # noqa: E402
from oracle import aj_oracle as orc  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))

CASES = {
    # the tiny fp32 workload, as specified
    "c1_tiny_f32": gen.C1,
    # the same shape in bf16 with a ragged vocabulary tail and three sequences
    "tiny_bf16_b3": gen.scaled(gen.C1, name="tiny_bf16_b3", B=3, K=6, dtype=gen.BF16, V=1000, seed=1),
}


# the variants of the step: (config, how the target's tokens are taken, tree or window)
VARIANTS = {
    "tiny_bf16_sampled": dict(cfg=gen.scaled(gen.C1, name="tiny_bf16_sampled", B=2, K=5, dtype=gen.BF16, V=1000, seed=2),
                              temperature=0.8, seed=11, step=3),
    "tiny_f32_tree": dict(cfg=gen.scaled(gen.C1, name="tiny_f32_tree", B=2, K=7, seed=3), parent=[-1, -1, 0, 0, 1, 2, 2]),
}


def compute_variant(cfg, temperature=0.0, seed=0, step=0, parent=None):
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    zeros = np.zeros((cfg.B, cfg.K), np.int32)
    out = {"generator": gen.GENERATOR_VERSION,
           "config": {k: getattr(cfg, k) for k in ("B", "K", "d", "d_draft", "V", "dtype", "seed", "tau")}}
    if parent is None:
        y = orc.verify(ht, hd, W, zeros, w, cfg.judge_b, cfg.tau, cfg.dtype, temperature=temperature, seed=seed, step=step).target_tok
        tok = gen.plant_draft_tokens(cfg, y)
        r = orc.verify(ht, hd, W, tok, w, cfg.judge_b, cfg.tau, cfg.dtype, temperature=temperature, seed=seed, step=step)
        out["noise"] = [round(orc.gumbel(seed, step, j, v), 12) for j, v in ((0, 0), (1, 7), (5, 999))]
    else:
        par = np.tile(np.array(parent, np.int32), (cfg.B, 1))
        y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
        tok = gen.plant_draft_tokens(cfg, np.stack([np.append(y[b][par[b] + 1], 0) for b in range(cfg.B)]))
        r = orc.verify_tree(ht, hd, W, tok, par, w, cfg.judge_b, cfg.tau, cfg.dtype)
        out["parent"] = parent
        out["best_node"] = r.best_node.tolist()
    out.update({
        "draft_tok": tok.tolist(), "target_tok": r.target_tok.tolist(), "accept_len": r.accept_len.tolist(), "next_tok": r.next_tok.tolist(),
        "top1": [[round(float(x), 12) for x in row] for row in r.top1],
        "judge_p": [[None if np.isnan(x) else round(float(x), 12) for x in row] for row in r.judge_p],
    })
    return out


def compute(cfg):
    W = gen.make_W(cfg)
    ht, hd = gen.make_hidden(cfg)
    w = gen.make_judge(cfg)
    y = np.stack([[orc.argmax(r)[0] for r in orc.logits(ht[b], W, cfg.dtype)] for b in range(cfg.B)])
    tok = gen.plant_draft_tokens(cfg, y)
    r = orc.verify(ht, hd, W, tok, w, cfg.judge_b, cfg.tau, cfg.dtype)
    return {
        "generator": gen.GENERATOR_VERSION,
        "config": {k: getattr(cfg, k) for k in ("B", "K", "d", "d_draft", "V", "dtype", "seed", "tau")},
        "draft_tok": tok.tolist(),
        "target_tok": r.target_tok.tolist(),
        "accept_len": r.accept_len.tolist(),
        "next_tok": r.next_tok.tolist(),
        "top1": [[round(float(x), 12) for x in row] for row in r.top1],
        "gap": [[round(float(x), 12) for x in row] for row in r.gap],
        "judge_p": [[None if np.isnan(x) else round(float(x), 12) for x in row] for row in r.judge_p],
    }


if __name__ == "__main__":
    for name, cfg in CASES.items():
        with open(os.path.join(HERE, f"{name}.json"), "w") as f:
            json.dump(compute(cfg), f, indent=1)
            f.write("\n")
        print("wrote", name)
    for name, v in VARIANTS.items():
        with open(os.path.join(HERE, f"{name}.json"), "w") as f:
            json.dump(compute_variant(**v), f, indent=1)
            f.write("\n")
        print("wrote", name)
