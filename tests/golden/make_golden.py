"""Writes tests/golden/oracle_tiny.json: a digest of what the CPU oracle computes on the seeded tiny workload
(attention-only stream, full decoder block, language-model head).  The paper (arXiv 2503.09387) prints no worked
numerical example, so these are not the paper's numbers: they are the oracle's own, stored so that a later change
to its arithmetic cannot pass unnoticed (tests/test_oracle_golden.py recomputes and compares them).  Calls the
oracle and the seeded input generator only.  Run from the repository root:  python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import videoscan_oracle as vo              # noqa: E402
from paper_2503_09387_b200 import synth                # noqa: E402


def digest(x):
    """A few exact statistics and samples of a tensor (fp64, printed with 17 significant digits)."""
    x = np.asarray(x, dtype=np.float64)
    flat = x.reshape(-1)
    idx = [(i * 7919) % flat.size for i in range(8)]
    return {"shape": list(x.shape), "sum": float(flat.sum()), "sum_abs": float(np.abs(flat).sum()),
            "sum_sq": float((flat * flat).sum()), "samples": [float(flat[i]) for i in idx]}


def compute():
    f64 = synth.bf16_bits_to_f64
    out = {}
    # Sections 3.2 / 3.3: attention-only stream on the tiny workload (evictions at frames 4..7)
    w = synth.workload("tiny")
    cfg = vo.OracleConfig(w.n_layers, w.d_model, w.n_q_heads, w.n_kv_heads, w.head_dim, w.bank_capacity,
                          use_rmsnorm=w.use_rmsnorm, residual=w.residual, rope_theta=w.rope_theta, rms_eps=w.rms_eps)
    st = vo.OracleStream(cfg, [f64(w.weight(l)) for l in range(w.n_layers)])
    out["prefix"] = digest(st.text_step(f64(w.prefix_hidden())))
    for t in range(w.n_frames):
        out[f"frame_{t}"] = digest(st.frame_step(f64(w.frame_hidden(t))))
    out["question"] = digest(st.text_step(f64(w.question_hidden()))) if w.question_len else None
    for i in range(w.decode_tokens):
        out[f"decode_{i}"] = digest(st.text_step(f64(w.decode_hidden(i))))
    out["bank_frame_ids"] = st.bank_frame_ids()
    out["bank_positions"] = st.bank_positions()
    out["evict_log"] = [list(map(int, e)) for e in st.evict_log]
    out["carriers_only_forward"] = digest(st.carriers_only_forward())
    # Section 4.1 backbone: two full decoder layers and the language-model head
    w2 = synth.workload("tiny", n_layers=2, use_rmsnorm=1, residual=1, n_q_heads=4, n_kv_heads=2, head_dim=64)
    cfg2 = vo.OracleConfig(2, w2.d_model, 4, 2, 64, w2.bank_capacity, use_rmsnorm=1, residual=1,
                           rope_theta=w2.rope_theta, rms_eps=w2.rms_eps)
    blocks = []
    for l in range(2):
        b = w2.block_weights(l, 192)
        blocks.append(vo.BlockWeights(f64(b["w_o"]), f64(b["w_gate"]), f64(b["w_up"]), f64(b["w_down"])))
    s2 = vo.OracleStream(cfg2, [f64(w2.weight(l)) for l in range(2)], None, None, blocks)
    s2.text_step(f64(w2.prefix_hidden()))
    for t in range(3):
        h = s2.frame_step(f64(w2.frame_hidden(t)))
    out["block_frame_2"] = digest(h)
    h = s2.text_step(f64(w2.decode_hidden(0)))
    out["block_decode_0"] = digest(h)
    logits, tok = vo.lm_head(h, f64(w2.lm_weights(256)), None, True, w2.rms_eps)
    out["lm_logits"] = digest(logits)
    out["lm_token"] = [int(t) for t in tok]
    return out


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_tiny.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
