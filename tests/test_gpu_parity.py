"""Parity of the CUDA path against the CPU oracle on the five workloads, called through the
C-ABI: tree indices, masks, retrieve rows, argmax, accepted path/tokens and the compacted
cache must be bit-exact; attention within max-abs 2e-2 / max-rel 1e-2."""
import os

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

SCALE = float(os.environ.get("RESPS_TEST_STEPS_SCALE", "1"))


def _run(index, n_steps, n_layers, attn_every, attn_seqs=None, cap=None):
    from harness import Runner
    from paper_2601_12212_b200 import synth
    w = synth.WORKLOADS[index]
    r = Runner(w, n_layers=n_layers, kv_capacity=cap)
    n_steps = max(1, int(n_steps * SCALE))
    for step in range(n_steps):
        layers = range(n_layers) if step % attn_every == 0 else ()
        r.step(step, attn_layers=layers, attn_seqs=attn_seqs)
    st = r.stats
    r.close()
    print(f"\n[cfg{index}] steps={st.steps} near_tie={st.near_tie_steps} (mismatch {st.near_tie_mismatch}) "
          f"attn_checks={st.attn_checks} max_abs={st.attn_max_abs:.2e} max_rel={st.attn_max_rel:.2e} "
          f"mean_accept={np.mean(st.accept_lens):.2f} mean_n={np.mean(st.n_nodes):.1f}")
    assert st.near_tie_mismatch <= max(1, st.steps // 50)
    return st


def test_config1_tiny():
    st = _run(1, 32, 1, 1)
    assert max(st.accept_lens) >= 1


def test_config2_llama8b_shape():
    st = _run(2, 6, 2, 2)
    assert st.n_nodes[0] == 60


def test_config3_vicuna13b_shape_varying_actions():
    st = _run(3, 16, 1, 4)
    assert len(set(st.n_nodes)) > 1          # (TT, d, k) really changes between steps


def test_config4_llama70b_shape():
    st = _run(4, 2, 1, 2)
    assert st.n_nodes[0] == 96


def test_config5_ragged_batch():
    st = _run(5, 5, 1, 4, attn_seqs=(0, 5))
    assert len(set(st.n_nodes)) > 2
