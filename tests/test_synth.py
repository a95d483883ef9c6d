"""The synthetic checkpoint generator: shapes, counts, determinism, distributions."""
import numpy as np
import torch

from paper_2406_11257_b200 import synth


def test_tensor_lists_have_the_stated_sizes():
    want = {"tiny": (28, 3_677_184), "pythia-410m": (292, 405_334_016),
            "pythia-1.4b": (292, 1_414_647_808), "llama-7b": (291, 6_738_415_616)}
    for name, (count, params) in want.items():
        lst = synth.tensor_list(synth.CONFIG_SHAPES[name])
        assert len(lst) == count
        assert sum(n for _, n in lst) == params
    assert max(n for _, n in synth.tensor_list(synth.CONFIG_SHAPES["llama-7b"])) == 32000 * 4096


def test_quads_are_seeded_and_follow_the_distributions():
    a = synth.make_quad(200_000, 5, 3)
    b = synth.make_quad(200_000, 5, 3)
    c = synth.make_quad(200_000, 5, 4)
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert not torch.equal(a[0], c[0])
    w_t, w_prev, ea, eas = (t.numpy() for t in a)
    assert all(t.dtype == np.float32 for t in (w_t, w_prev, ea, eas))
    assert abs(w_prev.std() - 0.02) < 5e-4
    d = (w_t.astype(np.float64) - w_prev)
    assert abs(np.median(np.abs(d)) / (1e-4 / np.sqrt(3)) - 0.7649) < 0.02   # median |t_3|
    assert abs(ea.std() - 1e-4) < 3e-6
    assert eas.min() >= 1e-12 and abs(np.sqrt(eas).mean() / 1e-4 - np.sqrt(2 / np.pi)) < 0.02
    out = synth.make_quad(200_000, 5, 3, outlier_frac=0.01)
    d2 = np.abs(out[0].numpy().astype(np.float64) - out[1].numpy())
    assert (d2 > 30e-4).mean() > 5 * (np.abs(d) > 30e-4).mean()


def test_chain_step_reuses_the_given_previous_weights():
    w_t, w_prev, _, _ = synth.make_quad(1000, 1, 0)
    w2, w1, _, _ = synth.make_quad(1000, 1, 0, step=1, w_prev=w_t)
    assert w1 is w_t and not torch.equal(w2, w_t)
