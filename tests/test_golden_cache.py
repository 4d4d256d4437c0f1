"""The stored full-size oracle outputs (tests/golden/full_size_confidence_*.npz) belong to the inputs the
generator makes today and to the oracle as it stands: the digests of the input bytes match, and rows
picked at random are recomputed by the oracle here and must reproduce the stored values."""
import numpy as np
import pytest

import oracle
import psd_inputs as gen
from psd_testlib import golden_confidence


@pytest.mark.parametrize("name", ["class_7b", "batched_serving", "deep_sweep"])
def test_stored_values_are_the_oracles(name):
    cfg = gen.CONFIGS[name]
    wl = gen.make(cfg)
    g = golden_confidence(name, wl)                       # fails if a digest differs
    assert g["token"].shape == (cfg.rows,) and g["token1"].shape == (cfg.B * cfg.M,)
    rng = np.random.default_rng(17)
    for hidden, sfx in ((wl.hidden_verify, ""), (wl.hidden_stage1, "1")):
        rows = np.sort(rng.choice(hidden.shape[0], size=3, replace=False))
        tok, conf, lse, gap = oracle.confidence(hidden[rows], wl.W)
        assert np.array_equal(tok, g["token" + sfx][rows])
        assert np.array_equal(conf, g["conf" + sfx][rows]) and np.array_equal(lse, g["lse" + sfx][rows])
        assert np.allclose(gap, g["gap" + sfx][rows], rtol=1e-6, atol=1e-7)       # stored as fp32
    # the stored values are confidences: in (0, 1], tokens inside the vocabulary, gaps non-negative
    assert (g["conf"] > 0).all() and (g["conf"] <= 1).all() and (g["gap"] >= 0).all()
    assert (g["token"] >= 0).all() and (g["token"] < cfg.V).all()
