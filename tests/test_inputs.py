"""The seeded workload generator: determinism, distributions, and that planted peaks do what the
workload descriptions need (confidences on both sides of the policy threshold)."""
import numpy as np

import oracle
import psd_inputs as gen


def test_counter_rng_is_a_pure_function():
    a = [gen.uniform(3, 1, i) for i in range(5)]
    b = [gen.uniform(3, 1, i) for i in reversed(range(5))][::-1]
    assert a == b and len(set(a)) == 5
    assert all(0.0 < x <= 1.0 for x in a)
    assert gen.uniform(3, 1, 0) != gen.uniform(4, 1, 0) != gen.uniform(3, 2, 0)


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, 3.1415927, -2.5], dtype=np.float32)
    bits = gen.bf16_bits(x)
    back = gen.bf16_to_f64(bits)
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7: ties go to the even significand (1.0);
    # 1 + 3*2^-8 is halfway between 1 + 2^-7 and 1 + 2^-6: ties go to 1 + 2^-6.
    assert back.tolist()[:3] == [1.0, 1.0, 1.015625]
    assert abs(back[3] - 3.1415927) < 2 ** -7 and back[4] == -2.5


def test_weights_and_hidden_statistics_and_determinism():
    cfg = gen.CONFIGS["tiny"]
    wl = gen.make(cfg)
    wl2 = gen.make(cfg)
    assert (wl.W == wl2.W).all() and (wl.hidden_verify == wl2.hidden_verify).all()
    W = gen.bf16_to_f64(wl.W)
    assert abs(W.std() - 0.02) < 5e-4 and abs(W.mean()) < 2e-4
    assert wl.hidden_verify.shape == (cfg.B * cfg.D * cfg.M, cfg.H)
    assert wl.hidden_stage1.shape == (cfg.B * cfg.M, cfg.H)
    plain = gen.bf16_to_f64(wl.hidden_verify[: cfg.M])[wl.present[0, :, 1] == 0]
    assert abs(plain.std() - 1.0) < 0.05
    frac = wl.present.mean()
    assert 0.3 < frac < 0.7
    # depth d keeps depth d-1's peak most of the time (rho = 0.8) but not always
    same = (wl.token[:, :, 1:] == wl.token[:, :, :-1]) & (wl.present[:, :, 1:] == wl.present[:, :, :-1])
    assert 0.5 < same.mean() < 1.0


def test_planted_peaks_control_confidence_and_token():
    cfg = gen.CONFIGS["tiny"]
    wl = gen.make(cfg)
    tok, conf, _, _ = oracle.confidence(wl.hidden_stage1, wl.W)
    pres = wl.present[0, :, 0] == 1
    assert (tok[pres] == wl.token[0, :, 0][pres]).all()
    assert (conf[pres] > 0.9).mean() >= 0.8 and (conf[~pres] < 0.05).all()


def test_peak_scale_range_spans_the_threshold():
    from dataclasses import replace
    cfg = replace(gen.CONFIGS["tiny"], s_lo=1.0, s_hi=6.0, frac=1.0, B=4, seed=9)
    wl = gen.make(cfg)
    _, conf, _, _ = oracle.confidence(wl.hidden_stage1, wl.W)
    assert (conf < 0.5).sum() >= 10 and (conf > 0.9).sum() >= 10


def test_literal_gain_mode_keeps_confidences_low():
    from dataclasses import replace
    cfg = replace(gen.CONFIGS["tiny"], gain_mode=0)
    wl = gen.make(cfg)
    _, conf, _, _ = oracle.confidence(wl.hidden_stage1, wl.W)
    assert conf.max() < 0.1


def test_table_body_rows_and_levels():
    """The stand-in body: row indexing by committed neighbours, and confidences that grow with context."""
    import oracle
    cfg = gen.Config("t", B=2, H=256, V=1024, M=8, D=2, frac=0.6, s_lo=2.5, s_hi=3.5, seed=3)
    W = gen.weights(cfg)
    table, token, present, scale = gen.table_body(cfg, W)
    assert table.shape == (2, 8, 3, 256) and table.dtype == np.uint16
    mask = np.array([[1, 1, 0, 1, 0, 0, 1, 1],      # sequence 0 of block 0
                     [0, 1, 1, 1, 1, 1, 1, 0],      # sequence 1 of block 0
                     [1, 1, 1, 1, 1, 1, 1, 1],      # block 1
                     [0, 0, 0, 0, 0, 0, 0, 0]])
    rows = gen.table_rows(mask, seq_per_block=2)
    c = rows % 3
    assert c[0].tolist() == [0, 1, 0, 2, 1, 1, 1, 0]
    assert c[1].tolist() == [0, 1, 0, 0, 0, 0, 1, 0]
    assert c[2].tolist() == [0] * 8 and c[3].tolist() == [1, 2, 2, 2, 2, 2, 2, 1]
    assert (rows // 3 == np.array([[0, 1, 2, 3, 4, 5, 6, 7]] * 2 + [[8, 9, 10, 11, 12, 13, 14, 15]] * 2)).all()
    tok, conf, _, _ = oracle.confidence(table.reshape(-1, 256), W)
    tok, conf = tok.reshape(2, 8, 3), conf.reshape(2, 8, 3)
    pl = present == 1
    assert pl.any() and (~pl).any()
    assert (conf[pl][:, 2] > conf[pl][:, 0]).all() and (conf[pl][:, 2] > 0.9).all()
    assert (tok[pl][:, 2] == token[pl][:, 2]).all()
    assert (conf[~pl] < 0.1).all()
