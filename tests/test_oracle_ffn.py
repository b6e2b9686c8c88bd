"""Pins for the oracle of Eq. 6 (s <- LN(FFN(s) + s)): scalar loops, a hand-computed layer norm, torch's library
routines, special cases with closed forms, invariants, and planted mistakes that the pins must catch."""
import math

import numpy as np
import torch

from oracle import ffn_oracle


def _weights(seed, d, hid):
    rng = np.random.default_rng(seed)
    return dict(W1=rng.standard_normal((d, hid)) / math.sqrt(d), b1=0.3 * rng.standard_normal(hid),
                W2=rng.standard_normal((hid, d)) / math.sqrt(hid), b2=0.3 * rng.standard_normal(d),
                g=1.0 + 0.2 * rng.standard_normal(d), beta=0.2 * rng.standard_normal(d))


def test_layer_norm_hand_computed():
    # y = (1, 2, 3, 4): mean 2.5, biased variance 1.25
    out = ffn_oracle.layer_norm(np.array([1.0, 2.0, 3.0, 4.0]), np.ones(4), np.zeros(4), eps=0.0)
    s = math.sqrt(1.25)
    np.testing.assert_allclose(out, [-1.5 / s, -0.5 / s, 0.5 / s, 1.5 / s], rtol=1e-15)
    # gain and shift act after the normalisation, element by element
    out = ffn_oracle.layer_norm(np.array([1.0, 2.0, 3.0, 4.0]), np.array([2.0, 0.0, 1.0, -1.0]),
                                np.array([0.5, 7.0, 0.0, 1.0]), eps=0.0)
    np.testing.assert_allclose(out, [-3.0 / s + 0.5, 7.0, 0.5 / s, -1.5 / s + 1.0], rtol=1e-15)
    # eps sits inside the square root, added to the variance
    out = ffn_oracle.layer_norm(np.array([0.0, 2.0]), np.ones(2), np.zeros(2), eps=3.0)   # var 1 -> sqrt(4) = 2
    np.testing.assert_allclose(out, [-0.5, 0.5], rtol=1e-15)


def test_rows_match_scalar_loops():
    d, hid = 5, 7
    w = _weights(1, d, hid)
    rng = np.random.default_rng(2)
    s = rng.standard_normal((3, d))
    got = ffn_oracle.ffn_rows(s, **w)
    for i in range(3):
        h = [max(sum(s[i, k] * w["W1"][k, j] for k in range(d)) + w["b1"][j], 0.0) for j in range(hid)]
        y = [sum(h[j] * w["W2"][j, e] for j in range(hid)) + w["b2"][e] + s[i, e] for e in range(d)]
        mean = sum(y) / d
        var = sum((v - mean) ** 2 for v in y) / d
        for e in range(d):
            want = (y[e] - mean) / math.sqrt(var + 1e-5) * w["g"][e] + w["beta"][e]
            assert abs(got[i, e] - want) < 1e-12


def test_rows_match_torch_library_routines():
    d, hid = 16, 64
    w = _weights(3, d, hid)
    rng = np.random.default_rng(4)
    s = rng.standard_normal((9, d))
    t = {k: torch.from_numpy(np.asarray(v)) for k, v in w.items()}
    x = torch.from_numpy(s)
    h = torch.relu(torch.nn.functional.linear(x, t["W1"].T, t["b1"]))
    y = torch.nn.functional.linear(h, t["W2"].T, t["b2"]) + x
    want = torch.nn.functional.layer_norm(y, (d,), t["g"], t["beta"], eps=1e-5).numpy()
    np.testing.assert_allclose(ffn_oracle.ffn_rows(s, **w), want, rtol=1e-12, atol=1e-12)


def test_zero_ffn_gives_layer_norm_of_the_input():
    d, hid = 8, 32
    w = _weights(5, d, hid)
    w["W2"] = np.zeros((hid, d))
    w["b2"] = np.zeros(d)
    s = np.random.default_rng(6).standard_normal((4, d))
    np.testing.assert_allclose(ffn_oracle.ffn_rows(s, **w), ffn_oracle.layer_norm(s, w["g"], w["beta"]), rtol=1e-14)


def test_relu_switches_off_negative_hidden_units():
    d, hid = 6, 12
    w = _weights(7, d, hid)
    s = np.abs(np.random.default_rng(8).standard_normal((5, d)))      # positive inputs
    w["W1"] = -np.abs(w["W1"])                                        # every pre-activation negative ...
    w["b1"] = -np.abs(w["b1"])
    want = ffn_oracle.layer_norm(s + w["b2"], w["g"], w["beta"])      # ... so FFN(s) = b2
    np.testing.assert_allclose(ffn_oracle.ffn_rows(s, **w), want, rtol=1e-14)
    # flipping the sign of the first layer makes every unit active: FFN is then affine, (s W1 + b1) W2 + b2
    w["W1"], w["b1"] = -w["W1"], -w["b1"]
    y = (s @ w["W1"] + w["b1"]) @ w["W2"] + w["b2"] + s
    np.testing.assert_allclose(ffn_oracle.ffn_rows(s, **w), ffn_oracle.layer_norm(y, w["g"], w["beta"]), rtol=1e-13)


def test_normalised_output_has_zero_mean_and_the_expected_variance():
    d, hid = 32, 128
    w = _weights(9, d, hid)
    w["g"] = np.ones(d)
    w["beta"] = np.zeros(d)
    s = np.random.default_rng(10).standard_normal((11, d))
    out = ffn_oracle.ffn_rows(s, **w)
    y = np.maximum(s @ w["W1"] + w["b1"], 0) @ w["W2"] + w["b2"] + s
    var = y.var(axis=1)                                               # biased
    np.testing.assert_allclose(out.mean(axis=1), 0.0, atol=1e-14)
    np.testing.assert_allclose(out.var(axis=1), var / (var + 1e-5), rtol=1e-12)


def test_forward_touches_only_the_rows_of_non_empty_segments():
    d, hid, S, Lp = 8, 32, 4, 5
    w = _weights(11, d, hid)
    rng = np.random.default_rng(12)
    lengths = np.array([20, 7, 0, 4], dtype=np.int32)                 # 5, 2, 0, 1 non-empty segments
    offs = np.array([0, 2, 5, 6, 8], dtype=np.int32)
    Hp = rng.standard_normal((8, Lp, d))
    out = ffn_oracle.ffn_forward(Hp, lengths, offs, S, **w)
    nseg = [5, 5, 2, 2, 2, 0, 1, 1]
    for c in range(8):
        for j in range(Lp):
            if j < nseg[c]:
                np.testing.assert_allclose(out[c, j], ffn_oracle.ffn_rows(Hp[c, j], **w), rtol=1e-14)
            else:
                assert not out[c, j].any()


def test_planted_mistakes_are_caught():
    """Each variant below is a plausible slip; every one must move the result well away from the oracle's."""
    d, hid = 8, 8                                                     # square so that a transposed weight still runs
    w = _weights(13, d, hid)
    s = np.random.default_rng(14).standard_normal((6, d))
    ref = ffn_oracle.ffn_rows(s, **w)

    def ln(y, biased=True, eps_inside=True):
        mean = y.mean(axis=1, keepdims=True)
        var = y.var(axis=1, keepdims=True, ddof=0 if biased else 1)
        den = np.sqrt(var + 1e-5) if eps_inside else np.sqrt(var) + 1e-5
        return (y - mean) / den * w["g"] + w["beta"]

    hidden = np.maximum(s @ w["W1"] + w["b1"], 0)
    variants = {
        "no residual": ln(hidden @ w["W2"] + w["b2"]),
        "W1 transposed": ln(np.maximum(s @ w["W1"].T + w["b1"], 0) @ w["W2"] + w["b2"] + s),
        "W2 transposed": ln(hidden @ w["W2"].T + w["b2"] + s),
        "no relu": ln((s @ w["W1"] + w["b1"]) @ w["W2"] + w["b2"] + s),
        "unbiased variance": ln(hidden @ w["W2"] + w["b2"] + s, biased=False),
        "no b1": ln(np.maximum(s @ w["W1"], 0) @ w["W2"] + w["b2"] + s),
        "gain before normalisation": ln((hidden @ w["W2"] + w["b2"] + s) * w["g"]) ,
    }
    np.testing.assert_allclose(ln(hidden @ w["W2"] + w["b2"] + s), ref, rtol=1e-13)   # the unmodified restatement agrees
    for name, v in variants.items():
        assert np.abs(v - ref).max() > 1e-2, name
