"""Pins for the oracle's two networks (Eq. 2, Eq. 6; architecture of Section 4.1.3)."""
import math

import numpy as np
import pytest
from scipy.special import expit

import oracle
import workloads as wl
from conftest import golden_lines

LN3 = math.log(3.0)


def _golden(name):
    for line in golden_lines("tiny_networks.txt"):
        key, val = line.split()
        if key == name:
            return float(val)
    raise KeyError(name)


def test_parameter_counts():
    # 1->128->128->128->32 and 128->64->64->64->64->1
    assert wl.enc_net_size() == 128 + 128 + 2 * (128 * 128 + 128) + 32 * 128 + 32 == 37408
    assert wl.head_net_size(128) == 128 * 64 + 64 + 3 * (64 * 64 + 64) + 64 + 1 == 20801


def test_encoder_hand_worked_value_and_layout():
    enc = np.array([LN3, 0.0, 0.0, 0.0,                # W1 [2][1], b1
                    0.0, 0.0, 4.0 / 3.0, 0.0, 0.0, 0.0,  # W2 [2][2] row-major [out][in], b2
                    1.0, 2.0, 0.5])                      # W3 [1][2], b3
    m = oracle.Model(1, 6.0, enc, np.zeros(16), k=1, l_max=0, enc_hidden=2, enc_layers=2,
                     head_hidden=1, head_layers=1)
    y, _ = oracle.encoder(m, 0, 0, 1.0)
    assert abs(y[0] - _golden("encoder_y")) < 1e-14


def test_head_hand_worked_value_and_layout():
    head = np.array([1.0, 0.0, -1.0, 0.0, 0.0, 0.0,      # W1 [2][2], b1
                     0.0, -4.0, 0.0, 0.0, 0.0, 0.0,      # W2 [2][2], b2
                     2.0, 4.0, -1.0])                    # w_out, b_out
    m = oracle.Model(1, 6.0, np.zeros(16), head, k=2, l_max=0, enc_hidden=1, enc_layers=1,
                     head_hidden=2, head_layers=2)
    e = oracle.head(m, 0, np.array([LN3, 5.0]))
    assert abs(e - _golden("head_e")) < 1e-14


def test_encoder_reduces_to_one_layer_when_inner_layers_are_zero():
    """With W2 = W3 = 0, b = 0 the residual layers add SiLU(0) = 0: y = W4 SiLU(w1 r + b1) + b4."""
    rng = np.random.default_rng(0)
    H, K = 128, 32
    w1, b1 = rng.standard_normal(H), rng.standard_normal(H)
    W4, b4 = rng.standard_normal((K, H)), rng.standard_normal(K)
    zero = np.zeros(H * H + H)
    enc = np.concatenate([w1, b1, zero, zero, W4.ravel(), b4])
    m = oracle.Model(1, 6.0, enc, np.zeros(wl.head_net_size(128)))
    for r in (0.7, 2.5, 5.9):
        pre = w1 * r + b1
        want = W4 @ (pre * expit(pre)) + b4
        y, _ = oracle.encoder(m, 0, 0, r)
        assert np.abs(y - want).max() < 1e-12


def test_encoder_selects_the_ordered_pair_network():
    enc, head = wl.make_weights(3, seed=5)
    m = oracle.Model(3, 6.0, enc, head)
    n = wl.enc_net_size()
    single = oracle.Model(1, 6.0, enc[(2 * 3 + 1) * n:(2 * 3 + 2) * n], head[:wl.head_net_size(128)])
    assert np.array_equal(oracle.encoder(m, 2, 1, 3.3)[0], oracle.encoder(single, 0, 0, 3.3)[0])
    assert not np.allclose(oracle.encoder(m, 2, 1, 3.3)[0], oracle.encoder(m, 1, 2, 3.3)[0])


def test_encoder_and_radial_derivatives_match_finite_differences():
    enc, head = wl.make_weights(2, seed=7)
    m = oracle.Model(2, 6.0, enc, head)
    for r in (1.3, 2.9, 4.4, 5.95):
        h = 1e-6
        for fn in (oracle.encoder, oracle.radial):
            _, d = fn(m, 1, 0, r)
            fd = (fn(m, 1, 0, r + h)[0] - fn(m, 1, 0, r - h)[0]) / (2 * h)
            assert np.abs(fd - d).max() < 1e-7 * max(1.0, np.abs(d).max())


def test_radial_feature_vanishes_smoothly_at_the_cutoff():
    enc, head = wl.make_weights(1, seed=9)
    m = oracle.Model(1, 6.0, enc, head)
    g, dg = oracle.radial(m, 0, 0, 6.0 - 1e-9)
    assert np.abs(g).max() < 1e-15 and np.abs(dg).max() < 1e-7
    g, dg = oracle.radial(m, 0, 0, 6.5)
    assert not g.any() and not dg.any()
    y, _ = oracle.encoder(m, 0, 0, 3.0)
    g, _ = oracle.radial(m, 0, 0, 3.0)           # envelope is exactly 1/2 at r_c / 2
    assert np.abs(g - 0.5 * y).max() < 1e-15


def test_head_gradient_matches_finite_differences_and_selects_species():
    enc, head = wl.make_weights(3, seed=11)
    m = oracle.Model(3, 6.0, enc, head)
    rng = np.random.default_rng(1)
    G = rng.standard_normal(128)
    e, dG = oracle.head(m, 1, G, want_grad=True)
    assert e == oracle.head(m, 1, G)
    assert e != oracle.head(m, 2, G)
    for i in (0, 31, 32, 77, 127):
        d = np.zeros(128); d[i] = 1e-6
        fd = (oracle.head(m, 1, G + d) - oracle.head(m, 1, G - d)) / 2e-6
        assert abs(fd - dG[i]) < 1e-8 * max(1.0, abs(dG[i]))


@pytest.mark.parametrize("chi_e,chi_r", [(1, 0), (2, 0), (0, 1), (2, 1)])
def test_species_conditioning_equals_the_pair_conditioned_model_with_tied_networks(chi_e, chi_r):
    """Section 3.2.2: an encoder conditioned on s_j only (or on nothing) is the pair-conditioned model whose C*C networks
    repeat the shared ones; likewise one universal regression network is C tied heads."""
    C = 3
    w = wl.make_workload(3, n_cells=3)
    enc, head = wl.workload_weights(3, C)
    ne, nh = wl.enc_net_size(), wl.head_net_size(128)
    enc_nets, head_nets = enc.reshape(C * C, ne), head.reshape(C, nh)
    enc_small = {0: enc_nets, 1: enc_nets[:C], 2: enc_nets[4:5]}[chi_e]
    head_small = {0: head_nets, 1: head_nets[1:2]}[chi_r]
    if chi_e == 0:
        tied_enc = enc_nets
    elif chi_e == 1:
        tied_enc = np.stack([enc_small[sj] for si in range(C) for sj in range(C)])
    else:
        tied_enc = np.stack([enc_small[0]] * (C * C))
    tied_head = head_nets if chi_r == 0 else np.stack([head_small[0]] * C)
    small = oracle.Model(C, w.r_cut, enc_small.ravel(), head_small.ravel(), chi_e=chi_e, chi_r=chi_r)
    tied = oracle.Model(C, w.r_cut, tied_enc.ravel(), tied_head.ravel())
    assert small.n_enc_nets == enc_small.shape[0] and small.n_head_nets == head_small.shape[0]
    rows = np.arange(0, w.n_atoms, 7)
    nl = oracle.neighbors(w.pos, w.species, C, w.box, w.r_cut, rows=rows)
    a = oracle.compute(small, w.pos, w.species, w.box, nl)
    b = oracle.compute(tied, w.pos, w.species, w.box, nl)
    assert abs(a["energy"] - b["energy"]) < 1e-12 * abs(b["energy"])
    assert np.abs(a["forces"] - b["forces"]).max() < 1e-13      # thread order of the force scatter differs run to run
    # and the conditioning matters: the fully conditioned model gives something else
    full = oracle.compute(oracle.Model(C, w.r_cut, enc, head), w.pos, w.species, w.box, nl)
    assert abs(full["energy"] - a["energy"]) > 1e-6 * abs(full["energy"])


def test_quintic_envelope_closed_form_values_and_contact_order():
    """f_c = 1 - 10 x^3 + 15 x^4 - 6 x^5: f_c(r_c / 2) = 1/2, f_c and its first two derivatives vanish at r_c, and
    f_c = 1 - O(x^3) near the origin.  Checked through g = f_c y on a random encoder."""
    enc, head = wl.make_weights(1, seed=9)
    m = oracle.Model(1, 6.0, enc, head, envelope=1)
    cosine = oracle.Model(1, 6.0, enc, head)

    def fc(r, eps=0.0):
        y, _ = oracle.encoder(m, 0, 0, r + eps)
        g, _ = oracle.radial(m, 0, 0, r + eps)
        return (g / y)[0]

    assert abs(fc(3.0) - 0.5) < 1e-15
    assert abs(fc(1.5) - (1 - 10 / 64 + 15 / 256 - 6 / 1024)) < 1e-15
    assert abs(fc(0.06) - 1.0) < 1.1e-5                        # 10 x^3 with x = 0.01
    # contact of third order at the cutoff: f_c(r_c - e) = 10 (e / r_c)^3 + O(e^4)
    for e in (0.06, 0.03):
        assert abs(fc(6.0 - e) / (10 * (e / 6.0) ** 3) - 1.0) < 3 * e / 6.0
    g, dg = oracle.radial(m, 0, 0, 6.2)
    assert not g.any() and not dg.any()
    # analytic derivative against a central difference, and the two envelopes really differ
    g0, dg0 = oracle.radial(m, 0, 0, 4.3)
    gp, _ = oracle.radial(m, 0, 0, 4.3 + 1e-6)
    gm, _ = oracle.radial(m, 0, 0, 4.3 - 1e-6)
    assert np.abs((gp - gm) / 2e-6 - dg0).max() < 1e-8 * max(1.0, np.abs(dg0).max())
    gc, _ = oracle.radial(cosine, 0, 0, 4.3)
    assert np.abs(gc - g0).max() > 1e-3 * np.abs(g0).max()
