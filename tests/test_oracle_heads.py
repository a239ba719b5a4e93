"""Pins (CPU only) of the oracle functions for the producers either side of the verify step: the LM head's
logits (a plain matrix product) and the drafter's LSTM cell, Eq. 1-8."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_07535_b200 import workloads as W


def _bits(rng, shape, scale=1.0):
    return W.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32)).reshape(shape)


def test_lm_head_logits_against_scalar_loops():
    rng = np.random.default_rng(0)
    h, w = _bits(rng, (3, 40)), _bits(rng, (7, 40))
    got = oracle.lm_head_logits(h, w)
    hf, wf = W.bf16_bits_to_f32(h).astype(np.float64), W.bf16_bits_to_f32(w).astype(np.float64)
    for n in range(3):
        for v in range(7):
            assert abs(got[n, v] - math.fsum(float(hf[n, k]) * float(wf[v, k]) for k in range(40))) < 1e-12
    # a one-hot hidden state picks a weight column; the arg-max over the vocabulary follows
    h1 = np.zeros((1, 40), np.uint16); h1[0, 5] = 0x3F80
    assert np.array_equal(oracle.lm_head_logits(h1, w)[0], wf[:, 5])
    assert oracle.row_argmax(oracle.lm_head_logits(h1, w).astype(np.float32))[0] == int(np.argmax(wf[:, 5]))


def test_alpha_of_eq_3_and_4():
    # n = 8 (the depth the paper drafts to), d = 12288 (Section 4.1): worked by hand
    a0 = 2.0 ** (-1.0 / 16.0)
    assert abs(a0 - 0.9576032806985737) < 1e-15
    assert abs(oracle.lstm_alpha(8, 12288) - 2 * a0 / ((1 - a0 * a0) * 12288)) < 1e-18
    assert abs(oracle.lstm_alpha(8, 12288) - 1.8776e-3) < 1e-6
    assert abs(oracle.lstm_alpha(1, 1) - 2 * 2 ** -0.5 / 0.5) < 1e-12          # alpha_0 = 1/sqrt(2): 2 sqrt(2)


def _torch_cell(h, e, w, z, alpha, eps=1e-5):
    """The same equations with library routines (torch fp64: linear, sigmoid, layer_norm, exact gelu)."""
    F = torch.nn.functional
    s = [F.linear(h, w[m]) + alpha * e for m in range(4)]
    gf, gi, go = torch.sigmoid(s[0]), torch.sigmoid(s[1]), torch.sigmoid(s[2])
    d = e.shape[-1]
    sc = F.gelu(F.layer_norm(s[3], (d,), eps=eps)) * gi
    zn = z * gf + sc
    return F.gelu(F.layer_norm(zn, (d,), eps=eps)) * go, zn


@pytest.mark.parametrize("M,d_in,d", [(1, 16, 24), (5, 64, 96), (3, 32, 32)])
def test_lstm_cell_against_library_routines(M, d_in, d):
    rng = np.random.default_rng(M)
    hb, eb, wb = _bits(rng, (M, d_in)), _bits(rng, (M, d)), _bits(rng, (4, d, d_in), 0.3)
    z = rng.standard_normal((M, d))
    alpha = 0.37
    hn, zn = oracle.lstm_cell(hb, eb, wb, z, alpha)
    t = lambda bits: torch.from_numpy(W.bf16_bits_to_f32(bits).astype(np.float64))
    rh, rz = _torch_cell(t(hb), t(eb), t(wb), torch.from_numpy(z), alpha)
    assert np.abs(hn - rh.numpy()).max() < 1e-12 and np.abs(zn - rz.numpy()).max() < 1e-12


def test_lstm_cell_special_cases():
    rng = np.random.default_rng(9)
    M, d_in, d = 2, 8, 12
    eb, z = _bits(rng, (M, d)), rng.standard_normal((M, d))
    hb = _bits(rng, (M, d_in))
    zero_w = np.zeros((4, d, d_in), np.uint16)
    # all weights zero and alpha = 0: every s is 0, gates are 1/2, f(0-vector) = gelu(0) = 0:
    # z' = z / 2 (Eq. 7) and h' = f(z / 2) / 2 (Eq. 8)
    hn, zn = oracle.lstm_cell(hb, eb, zero_w, z, 0.0)
    assert np.allclose(zn, z / 2, atol=1e-15)
    ln = (zn - zn.mean(-1, keepdims=True)) / np.sqrt(zn.var(-1, keepdims=True) + 1e-5)
    gelu = ln * 0.5 * (1 + np.vectorize(math.erf)(ln / math.sqrt(2)))
    assert np.allclose(hn, gelu / 2, atol=1e-14)
    # the cell state starts at zero: the first step's z is f(s^c) g^i alone, whatever the forget gate says
    wb = _bits(rng, (4, d, d_in))
    _, z1 = oracle.lstm_cell(hb, eb, wb, np.zeros((M, d)), 0.5)
    wb2 = wb.copy(); wb2[0] = _bits(rng, (d, d_in))           # another forget projection
    _, z2 = oracle.lstm_cell(hb, eb, wb2, np.zeros((M, d)), 0.5)
    assert np.array_equal(z1, z2)
    # alpha scales the embedding's share: with zero weights s = alpha e exactly
    _, z3 = oracle.lstm_cell(hb, eb, zero_w, np.zeros((M, d)), 2.0)
    e = W.bf16_bits_to_f32(eb).astype(np.float64)
    s = 2.0 * e
    ln = (s - s.mean(-1, keepdims=True)) / np.sqrt(s.var(-1, keepdims=True) + 1e-5)
    expect = ln * 0.5 * (1 + np.vectorize(math.erf)(ln / math.sqrt(2))) / (1 + np.exp(-s))
    assert np.allclose(z3, expect, atol=1e-14)
    # rows are independent
    hn_a, _ = oracle.lstm_cell(hb[:1], eb[:1], wb, z[:1], 0.5)
    hn_b, _ = oracle.lstm_cell(hb, eb, wb, z, 0.5)
    assert np.array_equal(hn_a[0], hn_b[0])


@pytest.mark.parametrize("mistake", ["gate_order", "norm_after_gate", "forget_on_candidate", "tanh_gelu"])
def test_planted_cell_mistakes_differ_from_the_library_form(mistake):
    """Plausible slips in the cell, written out on the CPU, are told apart by the library-routine pin."""
    rng = np.random.default_rng(4)
    M, d_in, d = 3, 16, 20
    t = lambda bits: torch.from_numpy(W.bf16_bits_to_f32(bits).astype(np.float64))
    h, e, w, z = t(_bits(rng, (M, d_in))), t(_bits(rng, (M, d))), t(_bits(rng, (4, d, d_in), 0.5)), torch.from_numpy(rng.standard_normal((M, d)))
    F = torch.nn.functional
    s = [F.linear(h, w[m]) + 0.4 * e for m in range(4)]
    gf, gi, go = torch.sigmoid(s[0]), torch.sigmoid(s[1]), torch.sigmoid(s[2])
    f = lambda x: F.gelu(F.layer_norm(x, (d,), eps=1e-5))
    if mistake == "gate_order":
        gf, gi = gi, gf
    sc = f(s[3]) * gi
    if mistake == "norm_after_gate":
        sc = f(s[3] * gi)
    zn = z * gf + sc
    if mistake == "forget_on_candidate":
        zn = z + sc * gf
    hn = f(zn) * go
    if mistake == "tanh_gelu":
        hn = F.gelu(F.layer_norm(zn, (d,), eps=1e-5), approximate="tanh") * go
    ref_h, ref_z = _torch_cell(h, e, w, z, 0.4)
    assert (hn - ref_h).abs().max() > 1e-6 or (zn - ref_z).abs().max() > 1e-6
