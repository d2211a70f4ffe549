"""Brute-force padded-and-masked dense computation of the same block (float64, tiny inputs only).

TEST INFRASTRUCTURE ONLY: a second, independent implementation used to pin the packed oracle.
It follows the reference-semantics contract of App. A: interpreting a packed result logically
must agree with the dense reference on the logically interpreted inputs.  Everything here lives in
the padded envelope ``[B, N_max, N_max, C]`` with a validity mask (true = valid, App. A): operands
are zeroed at invalid contraction indices, attention keys outside the sample get a ``-inf`` score,
and means divide by the true counts.  It imports nothing from the packed oracle.
"""
from __future__ import annotations

import numpy as np


def _ln(v, g, b, eps):
    m = v.sum(-1, keepdims=True) / v.shape[-1]
    c = v - m
    s2 = (c * c).sum(-1, keepdims=True) / v.shape[-1]
    return c * (s2 + eps) ** -0.5 * g + b


def _sig(v):
    return np.exp(-np.logaddexp(0.0, -v))


def pad_tokens(x, lengths):
    B, Nm = len(lengths), max(max(lengths), 1)
    xp = np.zeros((B, Nm, x.shape[1]))
    t = 0
    for s, n in enumerate(lengths):
        xp[s, :n] = x[t:t + n]
        t += n
    return xp


def masks(lengths):
    Nm = max(max(lengths), 1)
    valid1 = np.arange(Nm)[None, :] < np.asarray(lengths)[:, None]          # [B, Nm]
    valid2 = valid1[:, :, None] & valid1[:, None, :]                        # [B, Nm, Nm]
    return valid1, valid2


def unpad_pairs(zp, lengths):
    return np.concatenate([zp[s, :n, :n].reshape(n * n, -1) for s, n in enumerate(lengths)], axis=0)


def unpad_tokens(xp, lengths):
    return np.concatenate([xp[s, :n] for s, n in enumerate(lengths)], axis=0)


def block_forward_padded(x, lengths, w, H, d, eps=1e-5):
    """Returns (x' packed [T1, c_s], z packed [T2, c_z]) computed entirely in the padded envelope."""
    lengths = [int(n) for n in lengths]
    x = np.asarray(x, dtype=np.float64)
    W = {k: {kk: np.asarray(vv, dtype=np.float64) for kk, vv in v.items()} for k, v in w.items()}
    B, Nm = len(lengths), max(max(lengths), 1)
    valid1, valid2 = masks(lengths)
    xp = pad_tokens(x, lengths)

    # broadcast + LN over the envelope
    wb = W["broadcast"]
    u = np.einsum("bnc,zc->bnz", xp, wb["W_a"])
    v = np.einsum("bnc,zc->bnz", xp, wb["W_b"])
    z = _ln(u[:, :, None, :] + v[:, None, :, :], wb["ln_gamma"], wb["ln_beta"], eps)

    # triangle multiplicative update (outgoing): zero a, b where the (i,k) / (j,k) cell is invalid
    wt = W["trimul"]
    zh = _ln(z, wt["ln_in_gamma"], wt["ln_in_beta"], eps)
    a = _sig(np.einsum("bikc,hc->bikh", zh, wt["W_ag"])) * np.einsum("bikc,hc->bikh", zh, wt["W_ap"])
    b = _sig(np.einsum("bjkc,hc->bjkh", zh, wt["W_bg"])) * np.einsum("bjkc,hc->bjkh", zh, wt["W_bp"])
    a = a * valid2[..., None]
    b = b * valid2[..., None]
    g = _sig(np.einsum("bijc,zc->bijz", zh, wt["W_g"]))
    t = np.einsum("bikh,bjkh->bijh", a, b)
    z = z + g * np.einsum("bijh,zh->bijz", _ln(t, wt["ln_out_gamma"], wt["ln_out_beta"], eps), wt["W_o"])

    # row-wise pair-biased attention: keys outside the sample get -inf
    wa = W["attn"]
    zh = _ln(z, wa["ln_gamma"], wa["ln_beta"], eps)
    c_z = z.shape[-1]
    q = np.einsum("bijc,ec->bije", zh, wa["W_q"]).reshape(B, Nm, Nm, H, d)
    k = np.einsum("bijc,ec->bije", zh, wa["W_k"]).reshape(B, Nm, Nm, H, d)
    vv = np.einsum("bijc,ec->bije", zh, wa["W_v"]).reshape(B, Nm, Nm, H, d)
    bias = np.einsum("bjkc,hc->bjkh", zh, wa["W_b"])
    gate = _sig(np.einsum("bijc,ec->bije", zh, wa["W_g"]))
    o = np.zeros((B, Nm, Nm, H, d))
    for bb in range(B):
        for i in range(Nm):
            for h in range(H):
                S = q[bb, i, :, h, :] @ k[bb, i, :, h, :].T / np.sqrt(d) + bias[bb, :, :, h]
                S = np.where(valid1[bb][None, :], S, -np.inf)
                S = S - S.max(axis=1, keepdims=True)
                E = np.exp(S)
                o[bb, i, :, h, :] = (E / E.sum(axis=1, keepdims=True)) @ vv[bb, i, :, h, :]
    z = z + np.einsum("bije,ze->bijz", gate * o.reshape(B, Nm, Nm, H * d), wa["W_o"])

    # masked mean over j with the true counts, token update
    cnt = np.maximum(np.asarray(lengths, dtype=np.float64), 1.0)[:, None, None]
    m = (z * valid2[..., None]).sum(axis=2) / cnt
    xo = xp + np.einsum("bnz,sz->bns", m, W["reduce"]["W_r"])
    return unpad_tokens(xo, lengths), unpad_pairs(z, lengths)


def token_forward_padded(x, lengths, w, H, d):
    """Padded masked self-attention over tokens (zero bias, no LN, no gate) + masked mean pool."""
    lengths = [int(n) for n in lengths]
    x = np.asarray(x, dtype=np.float64)
    W = {k: np.asarray(v, dtype=np.float64) for k, v in w.items()}
    B, Nm = len(lengths), max(max(lengths), 1)
    valid1, _ = masks(lengths)
    xp = pad_tokens(x, lengths)
    q = (xp @ W["W_q"].T).reshape(B, Nm, H, d)
    k = (xp @ W["W_k"].T).reshape(B, Nm, H, d)
    v = (xp @ W["W_v"].T).reshape(B, Nm, H, d)
    S = np.einsum("bqhe,bkhe->bhqk", q, k) / np.sqrt(d)
    S = np.where(valid1[:, None, None, :], S, -np.inf)
    S = S - S.max(-1, keepdims=True)
    E = np.exp(S)
    A = E / E.sum(-1, keepdims=True)
    o = np.einsum("bhqk,bkhe->bqhe", A, v).reshape(B, Nm, H * d)
    xo = xp + o @ W["W_o"].T
    cnt = np.maximum(np.asarray(lengths, dtype=np.float64), 1.0)[:, None]
    pooled = (xo * valid1[..., None]).sum(axis=1) / cnt
    return unpad_tokens(xo, lengths), pooled
