"""CPU oracle for the forward pass of a Pairformer-style block on a packed multi-ragged pair state.

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, per-sample NumPy restatement of what the
method computes.  It shares no code with the CUDA library and the library never calls it; only
the tests, the smoke check and the benchmark's CPU-baseline leg may import it.

Form: one Python loop over samples; inside a sample, ordinary dense ``matmul``/``einsum`` on the
sample's own ``[N, N, C]`` view of the packed buffer (Eq. 2, packing: ``V[o_s:o_{s+1}]`` is the
sample's row-major reshape).  No padded ``B x N_max^2`` tensor is ever built here.  Working
precision is the ``dtype`` argument (float64 by default).

What each function follows:
  offsets_build        Sec. 3.1 (sample offsets ``o``), Fig. 2 (two-level row splits), Eq. 3
                       (coordinate map), App. A (invariants ``o_0 = 0``, ``o_{i+1}-o_i = p_i``, ``o_B = T``).
  pair_broadcast       Eq. 1 line 1 and Sec. 3.2 "Creating axes through broadcasting"; the
                       explicit-packed form ``u[rows] + v[cols]`` of the program figure; feature-wise
                       LayerNorm on the static tail (Sec. 3.3).  No activation at construction (App. A.1).
  tri_mul_out          Sec. 4.3 names the triangle multiplicative update of the Pairformer block;
                       its internals are the standard gated outgoing form (a reading; see below).
  tri_mul_in           the second direction of the same update (contraction over the first index); pinned by a
                       triple loop, torch einsum, and its relations to the outgoing form (transposed state, symmetric
                       state, a == b).
  row_attn_pairbias    Sec. 3.3 "Attention through packed blocks" (segments from cumulative lengths;
                       output adopts the query structure) and Sec. 4.3 (triangle attention with a
                       pair bias); internals are a reading (see below).
  col_attn_pairbias    the second (column-wise, "ending node") triangle attention of Sec. 4.3: the mirror image of
                       row_attn_pairbias; pinned by the exact transposition relation to it, library attention, and
                       scalar loops.
  single_attn_pairbias the pair-biased single attention of Sec. 4.3 (tokens attend tokens of the same sample, logits
                       biased by a projection of the pair state); pinned by library attention with an additive mask,
                       scalar loops, and its reduction to the token-order attention when the bias weights are zero.
  rect_*               the rectangular pair layout (N_i, M_i): Eq. 2 packing (sum N_i M_i rows), Eq. 4 (column reduction
                       over the M_i cells of a row; its mean divides by M_i, App. A.1), distinct row and column inputs.
  segment_reduce       Eq. 4 (pair reduction) and the mean of Eq. 1 line 3; App. A batch-axis
                       convention (``[1,2],[3,4]`` sums to ``[3,7]``).
  token_update         Eq. 1 line 3: ``X~ = X + g(mean_b P~[a,b,:])`` with ``g`` a bias-free projection.
  pair_transition      Eq. 1 line 2: ``P~ = P + h(LN(P))`` with ``h`` the SwiGLU feature update named there
                       (gate ``silu(x W_a^T)``, value ``x W_b^T``, output projection ``W_2``; expansion four in the
                       paper's settings, App. A.1), position-wise on the packed values.

Pins (tests/test_oracle_pins.py): the paper's printed (2,3) example, the ``[3,7]`` reduction,
structural invariants, closed forms, brute-force triple loops, an independent padded-and-masked
dense implementation (oracle/bruteforce_padded.py), and batch-composition invariance.

Parity unpinned: the *choice* of sub-layer internals (which gated form the triangle update takes,
that the row-wise attention is starting-node attention with a bias shared by all rows of a sample,
how blocks stack, the LayerNorm parameter draw).  The paper prints no value that depends on them;
they are pinned only by the agreement between this file and the brute-force padded computation.
"""
from __future__ import annotations

import numpy as np

LN_EPS = 1e-5


# --------------------------------------------------------------------------------------------
# structure
# --------------------------------------------------------------------------------------------
def offsets_build(lengths):
    """Offsets, level-2 row splits, position decode and gather maps for square pairs.

    tok_off[s]  = sum_{s'<s} N_s'            (token offsets, eta of Eq. 4)
    pair_off[s] = sum_{s'<s} N_s'^2          (sample offsets o in packed-cell space)
    row_splits[tok_off[s] + i] = pair_off[s] + i N_s, row_splits[T1] = T2   (1 + sum N entries)
    For packed position p = pair_off[s] + i N_s + j (Eq. 3): pos_sample[p] = s, pos_i[p] = i,
    pos_j[p] = j, rows[p] = tok_off[s] + i, cols[p] = tok_off[s] + j.
    Written as the literal nested loops over (s, i, j).
    """
    lengths = [int(n) for n in lengths]
    if any(n < 0 for n in lengths):
        raise ValueError("negative length")
    tok_off, pair_off = [0], [0]
    for n in lengths:
        tok_off.append(tok_off[-1] + n)
        pair_off.append(pair_off[-1] + n * n)
    row_splits, pos_s, pos_i, pos_j, rows, cols = [], [], [], [], [], []
    for s, n in enumerate(lengths):
        for i in range(n):
            row_splits.append(pair_off[s] + i * n)
            for j in range(n):
                pos_s.append(s)
                pos_i.append(i)
                pos_j.append(j)
                rows.append(tok_off[s] + i)
                cols.append(tok_off[s] + j)
    row_splits.append(pair_off[-1])
    return dict(
        tok_off=np.asarray(tok_off, dtype=np.int64),
        pair_off=np.asarray(pair_off, dtype=np.int64),
        row_splits=np.asarray(row_splits, dtype=np.int64),
        pos_sample=np.asarray(pos_s, dtype=np.int32),
        pos_i=np.asarray(pos_i, dtype=np.int32),
        pos_j=np.asarray(pos_j, dtype=np.int32),
        rows=np.asarray(rows, dtype=np.int64),
        cols=np.asarray(cols, dtype=np.int64),
    )


def offsets_only(lengths):
    """tok_off, pair_off and row_splits without the per-position maps (for large batches)."""
    lengths = [int(n) for n in lengths]
    tok_off, pair_off = [0], [0]
    for n in lengths:
        tok_off.append(tok_off[-1] + n)
        pair_off.append(pair_off[-1] + n * n)
    row_splits = []
    for s, n in enumerate(lengths):
        for i in range(n):
            row_splits.append(pair_off[s] + i * n)
    row_splits.append(pair_off[-1])
    return (np.asarray(tok_off, dtype=np.int64), np.asarray(pair_off, dtype=np.int64),
            np.asarray(row_splits, dtype=np.int64))


def decode_position(lengths, p):
    """(s, i, j) of one packed position p: the unique sample with pair_off[s] <= p < pair_off[s+1]
    (empty samples are never selected), then i = r div N_s, j = r mod N_s."""
    o = 0
    for s, n in enumerate(int(v) for v in lengths):
        if o <= p < o + n * n:
            r = p - o
            return s, r // n, r % n
        o += n * n
    raise IndexError("position outside the packed range")


# --------------------------------------------------------------------------------------------
# feature-wise pieces
# --------------------------------------------------------------------------------------------
def layer_norm(v, gamma, beta, eps=LN_EPS):
    """LayerNorm over the last (static feature) axis, biased variance, then affine."""
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    return (v - mu) / np.sqrt(var + eps) * gamma + beta


def sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def _as(dtype, *arrs):
    return [np.asarray(a, dtype=dtype) for a in arrs]


# --------------------------------------------------------------------------------------------
# the five calls
# --------------------------------------------------------------------------------------------
def pair_broadcast(x, lengths, W_a, W_b, ln_gamma, ln_beta, eps=LN_EPS, dtype=np.float64):
    """z[p,:] = LN_{c_z}(W_a x_i + W_b x_j) for p = (s,i,j).  Returns packed [T2, c_z]."""
    x, W_a, W_b, ln_gamma, ln_beta = _as(dtype, x, W_a, W_b, ln_gamma, ln_beta)
    out, t0 = [], 0
    for n in (int(v) for v in lengths):
        xs = x[t0:t0 + n]
        u = xs @ W_a.T                       # [n, c_z]  left projection
        v = xs @ W_b.T                       # [n, c_z]  right projection
        P = u[:, None, :] + v[None, :, :]    # (N,1,C)+(1,N,C) -> (N,N,C)
        out.append(layer_norm(P, ln_gamma, ln_beta, eps).reshape(n * n, W_a.shape[0]))
        t0 += n
    c_z = W_a.shape[0]
    return np.concatenate(out, axis=0) if out else np.zeros((0, c_z), dtype=dtype)


def tri_mul_out(z, lengths, W, eps=LN_EPS, dtype=np.float64, return_parts=False):
    """Outgoing triangle multiplicative update with residual, per sample:
        zh = LN_in(z);  a = sig(zh W_ag^T) * (zh W_ap^T);  b = sig(zh W_bg^T) * (zh W_bp^T)
        g = sig(zh W_g^T);  t[i,j,c] = sum_k a[i,k,c] b[j,k,c];  z <- z + g * (LN_out(t) W_o^T)
    """
    z = np.asarray(z, dtype=dtype)
    Wd = {k: np.asarray(v, dtype=dtype) for k, v in W.items()}
    out, parts, o = [], [], 0
    for n in (int(v) for v in lengths):
        zs = z[o:o + n * n].reshape(n, n, z.shape[1])
        zh = layer_norm(zs, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)
        a = sigmoid(zh @ Wd["W_ag"].T) * (zh @ Wd["W_ap"].T)
        b = sigmoid(zh @ Wd["W_bg"].T) * (zh @ Wd["W_bp"].T)
        g = sigmoid(zh @ Wd["W_g"].T)
        # per channel c the contraction is the matrix product A_c B_c^T; move c to the front so a
        # BLAS-backed batched matmul can serve as the step (still the plain per-sample definition)
        t = np.matmul(a.transpose(2, 0, 1), b.transpose(2, 1, 0)).transpose(1, 2, 0)
        upd = g * (layer_norm(t, Wd["ln_out_gamma"], Wd["ln_out_beta"], eps) @ Wd["W_o"].T)
        out.append((zs + upd).reshape(n * n, z.shape[1]))
        if return_parts:
            parts.append(dict(a=a, b=b, g=g, t=t))
        o += n * n
    res = np.concatenate(out, axis=0) if out else z.copy()
    return (res, parts) if return_parts else res


def tri_mul_in(z, lengths, W, eps=LN_EPS, dtype=np.float64, return_parts=False):
    """Incoming triangle multiplicative update with residual, per sample (Sec. 4.3 names the triangle
    multiplication of the Pairformer block; this is its second direction).  Same projections, gate, output
    normalisation and residual as the outgoing update; only the contraction runs over the FIRST index:
        t[i,j,c] = sum_k a[k,i,c] b[k,j,c]
    """
    z = np.asarray(z, dtype=dtype)
    Wd = {k: np.asarray(v, dtype=dtype) for k, v in W.items()}
    out, parts, o = [], [], 0
    for n in (int(v) for v in lengths):
        zs = z[o:o + n * n].reshape(n, n, z.shape[1])
        zh = layer_norm(zs, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)
        a = sigmoid(zh @ Wd["W_ag"].T) * (zh @ Wd["W_ap"].T)
        b = sigmoid(zh @ Wd["W_bg"].T) * (zh @ Wd["W_bp"].T)
        g = sigmoid(zh @ Wd["W_g"].T)
        # per channel c the contraction is the matrix product A_c^T B_c (a batched matmul serves as the step)
        t = np.matmul(a.transpose(2, 1, 0), b.transpose(2, 0, 1)).transpose(1, 2, 0)
        upd = g * (layer_norm(t, Wd["ln_out_gamma"], Wd["ln_out_beta"], eps) @ Wd["W_o"].T)
        out.append((zs + upd).reshape(n * n, z.shape[1]))
        if return_parts:
            parts.append(dict(a=a, b=b, g=g, t=t))
        o += n * n
    res = np.concatenate(out, axis=0) if out else z.copy()
    return (res, parts) if return_parts else res


def row_attn_pairbias(zx, lengths, W, H, d, eps=LN_EPS, order="pair", dtype=np.float64, return_parts=False):
    """Row-wise pair-biased softmax attention with residual.

    order="pair": zx is the packed pair state [T2, c].  For each sample, each pair row i and head h,
    the N positions j of the row attend over the positions k of the same row:
        zh = LN(z); q,k,v = zh W_{q,k,v}^T viewed [N,N,H,d]; bias = zh W_b^T [N,N,H]; g = sig(zh W_g^T)
        S[i,h,j,k] = <q[i,j,h,:], k[i,k,h,:]>/sqrt(d) + bias[j,k,h];  A = softmax_k S
        o[i,j,h,:] = sum_k A[i,h,j,k] v[i,k,h,:];  z <- z + (g * o) W_o^T
    The bias is shared by all rows i of the sample.
    order="token": zx is the packed token buffer [T1, c]; one attention row per sample
    (textbook variable-length self-attention over segments).
    ln_gamma/ln_beta absent -> no LN; W_b absent -> zero bias; W_g absent -> no gate.
    """
    zx = np.asarray(zx, dtype=dtype)
    Wd = {k: (None if v is None else np.asarray(v, dtype=dtype)) for k, v in W.items()}
    has_ln = Wd.get("ln_gamma") is not None
    W_b, W_g = Wd.get("W_b"), Wd.get("W_g")
    scale = 1.0 / np.sqrt(float(d))
    out, parts, o = [], [], 0
    for n in (int(v) for v in lengths):
        if n == 0:
            continue                              # an empty sample has no rows
        rows = n * n if order == "pair" else n
        R = n if order == "pair" else 1          # number of attention rows in this sample
        zs = zx[o:o + rows].reshape(R, n, zx.shape[1])
        zh = layer_norm(zs, Wd["ln_gamma"], Wd["ln_beta"], eps) if has_ln else zs
        q = (zh @ Wd["W_q"].T).reshape(R, n, H, d)
        k = (zh @ Wd["W_k"].T).reshape(R, n, H, d)
        v = (zh @ Wd["W_v"].T).reshape(R, n, H, d)
        # scores per (row, head) as a batched matrix product Q K^T (BLAS-backed, still the definition)
        S = np.matmul(q.transpose(0, 2, 1, 3), k.transpose(0, 2, 3, 1)) * scale      # [R, H, j, k]
        if W_b is not None:
            bias = zh @ W_b.T                    # [n, n, H] (pair order only: R == n)
            S = S + bias.transpose(2, 0, 1)[None, :, :, :]
        S = S - S.max(axis=-1, keepdims=True)
        A = np.exp(S)
        A = A / A.sum(axis=-1, keepdims=True)
        ov = np.matmul(A, v.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3).reshape(R, n, H * d)
        if W_g is not None:
            ov = sigmoid(zh @ W_g.T) * ov
        out.append((zs + ov @ Wd["W_o"].T).reshape(rows, zx.shape[1]))
        if return_parts:
            parts.append(dict(q=q, k=k, v=v, A=A, o=ov))
        o += rows
    res = np.concatenate(out, axis=0) if out else zx.copy()
    return (res, parts) if return_parts else res


def col_attn_pairbias(z, lengths, W, H, d, eps=LN_EPS, dtype=np.float64, return_parts=False):
    """Column-wise ("ending node") pair-biased softmax attention with residual, the second triangle attention of
    the Pairformer block (Sec. 4.3).  For each sample, each pair COLUMN j and head h, the N positions i of the
    column attend over the positions k of the same column:
        zh = LN(z); q,k,v = zh W_{q,k,v}^T viewed [N,N,H,d]; bias = zh W_b^T [N,N,H]; g = sig(zh W_g^T)
        S[j,h,i,k] = <q[i,j,h,:], k[k,j,h,:]>/sqrt(d) + bias[k,i,h];  A = softmax_k S
        o[i,j,h,:] = sum_k A[j,h,i,k] v[k,j,h,:];  z <- z + (g * o) W_o^T
    The bias is shared by all columns j of the sample.  (The mirror image of row_attn_pairbias: the same formulas
    with the roles of the two pair indices exchanged.)
    """
    z = np.asarray(z, dtype=dtype)
    Wd = {k: (None if v is None else np.asarray(v, dtype=dtype)) for k, v in W.items()}
    W_b, W_g = Wd.get("W_b"), Wd.get("W_g")
    scale = 1.0 / np.sqrt(float(d))
    out, parts, o = [], [], 0
    for n in (int(v) for v in lengths):
        if n == 0:
            continue
        zs = z[o:o + n * n].reshape(n, n, z.shape[1])
        zh = layer_norm(zs, Wd["ln_gamma"], Wd["ln_beta"], eps)
        q = (zh @ Wd["W_q"].T).reshape(n, n, H, d)           # [i, j, h, :]
        k = (zh @ Wd["W_k"].T).reshape(n, n, H, d)           # [k, j, h, :]
        v = (zh @ Wd["W_v"].T).reshape(n, n, H, d)
        # scores per (column j, head): Q_j K_j^T with Q_j = q[:, j], K_j = k[:, j]
        S = np.matmul(q.transpose(1, 2, 0, 3), k.transpose(1, 2, 3, 0)) * scale      # [j, h, i, k]
        if W_b is not None:
            bias = zh @ W_b.T                                # [row, col, H]; the score of (i, k) takes bias[k, i]
            S = S + bias.transpose(2, 1, 0)[None, :, :, :]
        S = S - S.max(axis=-1, keepdims=True)
        A = np.exp(S)
        A = A / A.sum(axis=-1, keepdims=True)
        ov = np.matmul(A, v.transpose(1, 2, 0, 3))           # [j, h, i, :]
        ov = ov.transpose(2, 0, 1, 3).reshape(n, n, H * d)   # [i, j, h d]
        if W_g is not None:
            ov = sigmoid(zh @ W_g.T) * ov
        out.append((zs + ov @ Wd["W_o"].T).reshape(n * n, z.shape[1]))
        if return_parts:
            parts.append(dict(q=q, k=k, v=v, A=A, o=ov))
        o += n * n
    res = np.concatenate(out, axis=0) if out else z.copy()
    return (res, parts) if return_parts else res


def single_attn_pairbias(x, z, lengths, W, H, d, eps=LN_EPS, dtype=np.float64, return_parts=False):
    """Pair-biased single attention (Sec. 4.3: the tokens of a sample attend the tokens of the same sample, the
    logits biased by a projection of the pair state), with residual, per sample:
        xh = LN_x(x); q,k,v = xh W_{q,k,v}^T viewed [N,H,d]; g = sig(xh W_g^T); bias = LN_z(z) W_b^T [N,N,H]
        S[h,j,k] = <q[j,h,:], k[k,h,:]>/sqrt(d) + bias[j,k,h];  A = softmax_k S
        o[j,h,:] = sum_k A[h,j,k] v[k,h,:];  x <- x + (g * o) W_o^T
    x [T1, c_s] packed tokens, z [T2, c_z] packed pair state (read only).
    """
    x = np.asarray(x, dtype=dtype)
    z = np.asarray(z, dtype=dtype)
    Wd = {k: (None if v is None else np.asarray(v, dtype=dtype)) for k, v in W.items()}
    scale = 1.0 / np.sqrt(float(d))
    out, parts, ot, op_ = [], [], 0, 0
    for n in (int(v) for v in lengths):
        if n == 0:
            continue
        xs = x[ot:ot + n]
        zs = z[op_:op_ + n * n].reshape(n, n, z.shape[1])
        xh = layer_norm(xs, Wd["ln_gamma"], Wd["ln_beta"], eps)
        q = (xh @ Wd["W_q"].T).reshape(n, H, d)
        k = (xh @ Wd["W_k"].T).reshape(n, H, d)
        v = (xh @ Wd["W_v"].T).reshape(n, H, d)
        bias = layer_norm(zs, Wd["ln_z_gamma"], Wd["ln_z_beta"], eps) @ Wd["W_b"].T      # [j, k, H]
        S = np.matmul(q.transpose(1, 0, 2), k.transpose(1, 2, 0)) * scale + bias.transpose(2, 0, 1)   # [H, j, k]
        S = S - S.max(axis=-1, keepdims=True)
        A = np.exp(S)
        A = A / A.sum(axis=-1, keepdims=True)
        ov = np.matmul(A, v.transpose(1, 0, 2)).transpose(1, 0, 2).reshape(n, H * d)
        ov = sigmoid(xh @ Wd["W_g"].T) * ov
        out.append(xs + ov @ Wd["W_o"].T)
        if return_parts:
            parts.append(dict(q=q, k=k, v=v, bias=bias, A=A, o=ov))
        ot += n
        op_ += n * n
    res = np.concatenate(out, axis=0) if out else x.copy()
    return (res, parts) if return_parts else res


# --------------------------------------------------------------------------------------------
# rectangular pairs (N_i, M_i): the paper's second pair layout (Eq. 2: pairs (N_i, M_i, C) pack as (sum N_i M_i, C);
# Eq. 4: a column reduction groups the M_i cells of one row; App. A.1: the rectangular variant has distinct row and
# column inputs and divides its column mean by M_i)
# --------------------------------------------------------------------------------------------
def rect_offsets(lengths_n, lengths_m):
    """Offsets of a batch of rectangular pairs: tokn_off / tokm_off (prefix sums of N_i / M_i), pair_off (prefix sums
    of N_i M_i), the level-2 row splits (one group of M_s cells per row (s, a): sum N + 1 entries), and the decode of
    every packed cell p = pair_off[s] + a M_s + b into (s, a, b)."""
    n = np.asarray(lengths_n, dtype=np.int64)
    m = np.asarray(lengths_m, dtype=np.int64)
    assert n.shape == m.shape and np.all(n >= 0) and np.all(m >= 0)
    tokn = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    tokm = np.concatenate([[0], np.cumsum(m)]).astype(np.int64)
    po = np.concatenate([[0], np.cumsum(n * m)]).astype(np.int64)
    rs = np.empty(int(tokn[-1]) + 1, dtype=np.int64)
    ps, pi, pj = [], [], []
    for s in range(len(n)):
        for a in range(int(n[s])):
            rs[tokn[s] + a] = po[s] + a * m[s]
        if n[s] and m[s]:
            ps.append(np.full(int(n[s] * m[s]), s, dtype=np.int32))
            pi.append(np.repeat(np.arange(n[s], dtype=np.int32), int(m[s])))
            pj.append(np.tile(np.arange(m[s], dtype=np.int32), int(n[s])))
    rs[-1] = po[-1]
    cat = lambda l: np.concatenate(l) if l else np.zeros(0, dtype=np.int32)
    return dict(tokn_off=tokn, tokm_off=tokm, pair_off=po, row_splits=rs, pos_sample=cat(ps), pos_i=cat(pi), pos_j=cat(pj))


def rect_pair_broadcast(x, y, lengths_n, lengths_m, W_a, W_b, ln_gamma, ln_beta, eps=LN_EPS, dtype=np.float64):
    """Rectangular broadcast: z[(s, a, b), :] = LN(W_a x_{s,a} + W_b y_{s,b}) gamma + beta with x the row tokens
    [sum N, c_s] and y the column tokens [sum M, c_s]; output [sum N M, c_z]."""
    x, y, W_a, W_b, g, bt = _as(dtype, x, y, W_a, W_b, ln_gamma, ln_beta)
    out, on, om = [], 0, 0
    for n, m in zip((int(v) for v in lengths_n), (int(v) for v in lengths_m)):
        u = x[on:on + n] @ W_a.T
        v = y[om:om + m] @ W_b.T
        out.append(layer_norm(u[:, None, :] + v[None, :, :], g, bt, eps).reshape(n * m, W_a.shape[0]))
        on += n
        om += m
    return np.concatenate(out, axis=0) if out else np.zeros((0, W_a.shape[0]), dtype=dtype)


def rect_block_forward(x, y, lengths_n, lengths_m, w, eps=LN_EPS, dtype=np.float64):
    """Single-pair-single block on rectangular pairs (Eq. 1 with distinct row and column inputs): broadcast + LN,
    the position-wise SwiGLU transition, the mean over the column axis (divided by M_s, Eq. 4) and the token update of
    the row tokens.  Returns (x', z)."""
    off = rect_offsets(lengths_n, lengths_m)
    z = rect_pair_broadcast(x, y, lengths_n, lengths_m, eps=eps, dtype=dtype, **w["broadcast"])
    z = pair_transition(z, w["transition"], eps=eps, dtype=dtype)
    mrow = segment_reduce(z, off["row_splits"], "mean", dtype=dtype)
    return token_update(x, mrow, w["reduce"]["W_r"], dtype=dtype), z


def segment_reduce(v, splits, op="mean", dtype=np.float64):
    """out[g,:] = sum (or mean) of rows splits[g] .. splits[g+1]-1 of v.  An empty segment gives
    zeros (there is nothing to average; the pair path never produces one because an empty
    sample has no rows)."""
    v = np.asarray(v, dtype=dtype)
    splits = [int(t) for t in splits]
    G = len(splits) - 1
    out = np.zeros((G,) + v.shape[1:], dtype=dtype)
    for g in range(G):
        lo, hi = splits[g], splits[g + 1]
        if hi > lo:
            acc = v[lo:hi].sum(axis=0)
            out[g] = acc / (hi - lo) if op == "mean" else acc
    return out


def token_update(x, m, W_r, dtype=np.float64):
    """x' = x + m W_r^T  (the projection g of Eq. 1 line 3, bias-free)."""
    x, m, W_r = _as(dtype, x, m, W_r)
    return x + m @ W_r.T


def silu(v):
    return v * sigmoid(v)


def pair_transition(z, W, eps=LN_EPS, dtype=np.float64):
    """Eq. 1 line 2 on the packed values: z' = z + (silu(LN(z) W_a^T) * (LN(z) W_b^T)) W_2^T, position by position
    (no sample structure enters: the update acts on the static channel tail only).  W: ln_gamma, ln_beta [c],
    W_a, W_b [hidden, c], W_2 [c, hidden]; all projections bias-free."""
    z = np.asarray(z, dtype=dtype)
    Wd = {k: np.asarray(v, dtype=dtype) for k, v in W.items()}
    zh = layer_norm(z, Wd["ln_gamma"], Wd["ln_beta"], eps)
    h = silu(zh @ Wd["W_a"].T) * (zh @ Wd["W_b"].T)
    return z + h @ Wd["W_2"].T


# --------------------------------------------------------------------------------------------
# the same definitions evaluated at selected positions of one sample (for samples too large to
# run whole on the CPU); pinned to the full functions above in tests/test_oracle_pins.py
# --------------------------------------------------------------------------------------------
def tri_mul_out_at(zs, W, positions, eps=LN_EPS, dtype=np.float64):
    """Outgoing triangle update of one sample at the listed (i, j).  ``zs[i]`` is pair row i of the
    sample's state, an [n, c_z] array (``zs`` may be the [n, n, c_z] array or a mapping that holds
    only the rows needed): only rows i and j enter t[i,j,:] = sum_k a[i,k,:] b[j,k,:]."""
    Wd = {k: np.asarray(v, dtype=dtype) for k, v in W.items()}
    out = []
    for (i, j) in positions:
        ri, rj = np.asarray(zs[i], dtype=dtype), np.asarray(zs[j], dtype=dtype)
        zi = layer_norm(ri, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)        # [n, c_z]
        zj = layer_norm(rj, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)
        a_i = sigmoid(zi @ Wd["W_ag"].T) * (zi @ Wd["W_ap"].T)               # a[i, k, :]
        b_j = sigmoid(zj @ Wd["W_bg"].T) * (zj @ Wd["W_bp"].T)               # b[j, k, :]
        t = (a_i * b_j).sum(axis=0)
        g = sigmoid(zi[j] @ Wd["W_g"].T)
        out.append(ri[j] + g * (layer_norm(t, Wd["ln_out_gamma"], Wd["ln_out_beta"], eps) @ Wd["W_o"].T))
    return np.stack(out)


def tri_mul_in_at(zs, W, positions, eps=LN_EPS, dtype=np.float64):
    """Incoming triangle update of one sample at the listed (i, j).  ``zs`` is the sample's [n, n, c_z]
    state (anything indexable as zs[:, i]): only columns i and j enter t[i,j,:] = sum_k a[k,i,:] b[k,j,:]."""
    Wd = {k: np.asarray(v, dtype=dtype) for k, v in W.items()}
    out = []
    for (i, j) in positions:
        ci, cj = np.asarray(zs[:, i], dtype=dtype), np.asarray(zs[:, j], dtype=dtype)   # [n, c_z] each
        zi = layer_norm(ci, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)
        zj = layer_norm(cj, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps)
        a_i = sigmoid(zi @ Wd["W_ag"].T) * (zi @ Wd["W_ap"].T)               # a[k, i, :]
        b_j = sigmoid(zj @ Wd["W_bg"].T) * (zj @ Wd["W_bp"].T)               # b[k, j, :]
        t = (a_i * b_j).sum(axis=0)
        zij = cj[i]                                                          # z[i, j]
        g = sigmoid(layer_norm(zij, Wd["ln_in_gamma"], Wd["ln_in_beta"], eps) @ Wd["W_g"].T)
        out.append(zij + g * (layer_norm(t, Wd["ln_out_gamma"], Wd["ln_out_beta"], eps) @ Wd["W_o"].T))
    return np.stack(out)


def row_attn_pairbias_at(zs, W, H, d, positions, eps=LN_EPS, dtype=np.float64):
    """Row-wise pair-biased attention of one sample at the listed (i, j) (``zs`` as in
    tri_mul_out_at): query j of row i attends over the keys of row i with bias[j, :, h] taken
    from pair row j."""
    Wd = {k: (None if v is None else np.asarray(v, dtype=dtype)) for k, v in W.items()}
    out = []
    for (i, j) in positions:
        ri, rj = np.asarray(zs[i], dtype=dtype), np.asarray(zs[j], dtype=dtype)
        n = ri.shape[0]
        zi = layer_norm(ri, Wd["ln_gamma"], Wd["ln_beta"], eps)
        zj = layer_norm(rj, Wd["ln_gamma"], Wd["ln_beta"], eps)
        q = (zi[j] @ Wd["W_q"].T).reshape(H, d)
        k = (zi @ Wd["W_k"].T).reshape(n, H, d)
        v = (zi @ Wd["W_v"].T).reshape(n, H, d)
        bias = zj @ Wd["W_b"].T                                               # [n(k), H]
        o = np.zeros((H, d), dtype=dtype)
        for h in range(H):
            sc = k[:, h, :] @ q[h] / np.sqrt(float(d)) + bias[:, h]
            sc = sc - sc.max()
            e = np.exp(sc)
            o[h] = (e / e.sum()) @ v[:, h, :]
        gate = sigmoid(zi[j] @ Wd["W_g"].T)
        out.append(ri[j] + (gate * o.reshape(H * d)) @ Wd["W_o"].T)
    return np.stack(out)


# --------------------------------------------------------------------------------------------
# compositions
# --------------------------------------------------------------------------------------------
def col_attn_pairbias_at(zs, W, H, d, positions, eps=LN_EPS, dtype=np.float64):
    """Column-wise pair-biased attention of one sample at the listed (i, j).  ``zs`` is indexable as zs[:, c]
    (pair column c, an [n, c_z] array): query i of column j attends over the keys of column j with
    bias[:, h] = bias[k, i, h] taken from pair column i."""
    Wd = {k: (None if v is None else np.asarray(v, dtype=dtype)) for k, v in W.items()}
    out = []
    for (i, j) in positions:
        ci, cj = np.asarray(zs[:, i], dtype=dtype), np.asarray(zs[:, j], dtype=dtype)
        n = cj.shape[0]
        zi = layer_norm(ci, Wd["ln_gamma"], Wd["ln_beta"], eps)               # LN(z[k, i]) over k
        zj = layer_norm(cj, Wd["ln_gamma"], Wd["ln_beta"], eps)               # LN(z[k, j]) over k
        q = (zj[i] @ Wd["W_q"].T).reshape(H, d)
        k = (zj @ Wd["W_k"].T).reshape(n, H, d)
        v = (zj @ Wd["W_v"].T).reshape(n, H, d)
        bias = zi @ Wd["W_b"].T if Wd.get("W_b") is not None else np.zeros((n, H), dtype=dtype)   # [k, H]
        o = np.zeros((H, d), dtype=dtype)
        for h in range(H):
            sc = k[:, h, :] @ q[h] / np.sqrt(float(d)) + bias[:, h]
            w = np.exp(sc - sc.max())
            o[h] = (w / w.sum()) @ v[:, h, :]
        ov = o.reshape(H * d)
        if Wd.get("W_g") is not None:
            ov = sigmoid(zj[i] @ Wd["W_g"].T) * ov
        out.append(cj[i] + ov @ Wd["W_o"].T)
    return np.stack(out)


def pair_broadcast_add(z_prev, x, lengths, W_a, W_b, ln_gamma, ln_beta, eps=LN_EPS, dtype=np.float64):
    """Persistent pair stream: z = z_prev + LN(u_i + v_j) gamma + beta, the broadcast of Eq. 1 line 1 accumulated onto
    the state of the previous block instead of replacing it."""
    return np.asarray(z_prev, dtype=dtype) + pair_broadcast(x, lengths, W_a, W_b, ln_gamma, ln_beta, eps=eps, dtype=dtype)


def block_forward(x, lengths, w, H, d, eps=LN_EPS, dtype=np.float64, z_prev=None):
    """One Pairformer-style block: broadcast+LN, outgoing triangle update, row-wise pair-biased
    attention, segmented mean over j and token update.  Returns (x', z).  With z_prev the broadcast is
    accumulated onto it (persistent pair stream)."""
    _, _, row_splits = offsets_only(lengths)
    if z_prev is None:
        z = pair_broadcast(x, lengths, eps=eps, dtype=dtype, **w["broadcast"])
    else:
        z = pair_broadcast_add(z_prev, x, lengths, eps=eps, dtype=dtype, **w["broadcast"])
    z = tri_mul_out(z, lengths, w["trimul"], eps=eps, dtype=dtype)
    z = row_attn_pairbias(z, lengths, w["attn"], H, d, eps=eps, order="pair", dtype=dtype)
    m = segment_reduce(z, row_splits, "mean", dtype=dtype)
    x2 = token_update(x, m, w["reduce"]["W_r"], dtype=dtype)
    return x2, z


def stack_forward(x, lengths, blocks, H, d, eps=LN_EPS, dtype=np.float64, persistent=False):
    """Stacked blocks.  persistent=False: block b+1 rebuilds the pair state from the tokens block b returned (Eq. 1).
    persistent=True: the pair state is a stream of its own, z_b = z_{b-1} + LN(broadcast of the tokens) before the
    pair sub-layers of block b (the Pairformer keeps a persistent pair state, Sec. 2); block 0 starts it."""
    z = None
    x = np.asarray(x, dtype=dtype)
    for w in blocks:
        x, z = block_forward(x, lengths, w, H, d, eps=eps, dtype=dtype, z_prev=z if persistent else None)
    return x, z


def token_forward(x, lengths, w, H, d, dtype=np.float64):
    """Single-ragged special case: zero-bias attention over each sample's tokens, residual,
    then a segmented mean over the token axis.  Returns (x', pooled [B, c])."""
    x2 = row_attn_pairbias(x, lengths, w, H, d, order="token", dtype=dtype)
    tok_off, _, _ = offsets_only(lengths)
    pooled = segment_reduce(x2, tok_off, "mean", dtype=dtype)
    return x2, pooled
