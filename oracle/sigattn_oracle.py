"""Plain float64 definition of sigmoid self-attention and of its analytic gradient.

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg, never by the product path.  No code is shared with
the CUDA kernels; this file depends on numpy alone.

What it computes, per (batch, head), all in float64:

  forward (Eq. 3 of Section 2; Algorithm 1 of Appendix F reaches the same result,
  tiling only reorders the sums)
      x_ij = scale * <q_i, k_j> + b - m_h * |i - j|
      P_ij = sigmoid(x_ij),  set to 0 where causal and j > i
      O    = P V

  backward (sigmoid column of the forward/backward table in Appendix F.1;
  Algorithm 2 reaches the same result)
      dV = P^T dO
      dP = dO V^T
      dS = P * (1 - P) * dP          (0 where masked)
      dQ = scale * dS K
      dK = scale * dS^T Q

Readings of the paper taken here
  * The bias b is added after the 1/sqrt(d) scaling, once per logit (Eq. 3 defines
    sigma(u) = sigmoid(u + b) with u the scaled logit).
  * The causal mask multiplies sigma(.) and keeps the diagonal (the n = 3 example in
    the sequence-length-normalisation ablation, Appendix G): a masked weight is
    exactly 0, not sigmoid(b), and passes no gradient.
  * The table in Appendix F.1 and Algorithm 2 print the factor sqrt(d) in dQ and dK.
    The chain rule through S = Q K^T / sqrt(d) gives 1/sqrt(d) = scale; central finite
    differences (tests) confirm scale and reject sqrt(d).  Algorithm 2 also swaps
    indices in its dV and dP lines; the table's dV = P^T dO and dP = dO V^T are used.
  * The paper prints no ALiBi formula.  The linear-bias form it cites is used: the
    head's positive slope m_h times the distance |i - j| is subtracted from the scaled
    logit (not multiplied by scale); for causal calls only j <= i survives, which is
    the usual m_h * (i - j).
  * The bias may differ per sequence and per head: the speech models use b = -log n with
    n the length of each sample and ablate a learnable bias (Section 5.4, Appendix G.4),
    and a learnable scalar b replaces LayerScale in Appendix G.2.2.  `bias` is therefore
    a scalar or anything that broadcasts to [B, H]; it enters x_ij additively, so its
    gradient is db[b, h] = sum_ij dS_ij (the chain rule through x = u + b; masked entries
    carry dS = 0).  The paper prints no formula for db.
  * Keys and values may have fewer heads than the queries (multi-query and grouped-query
    attention; the ablation of Section 5.1 uses multi-query attention): k, v are
    [B, H_kv, N, D] with H a multiple of H_kv, query head h reads key/value head
    h // (H / H_kv) (consecutive query heads share one), and dK, dV of a key/value head
    are the sums over the query heads that read it.  The paper gives no layout; this is
    the usual one.
  * The paper defines self-attention (as many queries as keys).  Generation with a cache
    of earlier keys and values, where its inference gains are measured (Appendix F.3), has
    N_q queries against N_k >= N_q keys: q is [B, H, N_q, D], k and v are [B, H_kv, N_k, D],
    and the queries are the LAST N_q positions, i.e. query i sits at position
    i + N_k - N_q for the causal mask (keys j <= i + N_k - N_q are kept) and for the
    position bias.  N_q = N_k is the paper's case.  Without a causal mask and without
    slopes the positions play no role and any N_q, N_k are allowed (cross-attention).
  * Keys and values split into contiguous shards (over devices, or over thread blocks):
    sigmoid attention has no row normalisation, so O is the plain sum over shards of the
    attention of all queries against one shard, dQ likewise, and dK, dV of a shard need only
    that shard (the distributed setting the paper leaves open in its Limitations).  A shard
    call must place the queries relative to ITS first key: `pos0` is the position of query
    row 0 minus the position of the shard's first key (default N_k - N_q as above) and may
    be negative; a query that lies before every key of the shard gets weight 0 everywhere.

  * Batches of sequences of different lengths, padded to a common N (the speech batches of
    Section 5.4): with `seqlens[b] = n_b <= N`, keys j >= n_b get weight 0 like masked keys,
    query rows i >= n_b produce all-zero rows of O and take no part in any gradient (their
    dQ rows are zero, dK and dV do not see them).  The paper does not print this; it is the
    usual padding mask, and it makes the call equal to separate calls on the unpadded
    sequences.  Only for N_q = N_k.
  * The same batches stored without padding, one after the other along the row axis (B = 1,
    T = sum of the lengths rows): `cu_seqlens` holds the S + 1 row offsets 0 = c_0 <= c_1 <= ...
    <= c_S = T, sequence s owns rows [c_s, c_{s+1}) of q, k and v.  The definition is the one
    mask the layout implies: the weight of (query i, key j) is kept only if both rows belong to
    the same sequence (a block-diagonal mask times, if asked for, the causal mask; positions are
    counted within the sequence, which leaves i - j unchanged), and `bias` may then be an array
    that broadcasts to [S, H], one bias per sequence and head (b = -log n_s).  That this equals
    separate calls on the S sequences is what the tests check.
  * Sequence-length normalisation (the ablation in Appendix G that compares b = -log n with
    the scaling n^-alpha sigma(Q K^T / sqrt(d)) V): every row of O is multiplied by one
    factor r_i.  Without a mask r_i = n^-alpha for all rows.  For the causal form the paper
    prints an n = 3 matrix whose rows read 1, 0.5^-alpha, 0.33^-alpha under the label
    n^-alpha; taken literally 0.5^-alpha = 2^alpha would grow with the row, against the
    label and against the purpose (dividing by the number of keys a row sees), so it is read
    as r_i = (i + 1)^-alpha = (1 / (i + 1))^alpha, i + 1 being the number of keys row i keeps.
    With N_q != N_k the count is pos_i + 1 with pos_i the query's position.  The factor does
    not depend on Q, K, V, so the backward is the plain one with dO replaced by r_i dO_i; a
    bias and slopes may be combined with it.  `row_scale` takes any vector of N_q factors,
    `seqlen_norm` builds the paper's.

Every function is pinned by tests that do not call back into this file's own
formulae (closed forms, brute-force loops, finite differences, the paper's second
form of the forward, the printed n = 3 mask): there is no "parity unpinned" part.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "sigmoid",
    "causal_mask",
    "position_bias",
    "attention_weights",
    "sigattn_fwd",
    "sigattn_bwd",
    "sigattn_bwd_dbias",
    "sigattn_fwd_sequence_form",
    "seqlen_norm",
]


def sigmoid(x):
    """sigmoid(x) = 1 / (1 + exp(-x)) (Eq. 3), evaluated without overflow.

    For x >= 0 the definition is used as printed; for x < 0 the algebraically equal
    exp(x) / (1 + exp(x)) is used so that exp never sees a large positive argument.
    """
    x = np.asarray(x, dtype=np.float64)
    out = np.empty_like(x)
    pos = x >= 0
    out[pos] = 1.0 / (1.0 + np.exp(-x[pos]))
    e = np.exp(x[~pos])
    out[~pos] = e / (1.0 + e)
    return out


def _query_offset(n, n_q, pos0):
    """Position of query row 0 relative to key 0: given, or n - n_q (queries at the end)."""
    n_q = n if n_q is None else n_q
    return n_q, (n - n_q if pos0 is None else int(pos0))


def causal_mask(n: int, i0: int = 0, i1: int | None = None, n_q: int | None = None, pos0: int | None = None):
    """Rows i0..i1-1 of the n x n lower-triangular 0/1 matrix, diagonal included
    (the matrix M printed for n = 3 in Appendix G's normalisation ablation).

    With n_q query rows against n keys query i sits at position i + pos0 relative to key
    0 (pos0 = n - n_q unless given; see the module header), so the row keeps keys
    j <= i + pos0; a row whose position lies before key 0 keeps none."""
    n_q, off = _query_offset(n, n_q, pos0)
    i1 = n_q if i1 is None else i1
    i = np.arange(i0, i1)[:, None] + off
    j = np.arange(n)[None, :]
    return (j <= i).astype(np.float64)


def position_bias(n: int, slope: float, i0: int = 0, i1: int | None = None, n_q: int | None = None,
                  pos0: int | None = None):
    """Additive linear position bias -slope * |i - j| for rows i0..i1-1 (Appendix F.4
    names ALiBi; see the module header for the reading); the distance is taken from the
    query's position i + pos0 (pos0 = n - n_q unless given)."""
    n_q, off = _query_offset(n, n_q, pos0)
    i1 = n_q if i1 is None else i1
    i = np.arange(i0, i1, dtype=np.float64)[:, None] + float(off)
    j = np.arange(n, dtype=np.float64)[None, :]
    return -float(slope) * np.abs(i - j)


def attention_weights(q, k, scale, bias, causal, slope=0.0, i0=0, i1=None, pos0=None, seqlen=None):
    """P for query rows i0..i1-1 of one head: sigmoid(scale * q k^T + b + position
    bias), times the causal mask and, with `seqlen`, times the padding mask (rows and
    columns >= seqlen are 0).  q: [n_q, d], k: [n, d] float64."""
    n_q, n = q.shape[0], k.shape[0]
    i1 = n_q if i1 is None else i1
    x = scale * (q[i0:i1] @ k.T) + bias
    if slope != 0.0:
        x = x + position_bias(n, slope, i0, i1, n_q, pos0)
    p = sigmoid(x)
    if causal:
        p = p * causal_mask(n, i0, i1, n_q, pos0)
    if seqlen is not None:
        valid_rows = (np.arange(i0, i1) < int(seqlen)).astype(np.float64)[:, None]
        valid_cols = (np.arange(n) < int(seqlen)).astype(np.float64)[None, :]
        p = p * valid_rows * valid_cols
    return p


def _as_f64(*arrays):
    return [np.ascontiguousarray(a, dtype=np.float64) for a in arrays]


def _slopes(alibi_slopes, num_heads):
    if alibi_slopes is None:
        return np.zeros(num_heads, dtype=np.float64)
    s = np.asarray(alibi_slopes, dtype=np.float64).reshape(-1)
    if s.shape[0] != num_heads:
        raise ValueError("alibi_slopes must hold one slope per head")
    return s


def _bias_per_head(bias, num_batch, num_heads):
    """Scalar, [B], [B, 1], [1, H] or [B, H] bias -> float64 [B, H]."""
    b = np.asarray(bias, dtype=np.float64)
    if b.ndim == 1 and b.shape[0] == num_batch and num_batch != num_heads:
        b = b[:, None]
    return np.ascontiguousarray(np.broadcast_to(b, (num_batch, num_heads)))


def _kv_group(num_heads, k):
    """Query heads per key/value head."""
    h_kv = k.shape[1]
    if h_kv < 1 or num_heads % h_kv != 0:
        raise ValueError("the number of query heads must be a multiple of the number of key/value heads")
    return num_heads // h_kv


def _seqlens(seqlens, num_batch, n_q, n_k):
    if seqlens is None:
        return [None] * num_batch
    if n_q != n_k:
        raise ValueError("seqlens need as many query rows as key rows")
    s = np.asarray(seqlens).reshape(-1)
    if s.shape[0] != num_batch or np.any(s < 0) or np.any(s > n_q):
        raise ValueError("seqlens must hold one length in [0, N] per batch entry")
    return [int(x) for x in s]


def seqlen_norm(n_q, alpha, causal, n_k=None, pos0=None):
    """Row factors of the sequence-length normalisation (Appendix G, ablation of n^-alpha
    against the bias; see the header for the reading of the causal form): without a mask
    n_k^-alpha for every row, causal (pos_i + 1)^-alpha with pos_i = i + pos0 the query's
    position, i.e. one over the number of keys the row keeps, to the power alpha.  A row
    that keeps no key (position before key 0) gets factor 0.  Returns float64 [n_q]."""
    n_k = n_q if n_k is None else n_k
    _, off = _query_offset(n_k, n_q, pos0)
    if not causal:
        return np.full(n_q, float(n_k) ** (-float(alpha)), dtype=np.float64)
    count = np.arange(n_q, dtype=np.float64) + float(off) + 1.0
    r = np.zeros(n_q, dtype=np.float64)
    r[count >= 1.0] = count[count >= 1.0] ** (-float(alpha))
    return r


def _row_scale(row_scale, n_q):
    if row_scale is None:
        return np.ones(n_q, dtype=np.float64)
    r = np.asarray(row_scale, dtype=np.float64).reshape(-1)
    if r.shape[0] != n_q:
        raise ValueError("row_scale must hold one factor per query row")
    return r


def _cu_seqlens(cu_seqlens, num_batch, n_q, n_k):
    """Row offsets of a packed batch -> (offsets, sequence index of every row)."""
    c = np.asarray(cu_seqlens).reshape(-1).astype(np.int64)
    if num_batch != 1 or n_q != n_k:
        raise ValueError("a packed batch has B = 1 and as many query rows as key rows")
    if c.shape[0] < 2 or c[0] != 0 or c[-1] != n_q or np.any(np.diff(c) < 0):
        raise ValueError("cu_seqlens must rise from 0 to the number of rows")
    seq_of_row = np.searchsorted(c, np.arange(n_q), side="right") - 1
    return c, seq_of_row


def _row_ranges(n, row_block):
    """Query rows are independent in the forward and enter dK, dV only through a sum
    over rows, so they may be visited in slabs to bound memory (an n x n float64 matrix
    is 2 GiB at n = 16384).  row_block=None visits all rows at once."""
    step = n if not row_block else int(row_block)
    return [(a, min(n, a + step)) for a in range(0, n, step)]


def sigattn_fwd(q, k, v, scale, bias, causal=False, alibi_slopes=None, row_block=None, pos0=None, seqlens=None,
                row_scale=None, cu_seqlens=None):
    """O = sigmoid(scale * Q K^T + b [+ position bias]) [* causal mask] V  (Eq. 3).

    q: [B, H, N, D]; k, v: [B, H_kv, N, D] with H a multiple of H_kv (any float dtype;
    converted to float64).
    bias: scalar, or an array that broadcasts to [B, H] (one bias per sequence and head).
    pos0: position of query row 0 relative to key row 0 (default: rows of k minus rows of q).
    row_scale: one factor per query row (sequence-length normalisation), or None.
    cu_seqlens: row offsets of a packed batch (B = 1; see header), or None.
    Returns O as float64 [B, H, N, D].
    """
    q, k, v = _as_f64(q, k, v)
    B, H, N, D = q.shape          # N counts query rows; k, v may hold more (or fewer) rows
    if cu_seqlens is not None:
        return _packed_all(q, k, v, None, scale, bias, causal, alibi_slopes, cu_seqlens)[0]
    group = _kv_group(H, k)
    slopes = _slopes(alibi_slopes, H)
    bias_bh = _bias_per_head(bias, B, H)
    lens = _seqlens(seqlens, B, N, k.shape[2])
    r = _row_scale(row_scale, N)
    o = np.zeros((B, H, N, D), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            hk = h // group
            for i0, i1 in _row_ranges(N, row_block):
                p = attention_weights(q[b, h], k[b, hk], scale, bias_bh[b, h], causal, slopes[h], i0, i1, pos0,
                                      lens[b])
                o[b, h, i0:i1] = r[i0:i1, None] * (p @ v[b, hk])
    return o


def _packed_all(q, k, v, d_o, scale, bias, causal, alibi_slopes, cu_seqlens):
    """Packed batch (see header): block-diagonal mask over the T x T weights of each head, one
    bias per (sequence, head).  Returns (O, dQ, dK, dV, dbias[S, H]); gradients are None without d_o."""
    B, H, T, D = q.shape
    group = _kv_group(H, k)
    slopes = _slopes(alibi_slopes, H)
    c, seq = _cu_seqlens(cu_seqlens, B, T, k.shape[2])
    S = c.shape[0] - 1
    bias_sh = _bias_per_head(bias, S, H)
    same = (seq[:, None] == seq[None, :]).astype(np.float64)       # both rows in one sequence
    o = np.zeros_like(q)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dbias = np.zeros((S, H), dtype=np.float64)
    for h in range(H):
        hk = h // group
        x = scale * (q[0, h] @ k[0, hk].T) + bias_sh[seq, h][:, None]
        if slopes[h] != 0.0:
            x = x + position_bias(T, slopes[h])
        p = sigmoid(x) * same
        if causal:
            p = p * causal_mask(T)
        o[0, h] = p @ v[0, hk]
        if d_o is None:
            continue
        dv[0, hk] += p.T @ d_o[0, h]
        dp = d_o[0, h] @ v[0, hk].T
        ds = p * (1.0 - p) * dp
        dq[0, h] = scale * (ds @ k[0, hk])
        dk[0, hk] += scale * (ds.T @ q[0, h])
        np.add.at(dbias[:, h], seq, ds.sum(axis=1))
    if d_o is None:
        return o, None, None, None, None
    return o, dq, dk, dv, dbias


def _bwd_all(q, k, v, d_o, scale, bias, causal, alibi_slopes, row_block, pos0=None, seqlens=None, row_scale=None,
             cu_seqlens=None):
    q, k, v, d_o = _as_f64(q, k, v, d_o)
    if cu_seqlens is not None:
        return _packed_all(q, k, v, d_o, scale, bias, causal, alibi_slopes, cu_seqlens)[1:]
    B, H, N, D = q.shape
    group = _kv_group(H, k)
    slopes = _slopes(alibi_slopes, H)
    bias_bh = _bias_per_head(bias, B, H)
    lens = _seqlens(seqlens, B, N, k.shape[2])
    r = _row_scale(row_scale, N)
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    dbias = np.zeros((B, H), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            hk = h // group
            for i0, i1 in _row_ranges(N, row_block):
                p = attention_weights(q[b, h], k[b, hk], scale, bias_bh[b, h], causal, slopes[h], i0, i1, pos0,
                                      lens[b])
                do_rows = r[i0:i1, None] * d_o[b, h, i0:i1]   # O = r (P V): the factor passes to dO
                dv[b, hk] += p.T @ do_rows
                dp = do_rows @ v[b, hk].T
                ds = p * (1.0 - p) * dp
                dq[b, h, i0:i1] = scale * (ds @ k[b, hk])
                dk[b, hk] += scale * (ds.T @ q[b, h, i0:i1])
                dbias[b, h] += ds.sum()
    return dq, dk, dv, dbias


def sigattn_bwd(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, row_block=None, pos0=None,
                seqlens=None, row_scale=None, cu_seqlens=None):
    """Gradients of L = sum(O * dO) with respect to Q, K, V (sigmoid column of the
    forward/backward table in Appendix F.1, with the 1/sqrt(d) factor; see header).

    bias: scalar, or an array that broadcasts to [B, H].  k, v may have fewer heads
    than q (see header).
    Returns (dQ, dK, dV), float64, shaped like q, k, v.
    """
    return _bwd_all(q, k, v, d_o, scale, bias, causal, alibi_slopes, row_block, pos0, seqlens, row_scale,
                    cu_seqlens)[:3]


def sigattn_bwd_dbias(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None, row_block=None, pos0=None,
                      seqlens=None, row_scale=None, cu_seqlens=None):
    """Gradient of L = sum(O * dO) with respect to a bias held per (batch, head):
    db[b, h] = sum_ij dS_ij with dS = P (1 - P) dP as in sigattn_bwd (see header).  A
    bias shared by several heads or sequences gets the sum of their entries.

    Returns float64 [B, H] ([S, H], one row per sequence, for a packed batch).
    """
    return _bwd_all(q, k, v, d_o, scale, bias, causal, alibi_slopes, row_block, pos0, seqlens, row_scale,
                    cu_seqlens)[3]


def sigattn_bwd_dtemp(q, k, v, d_o, scale, bias, causal=False, alibi_slopes=None):
    """Gradient of L = sum(O * dO) with respect to a temperature t that multiplies the scaled logit,
    x_ij = e^t * scale * <q_i, k_j> + b (the learnable temperature of Section 5 / Appendix G.2.2),
    taken at t = 0: the caller passes scale * e^t as `scale`.  dx_ij/dt = scale <q_i, k_j>, so
    dt[b, h] = sum_ij dS_ij * scale * <q_i, k_j> with dS = P (1 - P) dP as in sigattn_bwd; the position
    bias does not depend on t.  Written from the logits, not from dQ.  Plain [B, H, N, D] shapes only.

    Returns float64 [B, H].
    """
    q, k, v, d_o = _as_f64(q, k, v, d_o)
    B, H, N, D = q.shape
    slopes = _slopes(alibi_slopes, H)
    bias_bh = _bias_per_head(bias, B, H)
    dt = np.zeros((B, H), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            p = attention_weights(q[b, h], k[b, h], scale, bias_bh[b, h], causal, slopes[h])
            ds = p * (1.0 - p) * (d_o[b, h] @ v[b, h].T)
            dt[b, h] = np.sum(ds * (scale * (q[b, h] @ k[b, h].T)))
    return dt


def sigattn_fwd_sequence_form(q, k, v, scale, n_bias):
    """Second form of the forward, valid at b = -log(n_bias), non-causal, no position
    bias (Eq. 4): y_i = sum_j exp(s_ij) / (exp(s_ij) + n_bias) v_j with s the scaled
    logit.  Kept separate from sigattn_fwd on purpose: it never calls sigmoid()."""
    q, k, v = _as_f64(q, k, v)
    B, H, N, D = q.shape
    o = np.zeros((B, H, N, D), dtype=np.float64)
    for b in range(B):
        for h in range(H):
            e = np.exp(scale * (q[b, h] @ k[b, h].T))
            o[b, h] = (e / (e + float(n_bias))) @ v[b, h]
    return o
