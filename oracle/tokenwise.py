"""fp64 CPU oracle for the token-wise operators in front of the first-layer
attention (Sec. 3.3.2, EmbedCache and RoPECache; Eq. 1 without the rotation).

TEST INFRASTRUCTURE ONLY: only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import this module.  It shares no code with the CUDA
path and imports nothing from it.

Sec. 3.3.2 lists the operators that act on every token independently:
embedding H = Embed(x), the attention norm H^ = Norm(H) (an RMS norm for the
models the paper evaluates), and the projections Q, K = RoPE(H^ W_QK),
V = H^ W_V.  The rotation itself is `oracle.rope`; this module stops at the
pre-rotation projections, which is what the attention entry points consume.

Each function is the textbook definition written with numpy in double
precision; a library matmul is the only non-trivial primitive.

The paper runs its models in bf16 and says nothing more about the precision of
these operators.  Reading taken here ("model precision"): the norm output and
the projection output are each rounded once to bf16, as a bf16 model stores
them; everything between two roundings is exact (fp64).  `round_bf16`
implements that rounding from its definition.
"""
import numpy as np


def round_bf16(x):
    """Round to the nearest value with an 8-bit significand (bf16), ties to the
    even significand.  Values stay float64.  Normal range only: bf16 shares
    fp32's exponent range, which nothing here approaches."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                    # x = m * 2^e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0), e - 8)   # np.rint rounds halves to even


def embed(table, token_ids):
    """H = Embed(x): row `token_ids[i]` of the table (Sec. 3.3.2)."""
    table = np.asarray(table, dtype=np.float64)
    ids = np.asarray(token_ids, dtype=np.int64)
    if ids.size and (ids.min() < 0 or ids.max() >= table.shape[0]):
        raise IndexError("token id out of range")
    return table[ids]


def rms_norm(h, weight, eps):
    """H^ = Norm(H), RMS norm: h / sqrt(mean(h^2) + eps) * weight, per token."""
    h = np.asarray(h, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * w


def qkv_project(h_hat, w_qkv, n_q_heads, n_kv_heads, head_dim):
    """Pre-rotation projections of Eq. 1.  `w_qkv` is [(Hq + 2 Hkv) * d, d_model],
    one row per output feature: the Q heads, then the K heads, then the V
    heads.  Returns q [n, Hq, d], k [n, Hkv, d], v [n, Hkv, d]."""
    h_hat = np.asarray(h_hat, dtype=np.float64)
    w = np.asarray(w_qkv, dtype=np.float64)
    n = h_hat.shape[0]
    nq, nk = n_q_heads * head_dim, n_kv_heads * head_dim
    assert w.shape == (nq + 2 * nk, h_hat.shape[1])
    y = h_hat @ w.T
    q = y[:, :nq].reshape(n, n_q_heads, head_dim)
    k = y[:, nq:nq + nk].reshape(n, n_kv_heads, head_dim)
    v = y[:, nq + nk:].reshape(n, n_kv_heads, head_dim)
    return q, k, v


def tokenwise_qkv(table, norm_weight, w_qkv, eps, n_q_heads, n_kv_heads, head_dim,
                  token_ids=None, hidden=None, model_precision=True):
    """Embed -> Norm -> projections for a list of tokens (Sec. 3.3.2), from token
    ids or from given hidden states.  With `model_precision` the norm output and
    the projections are rounded to bf16 (see the module text); without it nothing
    is rounded.  Returns (h, q, k, v): h is the embedding output the EmbedCache
    keeps."""
    assert (token_ids is None) != (hidden is None)
    h = embed(table, token_ids) if hidden is None else np.asarray(hidden, dtype=np.float64)
    h_hat = rms_norm(h, norm_weight, eps)
    if model_precision:
        h_hat = round_bf16(h_hat)
    q, k, v = qkv_project(h_hat, w_qkv, n_q_heads, n_kv_heads, head_dim)
    if model_precision:
        q, k, v = round_bf16(q), round_bf16(k), round_bf16(v)
    return h, q, k, v
