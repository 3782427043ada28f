"""An independent brute-force checker used only to pin the oracle.

It lays the cache entries and the step block out as ONE token sequence with a
type per token, materialises the full boolean visibility matrix from the
paper's prose rules (Sec. 2.1.1 and Sec. 2.3), and runs naive softmax attention
with numpy.  It is written differently from the oracle on purpose (whole-matrix
operations on a concatenated sequence instead of a per-pair predicate)."""
import numpy as np
import torch


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().double().numpy()


def visibility_matrix(L: int, n_c: int, d: int, anchors=None, hidden_cache=None) -> np.ndarray:
    """[n_q x (L + n_q)] boolean matrix.

    Token sequence: L cache tokens (prompt / memory / output / accepted regular
    tokens: type 'C'), then n_c regular candidates (type 'R'), then d foresight
    tokens (type 'F').  Rules:
      1. start from the plain causal matrix over the whole sequence;
      2. a foresight token's column is hidden from every other token;
      3. a foresight token that follows only the first a candidates does not see
         candidates a, a+1, ...;
      4. cache entries listed in hidden_cache (an evicted verbose step) are hidden.
    """
    n_q = n_c + d
    N = L + n_q
    types = np.array(["C"] * L + ["R"] * n_c + ["F"] * d)
    full = np.tril(np.ones((N, N), dtype=bool))                     # rule 1
    is_f = types == "F"
    full[:, is_f] = False                                           # rule 2 ...
    full[np.arange(N), np.arange(N)] = True                         # ... except itself
    if anchors is not None:                                         # rule 3
        for k in range(d):
            row = L + n_c + k
            full[row, L + anchors[k]: L + n_c] = False
    if hidden_cache is not None:                                    # rule 4
        full[:, np.asarray(hidden_cache, dtype=np.int64)] = False
    return full[L:, :]


def dense_attention(q, k_all, v_all, vis, scale):
    """q [n_q][D], k_all/v_all [N][D] (fp64), vis [n_q][N] bool -> (out, lse)."""
    s = scale * (q @ k_all.T)
    s = np.where(vis, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    p = np.exp(s - m)
    den = p.sum(axis=1, keepdims=True)
    return (p @ v_all) / den, (m + np.log(den))[:, 0]
