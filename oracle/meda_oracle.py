"""Plain fp64 CPU oracle for the MEDA prefill KV-compression pass (arXiv 2502.17599).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import, call or link this
module: it exists so that the CUDA kernels have something independent to be compared
with.  It shares no code, table or helper with the CUDA path and never imports it.

Everything is NumPy in float64.  Each function follows one passage of the paper, in the
paper's order and notation, with no blocking, fusion or reordering beyond what the
equation states; `@` (a library matmul) is the only library primitive used as a step.
Inputs are the dtype-rounded values the GPU sees (bf16 / fp32 values widened exactly).

Where the paper is silent or ambiguous the reading taken is stated at the function.

Pinning status (see tests/test_oracle_pins.py): every function below is pinned to closed
forms, invariants, textbook special cases or brute force written with Python loops /
exact rationals.  The *choice* of integer rounding in `allocate_budgets` (bounded
proportional quota + largest remainder) and of the observation-window restriction of
Eq. 8 are readings, not statements of the paper; the paper prints no worked numeric
example of any step, so no value is pinned to a printed number.
"""
from __future__ import annotations

import numpy as np

TEXT = 0
VISUAL = 1

COS_EPS = 1e-8  # lower clamp on a key norm in the cosine similarity (Eq. 11 is silent on zero norms)


class BudgetInfeasible(ValueError):
    """The global budget cannot be met with every layer inside [min_budget, n_tokens]."""


# --------------------------------------------------------------------------------------
# Step 1: attention of the observation-window queries against the key cache
# --------------------------------------------------------------------------------------

def default_query_positions(n_tokens: int, window: int) -> np.ndarray:
    """Absolute positions of the observation window: the last `window` prompt tokens."""
    return np.arange(n_tokens - window, n_tokens, dtype=np.int64)


def head_logits(q_h: np.ndarray, k_g: np.ndarray, q_pos: np.ndarray) -> np.ndarray:
    """Scaled dot-product logits of one query head against its KV head (Eq. 4 / Eq. 8 argument).

    s[i, j] = q_i . k_j / sqrt(d) with d the head dimension (the paper writes sqrt(D) and calls
    D "the dimensionality of the embeddings"; read per head).  Decoder prefill attention is
    causal: query row i at absolute position q_pos[i] sees keys j <= q_pos[i]; the others get
    -inf.  q_h [w, d], k_g [n, d] -> [w, n].
    """
    d = q_h.shape[1]
    s = (q_h @ k_g.T) / np.sqrt(float(d))
    n = k_g.shape[0]
    hidden = np.arange(n)[None, :] > np.asarray(q_pos)[:, None]
    s[hidden] = -np.inf
    return s


def masked_softmax(s: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    """Row softmax over the key subset `allowed` (bool [n]) intersected with the visible keys.

    Keys outside the subset get probability 0.  A row with no visible key in the subset is
    returned as all zeros (it is not a distribution; callers skip such rows).
    """
    t = np.where(allowed[None, :], s, -np.inf)
    m = np.max(t, axis=1, keepdims=True)
    dead = ~np.isfinite(m)
    m = np.where(dead, 0.0, m)
    e = np.exp(t - m)
    z = np.sum(e, axis=1, keepdims=True)
    z = np.where(dead, 1.0, z)
    return e / z


def window_scores(q_win: np.ndarray, k: np.ndarray, q_pos: np.ndarray | None = None) -> np.ndarray:
    """Accumulated attention score per key and KV head (Eq. 8, rows restricted to the window).

    A_p = softmax(Q_p K_p^T / sqrt(d)) with the causal mask (Eq. 8 writes Attn(.); these are the
    attention weights of prompt encoding).  A_s[g, j] = sum over the query rows i and over the
    query heads h of KV group g of A_p[h, i, j].  With the window equal to the whole prompt
    this is Eq. 8 literally.  q_win [Hq, w, d], k [Hkv, n, d] -> [Hkv, n].
    """
    hq, w, _ = q_win.shape
    hkv, n, _ = k.shape
    group = hq // hkv
    if q_pos is None:
        q_pos = default_query_positions(n, w)
    everything = np.ones(n, dtype=bool)
    a_s = np.zeros((hkv, n))
    for h in range(hq):
        g = h // group
        p = masked_softmax(head_logits(q_win[h], k[g], q_pos), everything)
        a_s[g] += p.sum(axis=0)
    return a_s


def row_stats(q_win: np.ndarray, k: np.ndarray, modality: np.ndarray, q_pos: np.ndarray | None = None) -> np.ndarray:
    """Softmax normalisers of every window row: [Hq, w, 4] = (max, sum-exp) over all visible
    keys and (max, sum-exp) over the visible visual keys.  A row with no visible visual key has
    (-inf, 0) in the last two.  (Not in the paper: it is the intermediate the library exposes.)
    """
    hq, w, _ = q_win.shape
    hkv, n, _ = k.shape
    group = hq // hkv
    if q_pos is None:
        q_pos = default_query_positions(n, w)
    vis = np.asarray(modality) == VISUAL
    out = np.zeros((hq, w, 4))
    for h in range(hq):
        s = head_logits(q_win[h], k[h // group], q_pos)
        m = s.max(axis=1)
        out[h, :, 0] = m
        out[h, :, 1] = np.exp(s - m[:, None]).sum(axis=1)
        sv = np.where(vis[None, :], s, -np.inf)
        mv = sv.max(axis=1)
        ok = np.isfinite(mv)
        out[h, :, 2] = mv
        out[h, ok, 3] = np.exp(sv[ok] - mv[ok, None]).sum(axis=1)
    return out


# --------------------------------------------------------------------------------------
# Step 1 (cont.): cross-modal attention entropy, Eq. 4-6
# --------------------------------------------------------------------------------------

def _xlogx_sum(a: np.ndarray) -> np.ndarray:
    """sum_j a_ij log a_ij per row with 0 log 0 = 0 (natural log: it pairs with exp in Eq. 7)."""
    safe = np.where(a > 0.0, a, 1.0)
    return np.sum(a * np.log(safe), axis=1)


def directed_entropy_term(q: np.ndarray, k: np.ndarray, q_pos: np.ndarray, key_subset: np.ndarray,
                          entropy_mode: int = 0) -> float:
    """One line of Eq. 5: (1/rows) sum_i sum_j A[i, j] log A[i, j]  (a non-positive number).

    A is Eq. 4's cross-modal attention: the softmax is taken over the keys of the *other*
    modality only (`key_subset`), so every row is a distribution.  entropy_mode 0 (Sec. 3.2
    defines A as the per-head attention averaged over the heads): A = mean over the query heads of
    the per-head softmax, then the row entropies.  entropy_mode 1: the mean over heads of the
    per-head sums.  Rows with no visible key in the subset are skipped, and 1/rows counts the
    rows used; no usable row gives 0.
    """
    hq, w, _ = q.shape
    hkv = k.shape[0]
    group = hq // hkv
    n = k.shape[1]
    usable = np.array([np.any(key_subset[: int(p) + 1]) for p in q_pos])
    if not usable.any():
        return 0.0
    if entropy_mode == 0:
        a_mean = np.zeros((w, n))
        for h in range(hq):
            a_mean += masked_softmax(head_logits(q[h], k[h // group], q_pos), key_subset)
        a_mean /= hq
        per_row = _xlogx_sum(a_mean)
    else:
        per_row = np.zeros(w)
        for h in range(hq):
            per_row += _xlogx_sum(masked_softmax(head_logits(q[h], k[h // group], q_pos), key_subset))
        per_row /= hq
    return float(per_row[usable].sum() / usable.sum())


def cross_modal_entropy(q_win: np.ndarray, k: np.ndarray, modality: np.ndarray,
                        q_pos: np.ndarray | None = None,
                        q_vis: np.ndarray | None = None, q_vis_pos: np.ndarray | None = None,
                        entropy_mode: int = 0) -> float:
    """E_CM = -(E_TV + E_VT), Eq. 6.

    E_TV uses the text query rows `q_win` against the visual keys; E_VT uses the visual query
    rows `q_vis` (optional) against the text keys (Eq. 5 prints E_TV's index ranges twice; read
    as rows = visual queries, columns = text keys).  Without visual query rows the E_VT term is
    absent and E_CM = -E_TV, the mean row entropy of text-to-vision attention.
    """
    n = k.shape[1]
    if q_pos is None:
        q_pos = default_query_positions(n, q_win.shape[1])
    modality = np.asarray(modality)
    e_tv = directed_entropy_term(q_win, k, q_pos, modality == VISUAL, entropy_mode)
    e_vt = 0.0
    if q_vis is not None:
        e_vt = directed_entropy_term(q_vis, k, np.asarray(q_vis_pos), modality == TEXT, entropy_mode)
    return -(e_tv + e_vt)


# --------------------------------------------------------------------------------------
# Step 2: per-layer budgets, Eq. 7 (and the appendix derivation of alpha_l)
# --------------------------------------------------------------------------------------

def allocation_weights(entropy: np.ndarray, alloc_mode: int = 0) -> np.ndarray:
    """softmax over layers of E_CM (Eq. 7 without the L*rho factor).  Sec. 3.2's name for the rule
    suggests an inversion of the entropy, but Eq. 7 and App. A.3 are a direct softmax: higher
    entropy, larger share; the equations are followed.  alloc_mode 1 = Table 5's ablation row without dynamic allocation: uniform."""
    e = np.asarray(entropy, dtype=np.float64)
    if alloc_mode == 1:
        return np.full(e.shape, 1.0 / e.size)
    x = np.exp(e - e.max())
    return x / x.sum()


def bounded_quotas(weights: np.ndarray, total: int, lo: int, hi: int) -> tuple[np.ndarray, np.ndarray]:
    """Real-valued per-layer quotas q_l = clip(lambda * W_l, lo, hi) with lambda chosen so that
    sum_l q_l = total.  Unbounded this is Eq. 7: S_l = W_l * L * rho * n = W_l * total.

    The paper is silent on S_l > n or S_l ~ 0, both of which the softmax of raw nats produces.
    f(lambda) = sum_l clip(lambda W_l, lo, hi) is continuous and non-decreasing, so the solution
    is found by walking its breakpoints.  Returns (quotas, state) with state -1 / 0 / +1 for a
    layer clamped at lo / free / clamped at hi.  The free quotas are evaluated as
    (total - clamped) * W_l / sum_free W in ascending layer order.
    """
    w = np.asarray(weights, dtype=np.float64)
    n_l = w.size
    if total < n_l * lo or total > n_l * hi:
        raise BudgetInfeasible(f"budget {total} outside [{n_l * lo}, {n_l * hi}]")

    def f(lam: float) -> float:
        return float(np.clip(lam * w, lo, hi).sum())

    pos = w > 0
    cuts = sorted(set([0.0] + list(lo / w[pos]) + list(hi / w[pos])))
    # find the first breakpoint interval [a, b] with f(a) <= total <= f(b)
    lam = cuts[-1]
    for a, b in zip(cuts[:-1], cuts[1:]):
        if f(a) <= total <= f(b):
            lam = 0.5 * (a + b)  # any interior point identifies the clamp pattern
            if f(a) == total:
                lam = a
            elif f(b) == total:
                lam = b
            break
    raw = lam * w
    state = np.zeros(n_l, dtype=np.int64)
    state[raw <= lo] = -1
    state[raw >= hi] = +1
    if lo == hi:
        state[:] = -1
    free = state == 0
    clamped_total = int((state == -1).sum()) * lo + int((state == 1).sum()) * hi
    q = np.where(state == -1, float(lo), float(hi))
    if free.any():
        w_free = 0.0
        for l in range(n_l):  # ascending layer order
            if free[l]:
                w_free += w[l]
        q = q.copy()
        for l in range(n_l):
            if free[l]:
                q[l] = (total - clamped_total) * w[l] / w_free
    return q, state


def allocate_budgets(entropy: np.ndarray, global_budget: int, n_tokens: int, min_budget: int,
                     beta_recent: int = 3, beta_important: int = 1, alloc_mode: int = 0) -> np.ndarray:
    """Integer budgets [L, 3] = (S_l, M_l, N_l) with sum_l S_l = global_budget.

    Eq. 7 gives the real-valued share; integers follow by largest remainder: S_l = floor(q_l),
    and the units still missing go one each to the free (unclamped) layers in order of largest
    fractional part, ties to the lowest layer.  S_l is then split recent : important =
    beta_recent : beta_important (3:1 in the paper's implementation details):
    M_l = floor(S_l * beta_recent / (beta_recent + beta_important)), N_l = S_l - M_l.
    """
    w = allocation_weights(entropy, alloc_mode)
    q, state = bounded_quotas(w, int(global_budget), int(min_budget), int(n_tokens))
    s = np.floor(q).astype(np.int64)
    missing = int(global_budget) - int(s.sum())
    frac = q - np.floor(q)
    free = [l for l in range(len(s)) if state[l] == 0]
    order = sorted(free, key=lambda l: (-frac[l], l))
    assert 0 <= missing <= len(order) or not order, (missing, len(order))
    for l in order[:max(missing, 0)]:
        s[l] += 1
    m = (s * beta_recent) // (beta_recent + beta_important)
    out = np.stack([s, m, s - m], axis=1)
    return out


# --------------------------------------------------------------------------------------
# Step 3: selection, Eq. 9-10
# --------------------------------------------------------------------------------------

def select_topk(a_s: np.ndarray, modality: np.ndarray, n_recent: int, n_important: int) -> tuple[np.ndarray, np.ndarray]:
    """Conserved and less-important index sets of one (layer, KV head).

    Eq. 10: the last M = n_recent tokens are kept; among the others (A_s[:-M]) the top N =
    n_important are kept.  Eq. 9 first adds max(A_s) to the text tokens' scores, which puts
    every text token ahead of every visual one; here that is the lexicographic order
    (is_text descending, A_s descending), identical to Eq. 9 in exact arithmetic except that a
    text score of exactly 0 still beats the visual maximum.  Ties go to the lowest index.
    Both outputs are in ascending original index.
    """
    a_s = np.asarray(a_s, dtype=np.float64)
    n = a_s.size
    n_cand = n - n_recent
    if n_important > n_cand or n_recent > n or n_important < 0:
        raise ValueError("selection sizes do not fit the sequence")
    is_text = (np.asarray(modality)[:n_cand] == TEXT)
    cand = list(range(n_cand))
    cand.sort(key=lambda j: (0 if is_text[j] else 1, -a_s[j], j))
    keep = np.zeros(n, dtype=bool)
    keep[np.array(cand[:n_important], dtype=np.int64)] = True
    keep[n_cand:] = True
    conserved = np.nonzero(keep)[0]
    less = np.nonzero(~keep)[0]
    return conserved, less


# --------------------------------------------------------------------------------------
# Step 4: merging, Eq. 11-12
# --------------------------------------------------------------------------------------

def cosine_similarity(k_less: np.ndarray, k_c: np.ndarray) -> np.ndarray:
    """U[i, j] = k_i . k_j / (|k_i| |k_j|), Eq. 11; each norm is clamped below at COS_EPS so a
    zero key gives similarity 0 to everything."""
    ni = np.maximum(np.sqrt((k_less * k_less).sum(axis=1)), COS_EPS)
    nj = np.maximum(np.sqrt((k_c * k_c).sum(axis=1)), COS_EPS)
    return (k_less @ k_c.T) / (ni[:, None] * nj[None, :])


def nearest_conserved(k_g: np.ndarray, conserved: np.ndarray, less: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Many-to-one matching: for each less-important key the slot (position inside `conserved`)
    of its most similar conserved key; the first maximum in ascending slot order wins.
    Returns (target slot [L_less], U [L_less, L_c])."""
    u = cosine_similarity(k_g[less], k_g[conserved])
    if u.shape[0] == 0:
        return np.zeros(0, dtype=np.int64), u
    return np.argmax(u, axis=1).astype(np.int64), u


def average_merge(x_g: np.ndarray, conserved: np.ndarray, less: np.ndarray, target: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Eq. 12 for one tensor (keys or values) of one head: x_j <- (x_j + sum_{i in N_j} x_i) /
    (|N_j| + 1), all sums over the original rows (simultaneous, not sequential).
    Returns (merged [L_c, d] in fp64, counts |N_j| + 1)."""
    out = x_g[conserved].copy()
    counts = np.ones(conserved.size, dtype=np.int64)
    for p in range(less.size):  # ascending original index
        out[target[p]] += x_g[less[p]]
        counts[target[p]] += 1
    return out / counts[:, None], counts


def merge_kv(k_g: np.ndarray, v_g: np.ndarray, conserved: np.ndarray, less: np.ndarray,
             target: np.ndarray | None = None, merge_mode: int = 0):
    """Merge step for one (layer, KV head).  The similarity uses keys only and the same
    assignment is applied to the values.  merge_mode 1 = Table 5's ablation row without average merging:
    the less-important pairs are dropped.  Returns (K_c', V_c', counts, target)."""
    if merge_mode == 1:
        return (k_g[conserved].copy(), v_g[conserved].copy(),
                np.ones(conserved.size, dtype=np.int64), np.zeros(0, dtype=np.int64))
    if target is None:
        target, _ = nearest_conserved(k_g, conserved, less)
    k_m, counts = average_merge(k_g, conserved, less, target)
    v_m, _ = average_merge(v_g, conserved, less, target)
    return k_m, v_m, counts, target


# --------------------------------------------------------------------------------------
# Output rounding and the whole pass
# --------------------------------------------------------------------------------------

def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64 to the nearest bfloat16 value (8 significant bits, ties to even), returned as
    fp64.  Done directly from fp64 so there is no double rounding.  Subnormal bf16 outputs are
    not modelled (values below 2**-126 are flushed with the same grid as the smallest normal)."""
    x = np.asarray(x, dtype=np.float64)
    out = np.zeros_like(x)
    nz = (x != 0) & np.isfinite(x)
    _, e = np.frexp(x[nz])            # x = m * 2**e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)
    scaled = np.ldexp(x[nz], 8 - e)   # 128 <= |scaled| < 256
    out[nz] = np.ldexp(np.rint(scaled), e - 8)
    out[~np.isfinite(x)] = x[~np.isfinite(x)]
    return out


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    raise ValueError(dtype)


def compress_layer(k: np.ndarray, v: np.ndarray, a_s: np.ndarray, modality: np.ndarray,
                   n_recent: int, n_important: int, dtype: str, merge_mode: int = 0):
    """Selection + merging of every KV head of one layer.  k, v [Hkv, n, d]; a_s [Hkv, n].
    Returns a list over heads of dicts (conserved, less, target, k, v, counts)."""
    res = []
    for g in range(k.shape[0]):
        conserved, less = select_topk(a_s[g], modality, n_recent, n_important)
        k_m, v_m, counts, target = merge_kv(k[g], v[g], conserved, less, merge_mode=merge_mode)
        res.append(dict(conserved=conserved, less=less, target=target,
                        k=round_to_dtype(k_m, dtype), v=round_to_dtype(v_m, dtype), counts=counts))
    return res


def compress_pass(layers, modality: np.ndarray, global_budget: int, min_budget: int, dtype: str,
                  beta_recent: int = 3, beta_important: int = 1, entropy_mode: int = 0,
                  alloc_mode: int = 0, merge_mode: int = 0):
    """The whole pass.  `layers` is a sequence of (q_win, k, v) per layer.  Phase A (scores and
    entropy of every layer), then Eq. 7's allocation (which needs every layer's entropy), then
    phase B (selection and merging per layer)."""
    n = layers[0][1].shape[1]
    scores = [window_scores(q, k) for q, k, _ in layers]
    entropy = np.array([cross_modal_entropy(q, k, modality, entropy_mode=entropy_mode) for q, k, _ in layers])
    budgets = allocate_budgets(entropy, global_budget, n, min_budget, beta_recent, beta_important, alloc_mode)
    out = []
    for l, (_, k, v) in enumerate(layers):
        out.append(compress_layer(k, v, scores[l], modality, int(budgets[l, 1]), int(budgets[l, 2]), dtype, merge_mode))
    return dict(scores=scores, entropy=entropy, budgets=budgets, layers=out)


# --------------------------------------------------------------------------------------
# After the pass: one decoding step over a (compressed) cache, Eq. 3
# --------------------------------------------------------------------------------------

def decode_attention(q: np.ndarray, k_c: np.ndarray, v_c: np.ndarray) -> np.ndarray:
    """Attention of one new token's queries over a per-layer cache (Eq. 3): for every query head h of
    KV group g, out[h] = softmax(q_h K_g^T / sqrt(d)) V_g over all rows of the cache (the new token
    comes after every cached one, so nothing is masked).  The cache may be the full one or the
    compressed (K_c, V_c) of Eq. 10 / Eq. 12; merged rows are used as they are, with no weighting by
    how many pairs they absorbed (Eq. 3 has none).  q [Hq, d], k_c, v_c [Hkv, S, d] -> [Hq, d]."""
    hq, d = q.shape
    hkv = k_c.shape[0]
    group = hq // hkv
    out = np.zeros((hq, d))
    for h in range(hq):
        g = h // group
        s = (k_c[g] @ q[h]) / np.sqrt(float(d))
        p = np.exp(s - s.max())
        p /= p.sum()
        out[h] = p @ v_c[g]
    return out


# --------------------------------------------------------------------------------------
# Off the hot path: the appendix's KV-cache memory formula (context for Table 6)
# --------------------------------------------------------------------------------------

def kv_cache_gib(n_tokens: float, n_layers: int = 32, n_heads: int = 32, head_dim: int = 128, bytes_per_value: int = 2) -> float:
    """App. A.2: tokens x (bytes per value) x heads x layers x (head_dim x 2 for K and V) / 1024^3."""
    return n_tokens * bytes_per_value * n_heads * n_layers * (head_dim * 2) / 1024.0 ** 3
