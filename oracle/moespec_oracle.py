"""CPU oracle for the budgeted MoE verify layer.  TEST INFRASTRUCTURE, NOT PRODUCT.

Only tests, the smoke check and the benchmark's cpu_baseline / reference arm may
import this file.  It shares no code with the CUDA path and imports nothing from
it.  Everything is the paper's definition written out densely in fp64 with numpy
(a matrix product is the only library primitive); selection uses plain Python
sorting with an explicit (key descending, expert index ascending) order.  There
is no blocking, fusion or reordering beyond what the definitions state.

Inputs are fp64 arrays whose values are already rounded to the storage dtype of
the configuration (bf16 or fp32); the oracle reads those exact values.

Steps (notation of the paper: M tokens h_t, N experts, top-k, budget B):
  O1  router logits            z[t,i] = fp32( b_i + w_i . h_t )              Eq. 1 numerator, Algorithm 1 stage 1
  O2  routing probabilities    g_i(h_t) = softmax_i(z[t,:])                  Eq. 1
  O3  natural top-k T_k(h_t), union E(D), per-expert natural counts          Eq. 2, Eq. 3
  O4  router-based scores      s_i = sum_t g_i(h_t)                          Eq. 5, Algorithm 1 stage 2
  O5  shortlist S = B highest-scoring candidates                             Section 3.2, Algorithm 1 stage 3
  O6  per-token assignment A(t): substitution (Eq. 8) or truncation (Eq. 7)
  O7  mixing weights: substitution over the constrained selection, truncation
      over the original top-k; raw or renormalised per architecture          Section 2.1, Section 3.3
  O8  out_t = sum_{i in A(t)} wgt[t,i] * E_i(h_t), E_i a bias-free SwiGLU FFN Eq. 2 / 7 / 8
  O9  canonical per-expert gather order of routed (token, expert) pairs      Appendix C
  O10 static ranking: calibration counts c_i and the fixed ordering          Eq. 4
  O11 residual stack: x_{l+1} = storage(x_l + layer_l(x_l)), budget B_l per layer
      (Section 4: the budget is enforced at every MoE layer of the model)
  O12 oracle ranking: greedy minimisation of the reconstruction error        Eq. 6
  O13 reconstruction error ||O_S - O*||^2 / ||O*||^2                         Section 4.5

Readings of points the paper leaves open (tie-breaks, candidate set of the
shortlist, expert form, router bias) are listed in the repository's design
notes; each function states the one it takes.

Pins: every function here is pinned by tests that do not restate its formula
(brute force over subsets, invariants, closed forms, reductions to a plain
top-k MoE / a single SwiGLU FFN / a dense softmax mixture / a plain residual
SwiGLU stack, a hand-worked greedy example, the k = 1 closed form of Eq. 6, and
the identity between the objective of Eq. 6 and the error of the separately
pinned truncation layer of Eq. 7).  The one unpinned
item is statistical: the synthetic router's union sizes and coverage are only
reported beside the paper's Figure 2 / 4 / 7 numbers, which depend on trained
weights ("parity unpinned" for those statistics; no oracle output depends on
them).
"""
from __future__ import annotations

import numpy as np

SUBSTITUTION = 1   # Eq. 8
TRUNCATION = 2     # Eq. 7
FROM_ALL = 1       # Algorithm 1 literal: all N experts compete for the shortlist
FROM_UNION = 2     # only experts of the union E(D) compete (Section 3.1 framing)
STATIC = 3         # fixed ordering from calibration counts (Eq. 4, "Static Ranking")


# --------------------------------------------------------------------------- O1
def router_logits(H, Wr, bias=None):
    """z[t,i] = fp32(b_i + sum_j Wr[i,j] * H[t,j]), accumulated in fp64 (Eq. 1 numerator).

    The paper's router has no bias; `bias` exists because the synthetic
    workloads shape their routing tail with one.  None reproduces Eq. 1.
    The fp32 logits are the interface between the floating-point half and the
    integer (selection) half of the layer.
    """
    H = np.asarray(H, dtype=np.float64)
    Wr = np.asarray(Wr, dtype=np.float64)
    z = H @ Wr.T
    if bias is not None:
        z = z + np.asarray(bias, dtype=np.float64)[None, :]
    return z.astype(np.float32)


# --------------------------------------------------------------------------- O2
def softmax_rows(z):
    """g[t,i] = exp(z[t,i] - max_i z[t,:]) / sum_i exp(z[t,i] - max) in fp64 (Eq. 1)."""
    z = np.asarray(z, dtype=np.float64)
    M, N = z.shape
    p = np.empty((M, N), dtype=np.float64)
    for t in range(M):
        mx = z[t].max()
        e = np.exp(z[t] - mx)
        denom = 0.0
        for i in range(N):          # ascending expert index
            denom += e[i]
        p[t] = e / denom
    return p


# --------------------------------------------------------------------------- O3
def _ranked(keys, candidates):
    """Candidates ordered by (key descending, index ascending)."""
    return sorted(candidates, key=lambda i: (-keys[i], i))


def natural_topk(z, k):
    """T_k(h_t): the k experts with the largest logit, ties to the lower index.

    Ranking by the fp32 logit is ranking by g_i (softmax is monotone) without
    the rounding of exp.  Returns (list of per-token lists in rank order,
    sorted union E(D) (Eq. 3), natural per-expert counts).
    """
    z = np.asarray(z)
    M, N = z.shape
    kk = min(k, N)
    T = [_ranked(z[t], range(N))[:kk] for t in range(M)]
    natcnt = [0] * N
    for t in range(M):
        for i in T[t]:
            natcnt[i] += 1
    union = [i for i in range(N) if natcnt[i] > 0]
    return T, union, natcnt


# --------------------------------------------------------------------------- O4
def router_scores(p):
    """s_i = sum_{t=0..M-1} g_i(h_t), tokens added in ascending order in fp64 (Eq. 5)."""
    p = np.asarray(p, dtype=np.float64)
    M, N = p.shape
    s = np.zeros(N, dtype=np.float64)
    for t in range(M):
        s = s + p[t]
    return s


# --------------------------------------------------------------------------- O5
def shortlist(s, B, candidates):
    """S = the min(B, |candidates|) candidates with the highest score, ties to the lower index.

    Returned in rank order (best first).  `candidates` is range(N) under the
    literal reading of Algorithm 1 and the union E(D) under the union reading.
    """
    cand = list(candidates)
    return _ranked(s, cand)[:max(0, min(B, len(cand)))]


def static_counts(z_calib, k):
    """c_i = number of calibration tokens whose natural top-k contains expert i (Eq. 4)."""
    T, _, natcnt = natural_topk(z_calib, k)
    return natcnt


def static_ranking(counts):
    """Experts ordered by (selection count descending, index ascending): the fixed ordering of Eq. 4."""
    return _ranked(counts, range(len(counts)))


# --------------------------------------------------------------------------- O6
def assign(z, S, T, k, policy):
    """A(t): substitution = top-min(k,|S|) of S by logit (Eq. 8); truncation = T_k(t) /\\ S (Eq. 7).

    Lists are in rank order (by logit descending, index ascending).
    """
    z = np.asarray(z)
    M = z.shape[0]
    inS = set(S)
    A = []
    for t in range(M):
        if policy == SUBSTITUTION:
            A.append(_ranked(z[t], S)[:min(k, len(S))])
        elif policy == TRUNCATION:
            A.append([i for i in T[t] if i in inS])
        else:
            raise ValueError("policy")
    return A


# --------------------------------------------------------------------------- O7
def gate_weights(p, A, T, policy, renormalize):
    """Dense wgt[M,N] (zero where unassigned).

    Substitution: the full-softmax probabilities of the constrained selection,
    divided by their sum over A(t) when renormalising (Section 3.3).
    Truncation: probabilities "over the original top-k set (not re-computed)":
    the denominator, when renormalising, is the sum over T_k(t), so kept weights
    sum to at most 1 (Section 3.3).  Raw mode uses g_i unchanged (Section 2.1).
    """
    p = np.asarray(p, dtype=np.float64)
    M, N = p.shape
    W = np.zeros((M, N), dtype=np.float64)
    for t in range(M):
        base = A[t] if policy == SUBSTITUTION else T[t]
        denom = 1.0
        if renormalize:
            denom = 0.0
            for j in base:          # rank order
                denom += p[t, j]
        for i in A[t]:
            W[t, i] = p[t, i] / denom
    return W


# --------------------------------------------------------------------------- O8
def expert_ffn(X, W1, W3, W2):
    """E_i(x) = W2 (silu(W1 x) * (W3 x)), silu(a) = a / (1 + exp(-a)); no biases; fp64.

    X[M,d], W1[f,d] (gate), W3[f,d] (up), W2[d,f] (down) -> [M,d].
    """
    X = np.asarray(X, dtype=np.float64)
    a = X @ np.asarray(W1, dtype=np.float64).T
    u = X @ np.asarray(W3, dtype=np.float64).T
    m = (a / (1.0 + np.exp(-a))) * u
    return m @ np.asarray(W2, dtype=np.float64).T


def layer_output(H, Wt, w_gate, w_up, w_down, expert_rows=None):
    """out[t] = sum over experts i ascending of Wt[t,i] * E_i(h_t)  (Eq. 2 / 7 / 8 outer sum).

    Dense over tokens: every expert with any non-zero weight is evaluated on all
    M tokens and scaled by its weight column; experts whose column is all zero
    contribute exactly zero and are skipped.  A token with no kept expert gets
    an exact zero row (Section 3.3, truncation).
    `expert_rows[i]` gives the row of expert i inside w_gate/w_up/w_down when
    only a subset of experts was materialised (None = identity).
    """
    H = np.asarray(H, dtype=np.float64)
    M, d = H.shape
    N = Wt.shape[1]
    out = np.zeros((M, d), dtype=np.float64)
    for i in range(N):
        col = Wt[:, i]
        if not np.any(col != 0.0):
            continue
        r = i if expert_rows is None else expert_rows[i]
        y = expert_ffn(H, w_gate[r], w_up[r], w_down[r])
        out += col[:, None] * y
    return out


# --------------------------------------------------------------------------- O9
def canonical_permutation(A, N):
    """Gather order of routed (token, expert) pairs: expert id ascending, then token index ascending.

    Returns count[N], offset[N+1] (exclusive scan), active (experts with rows),
    perm_row2tok[R], and row_of[(t, i)] -> row.  (Appendix C: tokens routed to
    each expert are gathered and processed together.)
    """
    M = len(A)
    count = [0] * N
    for t in range(M):
        for i in A[t]:
            count[i] += 1
    offset = [0] * (N + 1)
    for i in range(N):
        offset[i + 1] = offset[i] + count[i]
    perm = []
    row_of = {}
    for i in range(N):
        for t in range(M):
            if i in A[t]:
                row_of[(t, i)] = len(perm)
                perm.append(t)
    active = [i for i in range(N) if count[i] > 0]
    return count, offset, active, perm, row_of


# ------------------------------------------------------------------ whole layer
def route(z, k, B, policy, shortlist_mode, renormalize, static_rank=None):
    """Steps O2..O7 and O9 from fp32 logits.  Returns a dict of every stage.

    With shortlist_mode STATIC the shortlist is the first B experts of `static_rank`
    (Section 3.2, "Static Ranking": the B experts with the highest calibration count);
    the router-based scores are still reported but do not choose S."""
    z = np.asarray(z, dtype=np.float32)
    M, N = z.shape
    p = softmax_rows(z)
    T, union, natcnt = natural_topk(z, k)
    s = router_scores(p)
    if shortlist_mode == STATIC:
        S = list(static_rank)[:max(0, min(B, len(static_rank)))]
    else:
        cand = range(N) if shortlist_mode == FROM_ALL else union
        S = shortlist(s, min(B, N), cand)
    A = assign(z, S, T, k, policy)
    Wt = gate_weights(p, A, T, policy, renormalize)
    count, offset, active, perm, row_of = canonical_permutation(A, N)
    coverage = float(sum(s[i] for i in S) / M) if M else 0.0
    return {"logits": z, "prob": p, "topk": T, "union": union, "natcnt": natcnt, "score": s,
            "S": S, "assign": A, "wgt": Wt, "count": count, "offset": offset, "active": active,
            "perm_row2tok": perm, "row_of": row_of, "coverage": coverage}


def verify_layer(H, router_w, router_bias, w_gate, w_up, w_down, k, B, policy, shortlist_mode,
                 renormalize, logits=None, expert_rows=None, static_rank=None):
    """Algorithm 1 end to end.  `logits` (fp32 [M,N]) replaces step O1 when given."""
    z = router_logits(H, router_w, router_bias) if logits is None else np.asarray(logits, dtype=np.float32)
    r = route(z, k, B, policy, shortlist_mode, renormalize, static_rank)
    r["out"] = layer_output(H, r["wgt"], w_gate, w_up, w_down, expert_rows)
    return r


# ------------------------------------------------------------ storage rounding
def round_bf16(x):
    """Round fp64/fp32 values to the nearest bf16 (ties to even), returned as fp64."""
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    out = (r & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32)
    return out.astype(np.float64).reshape(np.shape(x))


def round_storage(x, dtype):
    """Round to the storage dtype ("bf16", "fp16" or "fp32") and return fp64."""
    if dtype == "bf16":
        return round_bf16(x)
    if dtype == "fp16":
        return np.asarray(x, dtype=np.float64).astype(np.float16).astype(np.float64)
    return np.asarray(x, dtype=np.float32).astype(np.float64)


# -------------------------------------------------------------------------- O11
def verify_stack(H, layers, k, budgets, policy, shortlist_mode, renormalize, storage, static_ranks=None):
    """L budgeted MoE layers on a residual stream: x_0 = H, x_{l+1} = storage(x_l + out_l(x_l)).

    The budget is enforced at each MoE layer (abstract); the Limitations section
    names a per-layer budget as an extension, so `budgets` is one B per layer.  Only the MoE blocks
    are on this path: attention and normalisation between them are not part of
    the method.  `layers[l]` is a dict with router_w, router_bias, w_gate, w_up,
    w_down.  The stream is rounded to the storage dtype after every layer, as a
    model that keeps activations in that dtype does.  Returns the list
    [x_0, ..., x_L] and the per-layer routing dicts.
    """
    xs = [np.asarray(H, dtype=np.float64)]
    routes = []
    for l, Lw in enumerate(layers):
        r = verify_layer(xs[-1], Lw["router_w"], Lw["router_bias"], Lw["w_gate"], Lw["w_up"], Lw["w_down"], k,
                         budgets[l], policy, shortlist_mode, renormalize,
                         static_rank=None if static_ranks is None else static_ranks[l])
        xs.append(round_storage(xs[-1] + r["out"], storage))
        routes.append(r)
    return xs, routes


# -------------------------------------------------------------------------- O12
def expert_contributions(H, z, k, renormalize, w_gate, w_up, w_down):
    """C[t][i] = g_i(h_t) * E_i(h_t) for i in T_k(h_t): the terms of the gold output O* (Eq. 2, Eq. 6).

    g is the mixing weight of the unpruned model: the softmax probability, divided
    by the sum over T_k(h_t) when the architecture renormalises (Section 2.1).
    Returns (T, C) with C a list of dicts expert -> fp64 vector [d].
    """
    H = np.asarray(H, dtype=np.float64)
    z = np.asarray(z, dtype=np.float32)
    M, N = z.shape
    p = softmax_rows(z)
    T, _, _ = natural_topk(z, k)
    W = gate_weights(p, T, T, TRUNCATION, renormalize)
    C = [dict() for _ in range(M)]
    for i in range(N):
        toks = [t for t in range(M) if i in T[t]]
        if not toks:
            continue
        y = expert_ffn(H[toks], w_gate[i], w_up[i], w_down[i])
        for row, t in enumerate(toks):
            C[t][i] = W[t, i] * y[row]
    return T, C


def gold_output(T, C, d):
    """O*_t = sum_{i in T_k(h_t)} g_i(h_t) E_i(h_t), experts added in ascending index (Eq. 6, first line)."""
    out = np.zeros((len(T), d), dtype=np.float64)
    for t in range(len(T)):
        for i in sorted(T[t]):
            out[t] += C[t][i]
    return out


def subset_error(T, C, O_star, S):
    """sum_t || O*_t - sum_{j in S and in T_k(h_t)} g_j(h_t) E_j(h_t) ||^2: the objective of Eq. 6 for the set S.

    Reading: the inner sum runs over the experts of S that the token actually
    routes to; an expert outside T_k(h_t) has no term in O*_t and contributes
    nothing for that token (the truncation output with the original weights).
    """
    inS = set(S)
    err = 0.0
    for t in range(len(T)):
        approx = np.zeros_like(O_star[t])
        for j in sorted(T[t]):
            if j in inS:
                approx += C[t][j]
        diff = O_star[t] - approx
        err += float(diff @ diff)
    return err


def oracle_ranking(T, C, N, d, B):
    """Greedy ordering of Eq. 6: starting from the empty set, B times add the expert outside S
    whose addition leaves the smallest objective (ties -> lower expert index).

    Every candidate's objective is evaluated from its definition (no incremental
    update).  Returns (order, errors) with errors[b] the objective after b+1 picks.
    """
    O_star = gold_output(T, C, d)
    S, errs = [], []
    for _ in range(min(B, N)):
        best, best_err = -1, None
        for i in range(N):
            if i in S:
                continue
            e = subset_error(T, C, O_star, S + [i])
            if best_err is None or e < best_err:       # strict: the first (lowest) index keeps a tie
                best, best_err = i, e
        S.append(best)
        errs.append(best_err)
    return S, errs


# -------------------------------------------------------------------------- O13
def reconstruction_error(O_S, O_star):
    """||O_S - O*||_F^2 / ||O*||_F^2 over all tokens of the tree (Section 4.5)."""
    O_S = np.asarray(O_S, dtype=np.float64)
    O_star = np.asarray(O_star, dtype=np.float64)
    den = float(np.sum(O_star * O_star))
    num = float(np.sum((O_S - O_star) ** 2))
    return num / den if den > 0.0 else (0.0 if num == 0.0 else float("inf"))
