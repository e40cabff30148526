"""Float64 CPU oracle for one causal linear-attention layer with the causal
depthwise-convolution augmentation.  TEST INFRASTRUCTURE ONLY: it is slow on
purpose, shares no code with the CUDA path, and must never be imported by the
library itself (only by tests, the smoke check and the benchmark's CPU
baseline).

What it computes (notation of the paper, Sec. 3 "Linear Attentions" and
Sec. 4.1/4.2):

* Kernelised attention Sim(Q, K) ~ phi(Q) phi(K)^T reordered as
  phi(Q) (phi(K)^T V)  (Sec. 3).  In the causal case query t meets the
  cumulative sum  sum_{i<=t} K_i V_i  (Sec. 4.1, the "cumsum" sentence), i.e.

      a_ij  = phi(q_i) . phi(k_j)                       j <= i
      la_i  = sum_{j<=i} a_ij v_j / (sum_{j<=i} a_ij + eps)

  The paper writes only the numerator; the division by the summed weights is
  the usual normaliser of kernel attention and is part of this layer's
  definition here (reading 1 below).
* The masked depthwise convolution on the V branch (Sec. 4.1 "Revised LA
  Augmentation"): every channel c of head h is filtered along time with taps
  that only look backwards,  conv_i[c] = sum_{t<W} w[h,c,t] v_{i-t}[c],  and
  the result is added to the attention output:  o_i = la_i + conv_i.
* Grouped processing (Sec. 4.1): the sequence is cut into non-overlapping
  groups, groups are processed in parallel inside, and only the group-level
  cumulative sums of phi(K)^T V are carried between groups ("chunked" below).
* The three-branch block of Sec. 4.1 (`prefill_grouped_block`): between groups only the group-level sums
  (no linear-attention term inside a group), inside a group causal softmax attention, plus the
  convolution; alpha weighs the global term.
* Speculative verification (Sec. 4.2 "Proposed Solution" and Sec. 5.3
  "Comparison with Direct Integration"): every node of a draft-token tree sees
  the committed prefix (one shared state) plus its own ancestors, and the
  convolution is unfolded along that ancestor chain so a node never convolves
  over a sibling.

Readings taken where the paper is silent:
  1. normaliser as above, eps added to the denominator;
  2. phi is applied to q and k alike; "elu1": phi(x) = x + 1 for x > 0 and
     exp(x) otherwise; "relu": phi(x) = max(x, 0);
  3. the convolution acts on the raw v, is added after the division, has no
     bias, and sees zeros before the start of a fresh sequence;
  4. W counts live causal taps (current token and W-1 past ones);
  5. decode updates the state with the new token first and reads it afterwards
     (the cumulative sum is inclusive);
  6. a tree is a parent array in topological order (parent[n] < n, -1 for a
     child of the committed prefix); a node sees its ancestors and itself.

Pins (see tests/test_oracle_*.py): hand-derived rational values and geometric
series closed forms (tests/golden/), scalar brute force on tiny inputs,
cumulative-mean and convex-hull special cases, a library causal depthwise
conv1d, agreement of the quadratic / recurrent / chunked forms, causality under
perturbation, tree verification against sequential decoding along every
root-to-node path, and commit against repeated decode steps.  The paper prints
no numeric worked example for this layer, so there is no pin to a value printed
by the paper itself.

State layout (per batch entry b and head h):
  S   [B, H, d, d]   S[a, c] = sum_j phi(k_j)[a] v_j[c]
  z   [B, H, d]      z[a]    = sum_j phi(k_j)[a]
  win [B, H, W-1, d] the last W-1 values of v, oldest first
  pos [B]            tokens absorbed so far
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


# ---------------------------------------------------------------------------
# Elementary pieces
# ---------------------------------------------------------------------------

def phi(x: np.ndarray, kind: str) -> np.ndarray:
    """Feature map of Sec. 3 (Sim(Q,K) ~ phi(Q) phi(K)^T), elementwise and non-negative."""
    x = np.asarray(x, dtype=np.float64)
    if kind == "elu1":
        return np.where(x > 0.0, x + 1.0, np.exp(np.minimum(x, 0.0)))
    if kind == "relu":
        return np.maximum(x, 0.0)
    raise ValueError(f"unknown feature map {kind!r}")


@dataclass
class State:
    S: np.ndarray
    z: np.ndarray
    win: np.ndarray
    pos: np.ndarray

    def copy(self) -> "State":
        return State(self.S.copy(), self.z.copy(), self.win.copy(), self.pos.copy())


def empty_state(B: int, H: int, d: int, W: int) -> State:
    return State(np.zeros((B, H, d, d)), np.zeros((B, H, d)), np.zeros((B, H, W - 1, d)),
                 np.zeros((B,), dtype=np.int64))


def _f64(*xs):
    return tuple(np.asarray(x, dtype=np.float64) for x in xs)


def causal_dwconv(v: np.ndarray, w: np.ndarray, win: np.ndarray) -> np.ndarray:
    """Masked depthwise convolution of Sec. 4.1: conv_i[c] = sum_t w[h,c,t] v_{i-t}[c].

    v [B,H,T,d]; w [H,d,W]; win [B,H,W-1,d] holds v_{-(W-1)} .. v_{-1}.
    Only the current and earlier tokens are touched, which is the causal mask on
    the kernel that stops the leakage described in Sec. 3 ("Limitations").
    """
    B, H, T, d = v.shape
    W = w.shape[2]
    hist = np.concatenate([win, v], axis=2)          # index s holds v_{s-(W-1)}
    out = np.zeros_like(v)
    for t in range(W):
        # v_{i-t} for i = 0..T-1 sits at hist[:, :, i - t + W - 1]
        out += w[None, :, :, t][:, :, None, :] * hist[:, :, W - 1 - t: W - 1 - t + T, :]
    return out


def _next_window(win: np.ndarray, v: np.ndarray) -> np.ndarray:
    W1 = win.shape[2]
    if W1 == 0:
        return win.copy()
    return np.concatenate([win, v], axis=2)[:, :, -W1:, :].copy()


# ---------------------------------------------------------------------------
# Form Q: the definition (quadratic in T)
# ---------------------------------------------------------------------------

def prefill_quadratic(q, k, v, w, kind: str, eps: float, state: State | None = None):
    """o_i = sum_{j<=i} a_ij v_j / (sum_{j<=i} a_ij + eps) + conv_i, straight from the definition.

    With a carried state the sums also run over the tokens already absorbed,
    whose contribution is phi(q_i)^T S and phi(q_i) . z.
    Returns (o [B,H,T,d], new State).
    """
    q, k, v, w = _f64(q, k, v, w)
    B, H, T, d = q.shape
    W = w.shape[2]
    st = empty_state(B, H, d, W) if state is None else state
    fq, fk = phi(q, kind), phi(k, kind)
    a = np.matmul(fq, np.swapaxes(fk, -1, -2))       # a[i, j] = phi(q_i) . phi(k_j)
    a = np.tril(a)                                   # keep j <= i
    num = np.matmul(a, v) + np.matmul(fq, st.S)
    den = a.sum(axis=-1) + np.einsum("bhia,bha->bhi", fq, st.z)
    o = num / (den + eps)[..., None] + causal_dwconv(v, w, st.win)
    new = State(st.S + np.matmul(np.swapaxes(fk, -1, -2), v), st.z + fk.sum(axis=2),
                _next_window(st.win, v), st.pos + T)
    return o, new


# ---------------------------------------------------------------------------
# Form R: the recurrence (what decoding does)
# ---------------------------------------------------------------------------

def decode_step(q, k, v, w, kind: str, eps: float, state: State):
    """One token per sequence: S += phi(k) v^T, z += phi(k), then read with phi(q).

    q, k, v [B,H,d].  Returns (o [B,H,d], new State).  Sec. 4.1: Q_t meets the
    cumulative sum up to and including t.
    """
    q, k, v, w = _f64(q, k, v, w)
    fq, fk = phi(q, kind), phi(k, kind)
    S = state.S + fk[..., :, None] * v[..., None, :]
    z = state.z + fk
    num = np.einsum("bha,bhac->bhc", fq, S)
    den = np.einsum("bha,bha->bh", fq, z)
    conv = causal_dwconv(v[:, :, None, :], w, state.win)[:, :, 0, :]
    o = num / (den + eps)[..., None] + conv
    return o, State(S, z, _next_window(state.win, v[:, :, None, :]), state.pos + 1)


def prefill_recurrent(q, k, v, w, kind: str, eps: float, state: State | None = None):
    q, k, v, w = _f64(q, k, v, w)
    B, H, T, d = q.shape
    st = empty_state(B, H, d, w.shape[2]) if state is None else state
    o = np.zeros_like(v)
    for i in range(T):
        o[:, :, i, :], st = decode_step(q[:, :, i], k[:, :, i], v[:, :, i], w, kind, eps, st)
    return o, st


# ---------------------------------------------------------------------------
# Form C: grouped / chunkwise (what prefill does)
# ---------------------------------------------------------------------------

def prefill_chunked(q, k, v, w, kind: str, eps: float, chunk: int, state: State | None = None):
    """Sec. 4.1 grouping: inside a group the masked product phi(Q)phi(K)^T V, between groups
    only the group-level cumulative sums S and z."""
    q, k, v, w = _f64(q, k, v, w)
    B, H, T, d = q.shape
    st = empty_state(B, H, d, w.shape[2]) if state is None else state
    S, z = st.S.copy(), st.z.copy()
    o = np.zeros_like(v)
    for lo in range(0, T, chunk):
        hi = min(lo + chunk, T)
        fq, fk, vc = phi(q[:, :, lo:hi], kind), phi(k[:, :, lo:hi], kind), v[:, :, lo:hi]
        a = np.tril(np.matmul(fq, np.swapaxes(fk, -1, -2)))
        num = np.matmul(fq, S) + np.matmul(a, vc)
        den = np.einsum("bhia,bha->bhi", fq, z) + a.sum(axis=-1)
        o[:, :, lo:hi] = num / (den + eps)[..., None]
        S = S + np.matmul(np.swapaxes(fk, -1, -2), vc)
        z = z + fk.sum(axis=2)
    o += causal_dwconv(v, w, st.win)
    return o, State(S, z, _next_window(st.win, v), st.pos + T)


# ---------------------------------------------------------------------------
# The three-branch block of Sec. 4.1: grouped linear attention between groups, softmax
# attention inside a group, masked depthwise convolution
# ---------------------------------------------------------------------------

def prefill_grouped_block(q, k, v, w, kind: str, eps: float, group: int, alpha: float, scale: float,
                          state: State | None = None):
    """The augmented block as Sec. 4.1 describes it (Fig. "la_aug", three branches), token by token.

    The sequence is cut into non-overlapping groups of `group` tokens, counted from the first token of the
    sequence.  For token i in group g:

      middle branch  glob_i = phi(q_i)^T S_{<g} / (phi(q_i) . z_{<g} + eps): linear attention against the
                     group-level cumulative sums of the groups before g only ("within each group we bypass local
                     dependencies"); defined as 0 where that denominator is 0 (no earlier group and eps = 0);
      left branch    loc_i = sum_{j in g, j <= i} softmax_j(scale q_i . k_j) v_j: causal softmax attention inside
                     the group, on the raw q and k;
      right branch   conv_i: the masked depthwise convolution of v;
      o_i = alpha * glob_i + loc_i + conv_i   (alpha balances the global against the local term).

    Readings where the paper is silent: the softmax scale is an argument (1/sqrt(d) is the usual choice), alpha
    multiplies the global branch only, groups are aligned to the start of the sequence.  With a carried `state` the
    tokens absorbed so far must end at a group boundary (state.pos a multiple of `group`); the returned state holds
    S, z over all tokens, the convolution window and pos, as the other forms do.
    Returns (o [B,H,T,d], new State).
    """
    q, k, v, w = _f64(q, k, v, w)
    B, H, T, d = q.shape
    W = w.shape[2]
    st = empty_state(B, H, d, W) if state is None else state
    if np.any(st.pos % group != 0):
        raise ValueError("the carried state does not end at a group boundary")
    fq, fk = phi(q, kind), phi(k, kind)
    S, z = st.S.copy(), st.z.copy()
    o = np.zeros_like(v)
    for lo in range(0, T, group):
        hi = min(lo + group, T)
        for i in range(lo, hi):
            # middle branch: the groups before this one
            num = np.einsum("bha,bhac->bhc", fq[:, :, i], S)
            den = np.einsum("bha,bha->bh", fq[:, :, i], z) + eps
            glob = np.where(den[..., None] != 0.0, num / np.where(den != 0.0, den, 1.0)[..., None], 0.0)
            # left branch: softmax over the tokens of this group up to and including i
            logits = scale * np.einsum("bha,bhja->bhj", q[:, :, i], k[:, :, lo:i + 1])
            e = np.exp(logits - logits.max(axis=-1, keepdims=True))
            prob = e / e.sum(axis=-1, keepdims=True)
            loc = np.einsum("bhj,bhjc->bhc", prob, v[:, :, lo:i + 1])
            o[:, :, i] = alpha * glob + loc
        # the group is complete: its sums join the group-level cumulative sums
        S = S + np.matmul(np.swapaxes(fk[:, :, lo:hi], -1, -2), v[:, :, lo:hi])
        z = z + fk[:, :, lo:hi].sum(axis=2)
    o += causal_dwconv(v, w, st.win)
    return o, State(S, z, _next_window(st.win, v), st.pos + T)


# ---------------------------------------------------------------------------
# Draft trees: verification and commit (Sec. 4.2)
# ---------------------------------------------------------------------------

def check_tree(parent: np.ndarray) -> None:
    for n, p in enumerate(parent):
        if not (-1 <= int(p) < n):
            raise ValueError(f"node {n}: parent {int(p)} is not an earlier node or -1")


def ancestors_or_self(parent: np.ndarray, n: int) -> list[int]:
    """Root-to-node chain of node n (root first, n last)."""
    chain = []
    while n >= 0:
        chain.append(int(n))
        n = int(parent[n])
    chain.reverse()
    return chain


def verify_tree(q, k, v, parent, w, kind: str, eps: float, state: State):
    """Outputs for every node of a per-sequence draft tree; the state is left untouched.

    q, k, v [B,H,N,d]; parent [B,N].  Node n attends to the committed prefix
    (through the shared S, z: "identical prefixes are computed only once",
    Sec. 5.3) and to its ancestors and itself (tree mask, Sec. 4.2).  The
    convolution is unfolded along the ancestor chain: tap t reads the t-th
    ancestor while it exists and the committed window behind the tree
    otherwise, never a sibling (Fig. "DWConv" (b)).
    """
    q, k, v, w = _f64(q, k, v, w)
    B, H, N, d = q.shape
    W = w.shape[2]
    fq, fk = phi(q, kind), phi(k, kind)
    o = np.zeros_like(v)
    for b in range(B):
        check_tree(parent[b])
        for n in range(N):
            chain = ancestors_or_self(parent[b], n)          # root .. n
            depth = len(chain)
            S = state.S[b] + np.einsum("hma,hmc->hac", fk[b][:, chain, :], v[b][:, chain, :])
            z = state.z[b] + fk[b][:, chain, :].sum(axis=1)
            num = np.einsum("ha,hac->hc", fq[b, :, n], S)
            den = np.einsum("ha,ha->h", fq[b, :, n], z)
            conv = np.zeros((H, d))
            for t in range(W):
                if t < depth:
                    u = v[b][:, chain[depth - 1 - t], :]
                else:                                          # v_{-(t-depth+1)} of the committed prefix
                    u = state.win[b][:, (W - 1) - (t - depth + 1), :]
                conv += w[:, :, t] * u
            o[b, :, n, :] = num / (den + eps)[:, None] + conv
    return o


def commit(k, v, parent, accept_node, kind: str, state: State, max_depth: int):
    """Absorb the accepted root-to-node path as if its tokens had been decoded one by one.

    accept_node [B]: deepest accepted node, -1 for none.  Returns
    (new State, path [B, max_depth] padded with -1, commit_len [B]).
    """
    k, v = _f64(k, v)
    B, H, N, d = k.shape
    new = state.copy()
    path = np.full((B, max_depth), -1, dtype=np.int32)
    clen = np.zeros((B,), dtype=np.int32)
    for b in range(B):
        check_tree(parent[b])
        a = int(accept_node[b])
        if not (-1 <= a < N):
            raise ValueError(f"sequence {b}: accepted node {a} is not in the tree")
        chain = ancestors_or_self(parent[b], a) if a >= 0 else []
        if len(chain) > max_depth:
            raise ValueError(f"sequence {b}: accepted path longer than max_depth")
        clen[b] = len(chain)
        path[b, :len(chain)] = chain
        for n in chain:
            fk = phi(k[b, :, n], kind)
            new.S[b] += fk[:, :, None] * v[b, :, n][:, None, :]
            new.z[b] += fk
            new.win[b] = _next_window(new.win[b][None], v[b, :, n][None, :, None, :])[0]
        new.pos[b] += len(chain)
    return new, path, clen


def accept_greedy(parent, draft_token, pred_root, pred):
    """Greedy acceptance of a draft tree by the verifier's arg-max tokens (Sec. 4.2: the original model accepts or
    rejects the drafted tokens).

    Node n is accepted when draft_token[n] equals the verifier's token at the node it hangs from (pred_root for a
    child of the committed prefix, pred[parent[n]] otherwise) and that node is accepted itself.  Written as the
    definition, in node order (parent[n] < n, so a node's parent is decided before the node).

    parent, draft_token, pred: [B, N] integers; pred_root: [B].  Returns (accept_node [B], accept_len [B],
    next_token [B]): the deepest accepted node (the smallest index among equally deep ones, -1 for none), its depth,
    and the verifier's token that follows the accepted chain.
    """
    parent = np.asarray(parent)
    B, N = parent.shape
    node = np.full((B,), -1, dtype=np.int32)
    length = np.zeros((B,), dtype=np.int32)
    nxt = np.zeros((B,), dtype=np.int32)
    for b in range(B):
        check_tree(parent[b])
        accepted = [False] * N
        depth = [0] * N
        best, best_depth = -1, 0
        for n in range(N):
            p = int(parent[b, n])
            if p < 0:
                accepted[n] = int(draft_token[b][n]) == int(pred_root[b])
                depth[n] = 1
            else:
                accepted[n] = accepted[p] and int(draft_token[b][n]) == int(pred[b][p])
                depth[n] = depth[p] + 1
            if accepted[n] and depth[n] > best_depth:      # strict: the first (smallest) index of a depth wins
                best, best_depth = n, depth[n]
        node[b], length[b] = best, best_depth
        nxt[b] = int(pred[b][best]) if best >= 0 else int(pred_root[b])
    return node, length, nxt


def accept_threshold(parent, score, thresh):
    """Acceptance of a draft tree by a per-node score and threshold (Sec. 4.2: the original model accepts or rejects the
    drafted tokens, resampling if needed).

    The paper names no rule.  Both published families reduce to one comparison per node, and that is what this
    computes: node n passes when score[n] >= thresh[n] -- rejection sampling: score = p(token) / q(token) and thresh a
    uniform draw in [0, 1) that the caller supplies; typical acceptance: score = p(token) and thresh the
    entropy-dependent bound -- and it is accepted when it passes and the node it hangs from is accepted (a child of
    the committed prefix: when it passes).  A comparison with a NaN fails.  Written as the definition, in node order
    (parent[n] < n).

    parent [B, N] integers; score, thresh [B, N] float32 (compared as float32, as given).  Returns (accept_node [B],
    accept_len [B]): the deepest accepted node (the smallest index among equally deep ones, -1 for none) and its
    depth; the caller resamples after that node.
    """
    parent = np.asarray(parent)
    score = np.asarray(score, dtype=np.float32)
    thresh = np.asarray(thresh, dtype=np.float32)
    B, N = parent.shape
    node = np.full((B,), -1, dtype=np.int32)
    length = np.zeros((B,), dtype=np.int32)
    for b in range(B):
        check_tree(parent[b])
        accepted = [False] * N
        depth = [0] * N
        best, best_depth = -1, 0
        for n in range(N):
            p = int(parent[b, n])
            passes = bool(score[b, n] >= thresh[b, n])
            accepted[n] = passes and (p < 0 or accepted[p])
            depth[n] = 1 if p < 0 else depth[p] + 1
            if accepted[n] and depth[n] > best_depth:      # strict: the first (smallest) index of a depth wins
                best, best_depth = n, depth[n]
        node[b], length[b] = best, best_depth
    return node, length
