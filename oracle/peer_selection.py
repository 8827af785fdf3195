"""CPU oracle for the coordinator's peer selection (Algorithm 3, GenerateGossipMatrix).

TEST INFRASTRUCTURE ONLY; nothing on the product path imports this module and
this module imports nothing from the product.

Plain Python, written for checking by eye, not for speed (n <= 64).  The
maximum matching is Edmonds' blossom algorithm in its textbook form: grow an
alternating forest from the exposed vertices; an edge between two even vertices
of different trees gives an augmenting path; an edge between two even vertices
of the same tree closes an odd cycle, which is contracted to one vertex, the
search is repeated on the smaller graph, and the path found there is lifted
back through the cycle.

Readings taken where Algorithm 3 and Section II-C leave a choice
  * B is symmetrised by the elementwise minimum (Section II-C) and its diagonal
    is ignored.
  * B*_ij = 1 iff B_ij >= B_thres (GetNewConnectedGraph of Algorithm 1) and the
    link exists (B_ij > 0).  B_thres = inf stands for the bottleneck threshold:
    the largest one that still lets as many workers pair up as the link graph allows.
  * An edge is "recently connected" iff R_ij > t - T_thres; an edge that never
    carried an exchange is never recent (R starts at NEVER).
  * IfStronglyConnected on the symmetric Q is plain undirected connectivity.
  * GetOverTimeMatrix: every pair of vertices from two different components of
    the recent graph, provided the link exists at all (B_ij > 0).
  * GetUnmatch: every pair of still unmatched vertices with B_ij > 0.
  * When the first matching is already perfect, match' is empty.
  * The matching is of maximum cardinality on the 0/1 matrix E; bandwidth
    enters only through B*.
  * "Randomly starting from a different node": the vertices are visited in a
    caller-supplied order.  Any maximum matching of E is a correct answer.
  * After selection R_ij = R_ji = t for every chosen pair (both stages).
  * A vertex left without a partner (odd n, or missing links) keeps the
    identity row: pairs[i] = i.
"""
from __future__ import annotations

import math

import numpy as np

NEVER = -(1 << 62)


# ----------------------------------------------------------------------------
# inputs of Algorithm 3
# ----------------------------------------------------------------------------

def symmetrise(B) -> np.ndarray:
    """B_ij = B_ji = min(B_ij, B_ji); diagonal set to zero."""
    B = np.asarray(B, dtype=np.float64)
    S = np.minimum(B, B.T).copy()
    np.fill_diagonal(S, 0.0)
    return S


def default_b_thres(B) -> float:
    """Median of the off-diagonal entries of the symmetrised B (half the links pass)."""
    S = symmetrise(B)
    n = S.shape[0]
    vals = sorted(float(S[i, j]) for i in range(n) for j in range(i + 1, n))
    m = len(vals)
    if m == 0:
        return 0.0
    return vals[m // 2] if m % 2 else 0.5 * (vals[m // 2 - 1] + vals[m // 2])


def default_t_thres(n: int) -> int:
    """Matchings can at best halve the number of components per round, so the
    window has to be longer than log2(n) rounds."""
    return max(2, 2 * math.ceil(math.log2(n))) if n > 1 else 2


def new_timestamps(n: int) -> np.ndarray:
    return np.full((n, n), NEVER, dtype=np.int64)


def connected_graph(B, b_thres: float) -> np.ndarray:
    """GetNewConnectedGraph: B* as a boolean matrix."""
    S = symmetrise(B)
    Bs = (S >= b_thres) & (S > 0.0)       # a zero entry means "no link at all"
    np.fill_diagonal(Bs, False)
    return Bs


def recent_graph(R: np.ndarray, t: int, t_thres: int) -> np.ndarray:
    """Q of IfConnected / GetOverTimeMatrix."""
    n = R.shape[0]
    Q = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in range(n):
            if i != j and R[i, j] != NEVER and int(R[i, j]) > t - t_thres:
                Q[i, j] = Q[j, i] = True
    return Q


def components(Q: np.ndarray) -> list[int]:
    """FindConnectedSubgraph: component label of every vertex."""
    n = Q.shape[0]
    label = [-1] * n
    c = 0
    for s in range(n):
        if label[s] != -1:
            continue
        label[s] = c
        stack = [s]
        while stack:
            v = stack.pop()
            for w in range(n):
                if Q[v, w] and label[w] == -1:
                    label[w] = c
                    stack.append(w)
        c += 1
    return label


def is_connected(Q: np.ndarray) -> bool:
    return max(components(Q)) == 0


# ----------------------------------------------------------------------------
# maximum matching in a general graph (Edmonds), textbook contraction form
# ----------------------------------------------------------------------------

def _path_to_root(v, parent):
    p = [v]
    while parent[p[-1]] is not None:
        p.append(parent[p[-1]])
    return p


def _augmenting_path(adj, mate, order):
    """One augmenting path of the graph ``adj`` w.r.t. ``mate`` or None.

    adj: vertex -> set of neighbours; mate: vertex -> partner or None;
    order: the sequence in which vertices (and neighbours) are visited.
    """
    rank = {v: r for r, v in enumerate(order)}
    parent, root, level = {}, {}, {}
    queue = []
    for v in order:
        if mate[v] is None:
            parent[v], root[v], level[v] = None, v, 0
            queue.append(v)
    qi = 0
    while qi < len(queue):
        v = queue[qi]
        qi += 1
        for w in sorted(adj[v], key=rank.__getitem__):
            if w == mate[v]:
                continue
            if w not in level:
                # w is matched (all exposed vertices are roots): grow the tree by
                # the unmatched edge (v, w) and the matched edge (w, mate[w]).
                u = mate[w]
                parent[w], root[w], level[w] = v, root[v], level[v] + 1
                parent[u], root[u], level[u] = w, root[v], level[v] + 2
                queue.append(u)
            elif level[w] % 2 == 1:
                continue
            elif root[v] != root[w]:
                return _path_to_root(v, parent)[::-1] + _path_to_root(w, parent)
            else:
                return _through_blossom(adj, mate, order, v, w, parent)
    return None


def _through_blossom(adj, mate, order, v, w, parent):
    """(v, w) joins two even vertices of one tree: contract the odd cycle, search
    the contracted graph, lift the path."""
    pv, pw = _path_to_root(v, parent), _path_to_root(w, parent)
    on_pv = set(pv)
    base = next(u for u in pw if u in on_pv)
    down = pv[:pv.index(base) + 1][::-1]          # base ... v
    up = pw[:pw.index(base)]                      # w ... child of base
    cyc = down + up                               # odd length; matched edges (c1,c2),(c3,c4),...
    in_cyc = set(cyc)
    b = ("blossom", len(order), base)             # a fresh vertex name

    adj2 = {}
    for u in adj:
        if u in in_cyc:
            continue
        adj2[u] = {(b if z in in_cyc else z) for z in adj[u]}
    adj2[b] = {z for c in cyc for z in adj[c] if z not in in_cyc}
    mate2 = {u: (b if mate[u] in in_cyc else mate[u]) for u in adj2 if u != b}
    mate2[b] = mate[base]                         # the stem's matched edge, or None at a root
    order2 = [(b if u == base else u) for u in order if u == base or u not in in_cyc]

    p2 = _augmenting_path(adj2, mate2, order2)
    if p2 is None or b not in p2:
        return p2
    pos = p2.index(b)
    # orient the path so that b's unmatched edge leads forward: [..., mate(b), b, z, ...]
    if pos + 1 < len(p2) and p2[pos + 1] == mate2[b] and mate2[b] is not None:
        p2 = p2[::-1]
        pos = p2.index(b)
    if pos + 1 == len(p2):                        # b is the last vertex: exposed, turn around
        p2 = p2[::-1]
        pos = 0
    z = p2[pos + 1]
    i = next(i for i, c in enumerate(cyc) if z in adj[c])
    # even-length alternating walk base -> cyc[i] that arrives on a matched edge
    if i % 2 == 0:
        walk = cyc[:i + 1]
    else:
        walk = [cyc[0]] + cyc[i:][::-1]
    return p2[:pos] + walk + p2[pos + 1:]


def maximum_matching(E: np.ndarray, order=None) -> list[tuple[int, int]]:
    """Maximum-cardinality matching of the undirected graph with boolean adjacency E."""
    n = E.shape[0]
    order = list(range(n)) if order is None else [int(v) for v in order]
    assert sorted(order) == list(range(n))
    adj = {v: {w for w in range(n) if w != v and (E[v, w] or E[w, v])} for v in range(n)}
    mate = {v: None for v in range(n)}
    while True:
        p = _augmenting_path(adj, mate, order)
        if p is None:
            break
        assert len(p) % 2 == 0
        for a in range(0, len(p), 2):
            mate[p[a]], mate[p[a + 1]] = p[a + 1], p[a]
    return sorted((v, mate[v]) for v in range(n) if mate[v] is not None and v < mate[v])


# ----------------------------------------------------------------------------
# Algorithm 3
# ----------------------------------------------------------------------------

def bottleneck_threshold(B, order=None) -> float:
    """The largest threshold for which B* = [B >= threshold] still admits a matching as large
    as the whole link graph [B > 0] does: with it, the first-stage matching of Algorithm 3
    maximises the slowest chosen link (the "bandwidth utilisation" of Section IV-D).  The
    matching size can only shrink as the threshold rises, so a bisection over the sorted
    link speeds finds it."""
    S = symmetrise(B)
    n = S.shape[0]
    speeds = sorted({float(S[i, j]) for i in range(n) for j in range(i + 1, n) if S[i, j] > 0.0})
    if not speeds:
        return 0.0
    full = len(maximum_matching(S > 0.0, order))
    lo, hi = 0, len(speeds) - 1          # speeds[lo] always works
    while lo < hi:
        mid = (lo + hi + 1) // 2
        if len(maximum_matching(S >= speeds[mid], order)) == full:
            lo = mid
        else:
            hi = mid - 1
    return speeds[lo]


def candidate_edges(B, R, t: int, b_thres: float, t_thres: int):
    """Lines 1-5 of GenerateGossipMatrix: returns (E, mode).  b_thres = inf selects the
    bottleneck threshold of this B."""
    S = symmetrise(B)
    if b_thres == float("inf"):
        b_thres = bottleneck_threshold(B)
    Q = recent_graph(R, t, t_thres)
    if is_connected(Q):
        return connected_graph(B, b_thres), "bandwidth"
    label = components(Q)
    n = S.shape[0]
    E = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in range(n):
            if i != j and label[i] != label[j] and S[i, j] > 0.0:
                E[i, j] = True
    return E, "merge"


def generate_gossip_matrix(B, R, t: int, b_thres: float, t_thres: int, order1=None, order2=None):
    """Algorithm 3.  Returns (pairs, info); R is NOT modified (see record_round).

    pairs[i] = the peer of worker i, or i when it has none this round.
    info: mode, E, first-stage matching, second-stage matching.
    """
    S = symmetrise(B)
    n = S.shape[0]
    E, mode = candidate_edges(B, R, t, b_thres, t_thres)
    match = maximum_matching(E, order1)
    match2 = []
    if 2 * len(match) != n:
        taken = {v for e in match for v in e}
        E2 = np.zeros((n, n), dtype=bool)
        for i in range(n):
            for j in range(n):
                if i != j and i not in taken and j not in taken and S[i, j] > 0.0:
                    E2[i, j] = True
        match2 = maximum_matching(E2, order2)
    pairs = list(range(n))
    for i, j in match + match2:
        pairs[i], pairs[j] = j, i
    return pairs, {"mode": mode, "E": E, "match": match, "match2": match2}


def record_round(R: np.ndarray, pairs, t: int) -> None:
    """The timestamp matrix records the round's exchanges."""
    for i, j in enumerate(pairs):
        if j != i:
            R[i, j] = t
            R[j, i] = t


def generate_W(pairs) -> np.ndarray:
    """GenerateW: 1/2 on matched pairs and on their diagonal entries; a worker
    without a peer keeps the identity row so that W stays doubly stochastic."""
    n = len(pairs)
    W = np.zeros((n, n), dtype=np.float64)
    for i, j in enumerate(pairs):
        if i == j:
            W[i, i] = 1.0
        else:
            W[i, i] = 0.5
            W[i, j] = 0.5
    return W
