// Host-side peer selection: GenerateGossipMatrix (Algorithm 3) with GetNewConnectedGraph
// (Algorithm 1).  n <= 64, so this is control code that runs on the host ahead of the GPU.
//
// Choices where the paper leaves room:
//   B symmetrised by min (Section II-C); B*_ij = [B_ij >= B_thres]; an edge is recent iff
//   R_ij > t - T_thres and "never" is not recent; a disconnected recent graph yields every
//   cross-component link with B_ij > 0; leftovers are paired over every link with B_ij > 0;
//   the matching is maximum-cardinality (Edmonds' blossom algorithm), started "randomly from
//   different nodes" by relabelling the vertices with a (seed, t, stage)-keyed shuffle.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "../../include/saps.h"
#include "internal.h"

namespace saps {
namespace {

// Maximum-cardinality matching in a general graph: breadth-first alternating trees with
// blossoms kept contracted through a "base" label per vertex.
class BlossomMatcher {
public:
    BlossomMatcher(int n, const std::vector<uint8_t>& adj)
        : n_(n), adj_(adj), mate_(n, -1), up_(n), base_(n), seen_(n), in_blossom_(n), on_path_(n), fifo_(n) {}

    const std::vector<int>& solve()
    {
        // start from a greedy matching (first free neighbour of every free vertex): on the dense
        // graphs of this rule it is already close to maximum, and only the few vertices it
        // leaves free need a search for an augmenting path
        for (int v = 0; v < n_; ++v) {
            if (mate_[v] != -1) continue;
            for (int w = 0; w < n_; ++w) {
                if (w != v && mate_[w] == -1 && edge(v, w)) {
                    mate_[v] = w;
                    mate_[w] = v;
                    break;
                }
            }
        }
        for (int v = 0; v < n_; ++v) {
            if (mate_[v] != -1) continue;
            const int leaf = grow_tree(v);
            // flip the alternating path leaf -> root
            for (int w = leaf; w != -1;) {
                const int pv = up_[w];
                const int next = mate_[pv];
                mate_[w] = pv;
                mate_[pv] = w;
                w = next;
            }
        }
        return mate_;
    }

private:
    bool edge(int a, int b) const { return adj_[(size_t)a * n_ + b] != 0; }

    // first common blossom base on the two root paths
    int common_base(int a, int b)
    {
        std::fill(on_path_.begin(), on_path_.end(), 0);
        for (int v = a;;) {
            v = base_[v];
            on_path_[v] = 1;
            if (mate_[v] == -1) break;
            v = up_[mate_[v]];
        }
        for (int v = b;;) {
            v = base_[v];
            if (on_path_[v]) return v;
            v = up_[mate_[v]];
        }
    }

    // walk from v down to the blossom base b, marking the bases on the way and re-hanging
    // the odd vertices so that the path can later be flipped in either direction
    void mark_side(int v, int b, int child)
    {
        while (base_[v] != b) {
            in_blossom_[base_[v]] = 1;
            in_blossom_[base_[mate_[v]]] = 1;
            up_[v] = child;
            child = mate_[v];
            v = up_[mate_[v]];
        }
    }

    // returns the free vertex that ends an augmenting path from root, or -1
    int grow_tree(int root)
    {
        std::fill(seen_.begin(), seen_.end(), 0);
        std::fill(up_.begin(), up_.end(), -1);
        for (int i = 0; i < n_; ++i) base_[i] = i;
        int head = 0, tail = 0;
        fifo_[tail++] = root;
        seen_[root] = 1;
        while (head < tail) {
            const int v = fifo_[head++];
            for (int w = 0; w < n_; ++w) {
                if (!edge(v, w) || base_[v] == base_[w] || mate_[v] == w) continue;
                if (w == root || (mate_[w] != -1 && up_[mate_[w]] != -1)) {
                    // w is an even vertex of the tree: odd cycle, contract it
                    const int b = common_base(v, w);
                    std::fill(in_blossom_.begin(), in_blossom_.end(), 0);
                    mark_side(v, b, w);
                    mark_side(w, b, v);
                    for (int i = 0; i < n_; ++i) {
                        if (!in_blossom_[base_[i]]) continue;
                        base_[i] = b;
                        if (!seen_[i]) {
                            seen_[i] = 1;
                            fifo_[tail++] = i;
                        }
                    }
                } else if (up_[w] == -1) {
                    up_[w] = v;
                    if (mate_[w] == -1) return w;
                    seen_[mate_[w]] = 1;
                    fifo_[tail++] = mate_[w];
                }
            }
        }
        return -1;
    }

    int n_;
    const std::vector<uint8_t>& adj_;
    std::vector<int> mate_, up_, base_;
    std::vector<char> seen_, in_blossom_, on_path_;
    std::vector<int> fifo_;
};

// RandomlyMaxMatch: relabel the vertices by a keyed shuffle, match, map back.
// Returns the number of matched pairs; mate[v] = partner or -1.
int randomly_max_match(int n, const std::vector<uint8_t>& E, uint64_t seed, uint64_t t, uint32_t stage,
                       std::vector<int>& mate)
{
    const uint64_t s = seed ^ 0x5350454552ull;
    uint32_t h = mix32((uint32_t)(s & 0xFFFFFFFFull) ^ kSeedPad);
    h = mix32(h ^ (uint32_t)(s >> 32));
    h = mix32(h ^ (uint32_t)(t & 0xFFFFFFFFull));
    h = mix32(h ^ (uint32_t)(t >> 32));
    h = mix32(h ^ stage);
    std::vector<int> perm(n);
    for (int i = 0; i < n; ++i) perm[i] = i;
    for (int j = n - 1; j >= 1; --j) {
        const uint32_t r = mix32(h ^ (uint32_t)j) % (uint32_t)(j + 1);
        std::swap(perm[j], perm[r]);
    }
    std::vector<uint8_t> P((size_t)n * n);
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) P[(size_t)a * n + b] = E[(size_t)perm[a] * n + perm[b]];
    BlossomMatcher m(n, P);
    const std::vector<int>& pm = m.solve();
    mate.assign(n, -1);
    int pairs = 0;
    for (int a = 0; a < n; ++a) {
        if (pm[a] != -1) {
            mate[perm[a]] = perm[pm[a]];
            pairs += pm[a] > a;
        }
    }
    return pairs;
}

int matching_size(int n, const std::vector<uint8_t>& E)
{
    BlossomMatcher m(n, E);
    const std::vector<int>& mate = m.solve();
    int pairs = 0;
    for (int v = 0; v < n; ++v) pairs += mate[v] > v;
    return pairs;
}

// The largest threshold for which [B >= threshold] still admits a matching as large as the
// whole link graph [B > 0]: the first-stage matching then maximises the slowest chosen link.
// The matching size is monotone in the threshold, so bisect over the sorted link speeds.
double bottleneck_threshold(int n, const std::vector<double>& B)
{
    std::vector<double> speeds;
    for (int i = 0; i < n; ++i)
        for (int j = i + 1; j < n; ++j)
            if (B[(size_t)i * n + j] > 0.0) speeds.push_back(B[(size_t)i * n + j]);
    if (speeds.empty()) return 0.0;
    std::sort(speeds.begin(), speeds.end());
    speeds.erase(std::unique(speeds.begin(), speeds.end()), speeds.end());
    std::vector<uint8_t> E((size_t)n * n);
    auto size_at = [&](double thr) {
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j) {
                const double b = B[(size_t)i * n + j];
                E[(size_t)i * n + j] = i != j && b > 0.0 && b >= thr;
            }
        return matching_size(n, E);
    };
    const int full = size_at(0.0);
    size_t lo = 0, hi = speeds.size() - 1;
    while (lo < hi) {
        const size_t mid = (lo + hi + 1) / 2;
        if (size_at(speeds[mid]) == full)
            lo = mid;
        else
            hi = mid - 1;
    }
    return speeds[lo];
}

// FindConnectedSubgraph: component label per vertex; returns the number of components.
// n <= 64, so a row of the (symmetric) graph is one 64-bit mask and a component grows by whole
// rows at a time.
int label_components(int n, const uint64_t* row, std::vector<int>& label)
{
    label.assign(n, -1);
    uint64_t unvisited = n == 64 ? ~0ull : ((1ull << n) - 1);
    int c = 0;
    while (unvisited != 0) {
        const int s = __builtin_ctzll(unvisited);
        uint64_t comp = 1ull << s, frontier = comp;
        while (frontier != 0) {
            const int v = __builtin_ctzll(frontier);
            frontier &= frontier - 1;
            const uint64_t fresh = row[v] & ~comp;
            comp |= fresh;
            frontier |= fresh;
        }
        for (uint64_t m = comp; m != 0; m &= m - 1) label[__builtin_ctzll(m)] = c;
        unvisited &= ~comp;
        ++c;
    }
    return c;
}

}  // namespace

int select_peers(SelectState& st, const double* bandwidth, uint64_t t, int32_t* out_pairs)
{
    const int n = st.n;
    if (t < st.last_t) return SAPS_ERR_INVALID;
    for (int i = 0; i < n * n; ++i)
        if (bandwidth[i] != bandwidth[i] || bandwidth[i] < 0.0) return SAPS_ERR_INVALID;

    // B_ij = B_ji = min(B_ij, B_ji)
    std::vector<double> B((size_t)n * n, 0.0);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j)
            if (i != j) B[(size_t)i * n + j] = std::min(bandwidth[(size_t)i * n + j], bandwidth[(size_t)j * n + i]);

    double b_thres = st.b_thres;
    if (std::isinf(b_thres) && b_thres > 0.0) {
        b_thres = bottleneck_threshold(n, B);
    } else if (st.b_thres_default) {
        std::vector<double> links;
        links.reserve((size_t)n * (n - 1) / 2);
        for (int i = 0; i < n; ++i)
            for (int j = i + 1; j < n; ++j) links.push_back(B[(size_t)i * n + j]);
        // median without a full sort: the upper middle element, then the largest below it
        const size_t m = links.size();
        if (m == 0) {
            b_thres = 0.0;
        } else {
            std::nth_element(links.begin(), links.begin() + m / 2, links.end());
            const double upper = links[m / 2];
            b_thres = m % 2 ? upper : 0.5 * (*std::max_element(links.begin(), links.begin() + m / 2) + upper);
        }
    }
    int t_thres = st.t_thres;
    if (t_thres == 0) {
        int lg = 0;
        while ((1 << lg) < n) ++lg;
        t_thres = std::max(2, 2 * lg);
    }

    // IfConnected: recently connected edges, R_ij > t - T_thres.  "Never" is far below every
    // horizon, so the one comparison covers it; an edge counts when either direction is recent.
    const int64_t horizon = (int64_t)t - (int64_t)t_thres;
    uint64_t Q[kMaxWorkers] = {};
    for (int i = 0; i < n; ++i) {
        const int64_t* r = &st.R[(size_t)i * n];
        uint64_t bits = 0;
        for (int j = 0; j < n; ++j) bits |= (uint64_t)(r[j] > horizon) << j;
        Q[i] |= bits & ~(1ull << i);
    }
    for (int i = 0; i < n; ++i)
        for (uint64_t m = Q[i]; m != 0; m &= m - 1) Q[__builtin_ctzll(m)] |= 1ull << i;
    std::vector<int> label;
    const int ncomp = label_components(n, Q, label);

    std::vector<uint8_t> E((size_t)n * n, 0);
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) {
            if (i == j) continue;
            const double b = B[(size_t)i * n + j];
            E[(size_t)i * n + j] = ncomp == 1 ? (b >= b_thres && b > 0.0)        // E = B*
                                              : (label[i] != label[j] && b > 0.0);  // GetOverTimeMatrix
        }

    std::vector<int> mate;
    const int first = randomly_max_match(n, E, st.seed, t, 1, mate);
    if (2 * first != n) {
        // GetUnmatch: every link between two still unmatched workers, bandwidth ignored
        std::vector<uint8_t> E2((size_t)n * n, 0);
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j)
                if (i != j && mate[i] == -1 && mate[j] == -1 && B[(size_t)i * n + j] > 0.0)
                    E2[(size_t)i * n + j] = 1;
        std::vector<int> mate2;
        randomly_max_match(n, E2, st.seed, t, 2, mate2);
        for (int i = 0; i < n; ++i)
            if (mate2[i] != -1) mate[i] = mate2[i];
    }

    for (int i = 0; i < n; ++i) {
        out_pairs[i] = mate[i] == -1 ? i : mate[i];
        if (mate[i] != -1) st.R[(size_t)i * n + mate[i]] = (int64_t)t;
    }
    st.last_t = t;
    return SAPS_OK;
}

}  // namespace saps
