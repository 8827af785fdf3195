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
// blossoms kept contracted through a "base" label per vertex.  n <= 64: a row of the adjacency
// matrix is one 64-bit mask (bit w of row v = edge v-w), neighbours are visited in ascending order
// by peeling the lowest set bit, and all working storage is fixed-size.
class BlossomMatcher {
public:
    BlossomMatcher(int n, const uint64_t* rows) : n_(n), row_(rows)
    {
        for (int v = 0; v < n; ++v) mate_[v] = -1;
    }

    const int* solve()
    {
        // start from a greedy matching (first free neighbour of every free vertex): on the dense
        // graphs of this rule it is already close to maximum, and only the few vertices it
        // leaves free need a search for an augmenting path
        uint64_t free_mask = n_ == 64 ? ~0ull : ((1ull << n_) - 1);
        for (int v = 0; v < n_; ++v) {
            if (mate_[v] != -1) continue;
            const uint64_t cand = row_[v] & free_mask & ~(1ull << v);
            if (cand != 0) {
                const int w = __builtin_ctzll(cand);
                mate_[v] = w;
                mate_[w] = v;
                free_mask &= ~((1ull << v) | (1ull << w));
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
    // first common blossom base on the two root paths
    int common_base(int a, int b)
    {
        uint64_t on_path = 0;
        for (int v = a;;) {
            v = base_[v];
            on_path |= 1ull << v;
            if (mate_[v] == -1) break;
            v = up_[mate_[v]];
        }
        for (int v = b;;) {
            v = base_[v];
            if ((on_path >> v) & 1ull) return v;
            v = up_[mate_[v]];
        }
    }

    // walk from v down to the blossom base b, marking the bases on the way and re-hanging
    // the odd vertices so that the path can later be flipped in either direction
    void mark_side(int v, int b, int child, uint64_t& in_blossom)
    {
        while (base_[v] != b) {
            in_blossom |= 1ull << base_[v];
            in_blossom |= 1ull << base_[mate_[v]];
            up_[v] = child;
            child = mate_[v];
            v = up_[mate_[v]];
        }
    }

    // returns the free vertex that ends an augmenting path from root, or -1
    int grow_tree(int root)
    {
        uint64_t seen = 1ull << root;
        for (int i = 0; i < n_; ++i) {
            up_[i] = -1;
            base_[i] = i;
        }
        int head = 0, tail = 0;
        fifo_[tail++] = root;
        while (head < tail) {
            const int v = fifo_[head++];
            for (uint64_t nb = row_[v]; nb != 0; nb &= nb - 1) {
                const int w = __builtin_ctzll(nb);
                if (base_[v] == base_[w] || mate_[v] == w) continue;
                if (w == root || (mate_[w] != -1 && up_[mate_[w]] != -1)) {
                    // w is an even vertex of the tree: odd cycle, contract it
                    const int b = common_base(v, w);
                    uint64_t in_blossom = 0;
                    mark_side(v, b, w, in_blossom);
                    mark_side(w, b, v, in_blossom);
                    for (int i = 0; i < n_; ++i) {
                        if (!((in_blossom >> base_[i]) & 1ull)) continue;
                        base_[i] = b;
                        if (!((seen >> i) & 1ull)) {
                            seen |= 1ull << i;
                            fifo_[tail++] = i;
                        }
                    }
                } else if (up_[w] == -1) {
                    up_[w] = v;
                    if (mate_[w] == -1) return w;
                    seen |= 1ull << mate_[w];
                    fifo_[tail++] = mate_[w];
                }
            }
        }
        return -1;
    }

    int n_;
    const uint64_t* row_;
    int mate_[kMaxWorkers], up_[kMaxWorkers], base_[kMaxWorkers], fifo_[kMaxWorkers];
};

// Adjacency rows (bit j of row i) of a 0/1 matrix stored as bytes.
void rows_of(int n, const std::vector<uint8_t>& E, uint64_t* rows)
{
    for (int i = 0; i < n; ++i) {
        uint64_t bits = 0;
        for (int j = 0; j < n; ++j) bits |= (uint64_t)(E[(size_t)i * n + j] != 0 && i != j) << j;
        rows[i] = bits;
    }
}

// RandomlyMaxMatch: relabel the vertices by a keyed shuffle, match, map back.
// rows: adjacency of E as 64-bit masks.  Returns the number of matched pairs; mate[v] = partner or -1.
int randomly_max_match(int n, const uint64_t* rows, uint64_t seed, uint64_t t, uint32_t stage, int* mate)
{
    const uint64_t s = seed ^ 0x5350454552ull;
    uint32_t h = mix32((uint32_t)(s & 0xFFFFFFFFull) ^ kSeedPad);
    h = mix32(h ^ (uint32_t)(s >> 32));
    h = mix32(h ^ (uint32_t)(t & 0xFFFFFFFFull));
    h = mix32(h ^ (uint32_t)(t >> 32));
    h = mix32(h ^ stage);
    int perm[kMaxWorkers], where[kMaxWorkers];
    for (int i = 0; i < n; ++i) perm[i] = i;
    for (int j = n - 1; j >= 1; --j) {
        const uint32_t r = mix32(h ^ (uint32_t)j) % (uint32_t)(j + 1);
        std::swap(perm[j], perm[r]);
    }
    for (int a = 0; a < n; ++a) where[perm[a]] = a;
    // relabelled graph: vertex a stands for perm[a]; its neighbours are where[] of perm[a]'s
    uint64_t P[kMaxWorkers];
    for (int a = 0; a < n; ++a) {
        uint64_t bits = 0;
        for (uint64_t m = rows[perm[a]]; m != 0; m &= m - 1) bits |= 1ull << where[__builtin_ctzll(m)];
        P[a] = bits;
    }
    BlossomMatcher m(n, P);
    const int* pm = m.solve();
    int pairs = 0;
    for (int i = 0; i < n; ++i) mate[i] = -1;
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
    uint64_t rows[kMaxWorkers];
    rows_of(n, E, rows);
    BlossomMatcher m(n, rows);
    const int* mate = m.solve();
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
    // Everything that depends on the bandwidth matrix and the threshold setting alone is derived
    // once and kept while the caller passes the same values again (compared byte for byte).
    const size_t cells = (size_t)n * n;
    const bool same_setting = st.seen_b_thres_default == st.b_thres_default &&
                              (st.b_thres_default || std::memcmp(&st.seen_b_thres_setting, &st.b_thres, sizeof(double)) == 0);
    if (!(st.derived_valid && same_setting && st.seen_bandwidth.size() == cells &&
          std::memcmp(st.seen_bandwidth.data(), bandwidth, cells * sizeof(double)) == 0)) {
        st.derived_valid = false;
        for (size_t i = 0; i < cells; ++i)
            if (bandwidth[i] != bandwidth[i] || bandwidth[i] < 0.0) return SAPS_ERR_INVALID;

        // B_ij = B_ji = min(B_ij, B_ji)
        std::vector<double>& S = st.sym_bandwidth;
        S.assign(cells, 0.0);
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j)
                if (i != j) S[(size_t)i * n + j] = std::min(bandwidth[(size_t)i * n + j], bandwidth[(size_t)j * n + i]);

        double thres = st.b_thres;
        if (std::isinf(thres) && thres > 0.0) {
            thres = bottleneck_threshold(n, S);
        } else if (st.b_thres_default) {
            std::vector<double> links;
            links.reserve((size_t)n * (n - 1) / 2);
            for (int i = 0; i < n; ++i)
                for (int j = i + 1; j < n; ++j) links.push_back(S[(size_t)i * n + j]);
            // median without a full sort: the upper middle element, then the largest below it
            const size_t m = links.size();
            if (m == 0) {
                thres = 0.0;
            } else {
                std::nth_element(links.begin(), links.begin() + m / 2, links.end());
                const double upper = links[m / 2];
                thres = m % 2 ? upper : 0.5 * (*std::max_element(links.begin(), links.begin() + m / 2) + upper);
            }
        }
        // links with B_ij > 0 and links of B* as row masks
        for (int i = 0; i < n; ++i) {
            uint64_t any = 0, fast = 0;
            const double* b = &S[(size_t)i * n];
            for (int j = 0; j < n; ++j) {
                any |= (uint64_t)(b[j] > 0.0) << j;
                fast |= (uint64_t)(b[j] > 0.0 && b[j] >= thres) << j;
            }
            st.any_link[i] = any & ~(1ull << i);
            st.fast_link[i] = fast & ~(1ull << i);
        }
        st.seen_bandwidth.assign(bandwidth, bandwidth + cells);
        st.seen_b_thres_setting = st.b_thres;
        st.seen_b_thres_default = st.b_thres_default;
        st.derived_b_thres = thres;
        st.derived_valid = true;
    }
    const uint64_t* any_link = st.any_link;
    const uint64_t* fast_link = st.fast_link;
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

    uint64_t E[kMaxWorkers] = {};
    if (ncomp == 1) {
        for (int i = 0; i < n; ++i) E[i] = fast_link[i];                      // E = B*
    } else {
        uint64_t members[kMaxWorkers] = {};                                    // GetOverTimeMatrix
        for (int i = 0; i < n; ++i) members[label[i]] |= 1ull << i;
        for (int i = 0; i < n; ++i) E[i] = any_link[i] & ~members[label[i]];
    }

    int mate[kMaxWorkers];
    const int first = randomly_max_match(n, E, st.seed, t, 1, mate);
    if (2 * first != n) {
        // GetUnmatch: every link between two still unmatched workers, bandwidth ignored
        uint64_t unmatched = 0;
        for (int i = 0; i < n; ++i) unmatched |= (uint64_t)(mate[i] == -1) << i;
        uint64_t E2[kMaxWorkers] = {};
        for (int i = 0; i < n; ++i) E2[i] = ((unmatched >> i) & 1ull) ? (any_link[i] & unmatched) : 0ull;
        int mate2[kMaxWorkers];
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
