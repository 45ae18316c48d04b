// Graph / schedule builder and seeded initial vectors (host only).
#include "pg_schedule.h"

#include <algorithm>
#include <cmath>
#include <numeric>

namespace pg {

namespace {
inline void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
    const uint64_t p = static_cast<uint64_t>(a) * static_cast<uint64_t>(b);
    hi = static_cast<uint32_t>(p >> 32);
    lo = static_cast<uint32_t>(p);
}
}  // namespace

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
    uint32_t x[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
    uint32_t k[2] = {key[0], key[1]};
    for (int r = 0; r < 10; ++r) {
        if (r > 0) {
            k[0] += kWeyl0;
            k[1] += kWeyl1;
        }
        uint32_t hi0, lo0, hi1, lo1;
        mulhilo(kMul0, x[0], hi0, lo0);
        mulhilo(kMul1, x[2], hi1, lo1);
        const uint32_t y0 = hi1 ^ x[1] ^ k[0];
        const uint32_t y2 = hi0 ^ x[3] ^ k[1];
        x[0] = y0;
        x[1] = lo1;
        x[2] = y2;
        x[3] = lo0;
    }
    for (int t = 0; t < 4; ++t) out[t] = x[t];
}

void canonicalise(std::vector<Edge>& edges) {
    std::vector<Edge> tmp;
    tmp.reserve(edges.size());
    for (const Edge& e : edges) {
        if (e.i == e.j) continue;
        tmp.push_back(Edge{std::min(e.i, e.j), std::max(e.i, e.j)});
    }
    std::sort(tmp.begin(), tmp.end(), [](const Edge& a, const Edge& b) {
        return a.i != b.i ? a.i < b.i : a.j < b.j;
    });
    tmp.erase(std::unique(tmp.begin(), tmp.end(),
                          [](const Edge& a, const Edge& b) { return a.i == b.i && a.j == b.j; }),
              tmp.end());
    edges.swap(tmp);
}

bool build_edges(const Topology& t, uint64_t seed, int64_t round, std::vector<Edge>& out) {
    out.clear();
    const int N = t.n_workers;
    if (N < 2) return false;
    switch (t.kind) {
        case 0: {  // ring
            for (int w = 0; w < N; ++w) out.push_back(Edge{w, (w + 1) % N});
            break;
        }
        case 1: {  // torus
            const int R = t.torus_rows, C = t.torus_cols;
            if (R < 1 || C < 1 || static_cast<int64_t>(R) * C != N) return false;
            for (int w = 0; w < N; ++w) {
                const int r = w / C, c = w % C;
                out.push_back(Edge{w, r * C + (c + 1) % C});      // right
                out.push_back(Edge{w, ((r + 1) % R) * C + c});    // down
            }
            break;
        }
        case 2: {  // a fresh perfect matching per round
            if (N % 2 != 0) return false;
            std::vector<int> perm(N);
            std::iota(perm.begin(), perm.end(), 0);
            const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
            const uint64_t ur = static_cast<uint64_t>(round);
            for (int k = N - 1; k >= 1; --k) {
                const uint32_t ctr[4] = {static_cast<uint32_t>(k), static_cast<uint32_t>(ur),
                                         static_cast<uint32_t>(ur >> 32), 0xFFFFFFFFu};
                uint32_t x[4];
                philox4x32_10(ctr, key, x);
                const uint64_t draw = (static_cast<uint64_t>(x[1]) << 32) | x[0];
                std::swap(perm[k], perm[static_cast<int>(draw % static_cast<uint64_t>(k + 1))]);
            }
            for (int a = 0; a + 1 < N; a += 2) out.push_back(Edge{perm[a], perm[a + 1]});
            break;
        }
        case 3: {  // custom
            for (const Edge& e : t.custom) {
                if (e.i < 0 || e.j < 0 || e.i >= N || e.j >= N) return false;
                out.push_back(e);
            }
            break;
        }
        default:
            return false;
    }
    canonicalise(out);
    return !out.empty();
}

bool topology_bounds(const Topology& t, int* max_edges, int* max_degree) {
    std::vector<Edge> e;
    if (!build_edges(t, 0, 0, e)) return false;
    if (t.kind == 2) {
        *max_edges = t.n_workers / 2;
        *max_degree = 1;
        return true;
    }
    std::vector<int> deg(t.n_workers, 0);
    for (const Edge& x : e) {
        ++deg[x.i];
        ++deg[x.j];
    }
    *max_edges = static_cast<int>(e.size());
    *max_degree = *std::max_element(deg.begin(), deg.end());
    return true;
}

bool edge_weights(const Topology& t, const std::vector<Edge>& edges, std::vector<float>& w) {
    const int N = t.n_workers;
    w.assign(edges.size(), 0.0f);
    if (t.kind == 2) {  // matched pairs have degree one: Metropolis weight 1/2
        std::fill(w.begin(), w.end(), 0.5f);
        return true;
    }
    std::vector<int> deg(N, 0);
    for (const Edge& e : edges) {
        ++deg[e.i];
        ++deg[e.j];
    }
    const int dmax = *std::max_element(deg.begin(), deg.end());
    if (t.weight_rule == 0) {
        for (float& x : w) x = static_cast<float>(1.0 / static_cast<double>(dmax + 1));
        return true;
    }
    if (t.weight_rule == 1) {
        for (size_t e = 0; e < edges.size(); ++e)
            w[e] = static_cast<float>(1.0 / static_cast<double>(1 + std::max(deg[edges[e].i], deg[edges[e].j])));
        return true;
    }
    if (t.weight_rule != 2 || t.W.size() != static_cast<size_t>(N) * N) return false;
    // Assumption A4 on an explicit matrix
    std::vector<char> on_edge(static_cast<size_t>(N) * N, 0);
    for (size_t e = 0; e < edges.size(); ++e) {
        const size_t a = static_cast<size_t>(edges[e].i) * N + edges[e].j;
        const size_t b = static_cast<size_t>(edges[e].j) * N + edges[e].i;
        on_edge[a] = on_edge[b] = 1;
        w[e] = t.W[a];
        if (t.kind != 3 && !(w[e] > 0.0f)) return false;
    }
    for (int r = 0; r < N; ++r) {
        double sum = 0.0;
        for (int c = 0; c < N; ++c) {
            const float v = t.W[static_cast<size_t>(r) * N + c];
            if (v != t.W[static_cast<size_t>(c) * N + r]) return false;      // symmetric
            if (r != c && v < 0.0f) return false;
            if (r != c && v != 0.0f && !on_edge[static_cast<size_t>(r) * N + c]) return false;
            if (!std::isfinite(v)) return false;
            sum += static_cast<double>(v);
        }
        if (std::fabs(sum - 1.0) > 1e-5) return false;                        // stochastic
    }
    return true;
}

int64_t PairIndex::count() const {
    if (triangular) return static_cast<int64_t>(n_workers) * (n_workers - 1) / 2;
    return static_cast<int64_t>(static_edges.size());
}

int64_t PairIndex::of(int i, int j) const {
    if (i == j || i < 0 || j < 0 || i >= n_workers || j >= n_workers) return -1;
    const int a = std::min(i, j), b = std::max(i, j);
    if (triangular) {
        // pairs (0,1),(0,2),...,(0,N-1),(1,2),...
        const int64_t before = static_cast<int64_t>(a) * n_workers - static_cast<int64_t>(a) * (a + 1) / 2;
        return before + (b - a - 1);
    }
    const auto it = std::lower_bound(static_edges.begin(), static_edges.end(), Edge{a, b},
                                     [](const Edge& x, const Edge& y) {
                                         return x.i != y.i ? x.i < y.i : x.j < y.j;
                                     });
    if (it == static_edges.end() || it->i != a || it->j != b) return -1;
    return static_cast<int64_t>(it - static_edges.begin());
}

void init_q_column(uint64_t seed, int i, int j, int layer, int col, int m, float* out) {
    const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
    const double kTwoPi = 6.283185307179586476925286766559;
    const double kInv32 = 1.0 / 4294967296.0;
    const int blocks = (m + 3) / 4;
    for (int b = 0; b < blocks; ++b) {
        const uint32_t ctr[4] = {static_cast<uint32_t>(b), static_cast<uint32_t>(layer),
                                 static_cast<uint32_t>(i),
                                 static_cast<uint32_t>(j) * 256u + static_cast<uint32_t>(col)};
        uint32_t x[4];
        philox4x32_10(ctr, key, x);
        float z[4];
        for (int h = 0; h < 2; ++h) {
            const double u1 = (static_cast<double>(x[2 * h]) + 0.5) * kInv32;
            const double u2 = (static_cast<double>(x[2 * h + 1]) + 0.5) * kInv32;
            const double radius = std::sqrt(-2.0 * std::log(u1));
            z[2 * h] = static_cast<float>(radius * std::cos(kTwoPi * u2));
            z[2 * h + 1] = static_cast<float>(radius * std::sin(kTwoPi * u2));
        }
        for (int t = 0; t < 4; ++t)
            if (4 * b + t < m) out[4 * b + t] = z[t];
    }
}

void build_slots(int n_workers, const std::vector<Edge>& edges, RoundSlots& out) {
    out.degree.assign(n_workers, 0);
    out.slot_edge.assign(n_workers, {});
    out.slot_sign.assign(n_workers, {});
    out.slot_at_i.assign(edges.size(), -1);
    out.slot_at_j.assign(edges.size(), -1);
    // neighbours of every worker with the edge that reaches them
    std::vector<std::vector<std::pair<int, int>>> nb(n_workers);
    for (size_t e = 0; e < edges.size(); ++e) {
        nb[edges[e].i].push_back({edges[e].j, static_cast<int>(e)});
        nb[edges[e].j].push_back({edges[e].i, static_cast<int>(e)});
    }
    for (int w = 0; w < n_workers; ++w) {
        std::sort(nb[w].begin(), nb[w].end());
        out.degree[w] = static_cast<int>(nb[w].size());
        for (size_t s = 0; s < nb[w].size(); ++s) {
            const int e = nb[w][s].second;
            out.slot_edge[w].push_back(e);
            const bool smaller = edges[e].i == w;
            out.slot_sign[w].push_back(smaller ? 1.0f : -1.0f);
            (smaller ? out.slot_at_i : out.slot_at_j)[e] = static_cast<int>(s);
        }
    }
}

}  // namespace pg
