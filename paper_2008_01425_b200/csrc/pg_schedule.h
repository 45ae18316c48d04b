// Host-side graph and schedule builder of the PowerGossip library: edge lists
// for ring / torus / per-round matching / custom graphs, gossip weights
// (Assumption A4), per-worker slot tables and the seeded initial vectors of
// Algorithm 2.  Integer results are exact by construction.
#pragma once
#include <cstdint>
#include <utility>
#include <vector>

namespace pg {

struct Edge {
    int32_t i, j;  // i < j
};

struct Topology {
    int kind = 0;
    int n_workers = 0;
    int torus_rows = 0, torus_cols = 0;
    int weight_rule = 0;
    std::vector<Edge> custom;   // canonicalised
    std::vector<float> W;       // N x N, only for the explicit rule
};

// One Philox4x32-10 block (Salmon et al., SC'11).
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

// Sort pairs as (min, max), drop self loops and duplicates.
void canonicalise(std::vector<Edge>& edges);

// Edge list of one round.  false when the topology is invalid.
bool build_edges(const Topology& t, uint64_t seed, int64_t round, std::vector<Edge>& out);

// Largest number of edges any round can have, and the largest degree.
bool topology_bounds(const Topology& t, int* max_edges, int* max_degree);

// Gossip weight of every edge; false when an explicit matrix breaks A4.
bool edge_weights(const Topology& t, const std::vector<Edge>& edges, std::vector<float>& w);

// Index of the unordered pair {i<j} in the per-pair state: the position in the
// static edge list, or the triangular index when the graph varies over time.
struct PairIndex {
    bool triangular = false;
    int n_workers = 0;
    std::vector<Edge> static_edges;
    int64_t count() const;
    int64_t of(int i, int j) const;   // -1 if the pair has no state
};

// Column `col` of the initial vector of pair (i<j), layer `layer`: m standard
// normals, entry e from Philox counter (e/4, layer, i, j*256+col), Box-Muller.
void init_q_column(uint64_t seed, int i, int j, int layer, int col, int m, float* out);

// Per-worker view of one round: slot s of worker w is its s-th neighbour in
// ascending id order.
struct RoundSlots {
    std::vector<int> degree;                  // per worker
    std::vector<std::vector<int>> slot_edge;  // [worker][slot] -> edge index
    std::vector<std::vector<float>> slot_sign;// +1 if the worker is the edge's smaller end
    std::vector<int> slot_at_i, slot_at_j;    // per edge
};
void build_slots(int n_workers, const std::vector<Edge>& edges, RoundSlots& out);

}  // namespace pg
