// Host side of the C ABI declared in include/powergossip.h: argument checks,
// workspace carve-up, per-round tables and the order in which the kernels of a
// gossip round are enqueued.  No arithmetic of the method happens here.
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "powergossip.h"
#include "pg_device.h"
#include "pg_schedule.h"

namespace {

using pg::DevState;
using pg::Edge;
using pg::LayerGeom;
using pg::TabLayout;
using pg::Tile;

constexpr int kTabRing = 4;          // device copies of per-round tables kept alive
constexpr size_t kAlign = 256;       // every workspace section starts on this boundary

inline long long round_up(long long v, long long a) { return (v + a - 1) / a * a; }

// Byte offsets of the workspace sections.
struct Layout {
    std::vector<LayerGeom> layers;
    long long x_stride = 0, q_stride = 0, y_stride = 0, ph_stride = 0, z_stride = 0;
    long long up_stride = 0, sp_stride = 0;
    long long n_pairs = 0;
    bool pair_mode = false;        // rank 1 and degree <= 2: layers run through the pair sweep
    int pend_slots = 1;            // corrections that can be pending at a worker in pair mode (its degree)
    bool two_copies = false;       // pair mode on a static graph where rows have several readers: the sweep writes
                                   // to a second copy of X, and the pair vectors live in two copies as well
    bool single_owner = false;     // there, no edge has to write the rows of both of its ends
    bool small_stack = false;      // at most 48 MiB of parameters: the latency regime
    long long n_pair_tiles = 0, n_flush_tiles = 0;
    long long row_tile_cap = 0, col_tile_cap = 0;   // room for the lists with every layer on the three-sweep path
    long long n_pair_tiles_cap = 0, n_flush_tiles_cap = 0;
    int max_edges = 0, max_degree = 0;
    TabLayout tab{};
    long long n_row_tiles = 0, n_col_tiles = 0;
    size_t off_Qn2 = 0, off_Pn = 0, off_edge_tab = 0, off_stage = 0, off_Q2 = 0;
    long long stage_elems = 0;     // largest dense matrix whose rows need padding on upload
    size_t off_X = 0, off_Q = 0, off_Qinv = 0, off_Y = 0, off_Ph = 0, off_Z = 0, off_live = 0,
           off_Up = 0, off_Sp = 0, off_pair_tiles = 0, off_flush_tiles = 0, off_status = 0, off_layers = 0, off_tabs = 0, off_row_tiles = 0, off_col_tiles = 0;
    size_t total = 0;
};

int make_topology(const pg_topology* topo, const float* W_host, pg::Topology& out) {
    if (!topo || topo->n_workers < 2 || topo->n_workers > 32768) return PG_ERR_INVALID;
    if (topo->kind < PG_RING || topo->kind > PG_CUSTOM) return PG_ERR_INVALID;
    out.kind = topo->kind;
    out.n_workers = topo->n_workers;
    out.torus_rows = topo->torus_rows;
    out.torus_cols = topo->torus_cols;
    out.weight_rule = topo->weight_rule;
    out.custom.clear();
    if (topo->kind == PG_CUSTOM) {
        if (topo->n_custom_edges < 1 || !topo->custom_edges) return PG_ERR_INVALID;
        for (int e = 0; e < topo->n_custom_edges; ++e) {
            const int a = topo->custom_edges[2 * e], b = topo->custom_edges[2 * e + 1];
            if (a < 0 || b < 0 || a >= topo->n_workers || b >= topo->n_workers) return PG_ERR_INVALID;
            out.custom.push_back(Edge{a, b});
        }
        pg::canonicalise(out.custom);
        if (out.custom.empty()) return PG_ERR_INVALID;
    }
    if (topo->kind != PG_MATCHING) {
        if (topo->weight_rule < PG_W_UNIFORM || topo->weight_rule > PG_W_EXPLICIT) return PG_ERR_INVALID;
        if (topo->weight_rule == PG_W_EXPLICIT) {
            if (!W_host) return PG_ERR_INVALID;
            out.W.assign(W_host, W_host + static_cast<size_t>(topo->n_workers) * topo->n_workers);
        }
    }
    return PG_OK;
}

// The pair sweep can be switched off (PG_DISABLE_PAIR_SWEEP=1 in the environment
// when the context is created) so that both paths can be compared on one graph.
bool pair_sweep_allowed() {
    const char* v = std::getenv("PG_DISABLE_PAIR_SWEEP");
    return !(v && v[0] == '1');
}

constexpr int kPairChains = 2;       // chains the pair-sweep layers of a large stack are spread over

// Rows per cluster tile of a wide pair-sweep layer: with `resident` clusters
// running at once, split every edge's rows into S equal parts so that the
// max_edges * S tiles fill whole waves as nearly as possible.
int wide_tile_rows(int n, int max_edges, int resident) {
    if (resident <= 0) return pg::kPairWideRows;
    int best_s = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= pg::kPairWideMaxTiles && s * 8 <= std::max(n, 8); ++s) {
        const double waves = static_cast<double>(max_edges) * s / resident;
        const double eff = waves / std::ceil(waves);
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best_s = s;
        }
    }
    const int rows = (n + best_s - 1) / best_s;
    return (rows + pg::kPairWideStep - 1) / pg::kPairWideStep * pg::kPairWideStep;
}

// query_device: ask the current device how many clusters of the wide pair sweep
// fit at once and shape its tiles accordingly.  Section sizes do not depend on
// the answer, so a sizing pass without a device gives the same total.
// Which kernel families are launched with programmatic stream serialisation (the next
// kernel is scheduled during the tail of the previous one and waits for it on the device).
// Measured on B200: the sweeps gain (tiny ring 12.7 -> 9.2 us per round, torus 166 -> 159 us);
// the cluster pair sweep loses badly as a dependent (1.98 -> 2.31 ms on the LSTM-shaped
// stack), so it never is one; the pair edge step gains on small stacks and loses next to
// a side stream, so it is one only on small stacks; a stack with layers on both paths,
// whose round runs on two streams, launches plainly (0.85 vs 0.87 ms on the VGG-shaped ring).
// PG_DEPENDENT_LAUNCH=<mask> overrides (0 = plain launches everywhere).
int dependent_launch_mask(bool small_stack, bool two_streams) {
    if (const char* v = std::getenv("PG_DEPENDENT_LAUNCH")) return std::atoi(v) & 31;
    if (two_streams) return 0;
    return pg::kDepSweep | pg::kDepPairRow | pg::kDepPairMid | (small_stack ? pg::kDepPairEdge : 0);
}

// Which edge writes a worker's corrected rows in the pair sweep: every worker gets exactly one of
// its edges.  Where possible no edge gets both of its ends (a bipartite matching of workers to
// incident edges by augmenting paths; it exists unless a component of the graph is a tree), so that
// the sweep's CTAs all do about the same work; the rest fall back to the worker's first edge.
// own[e]: bit 0 = the smaller end, bit 1 = the larger end.  Returns true if no edge has both bits.
bool assign_owners(int n_workers, const std::vector<Edge>& edges, std::vector<int>& own) {
    const int E = static_cast<int>(edges.size());
    std::vector<std::vector<int>> incident(n_workers);
    for (int e = 0; e < E; ++e) {
        incident[edges[e].i].push_back(e);
        incident[edges[e].j].push_back(e);
    }
    std::vector<int> edge_owner(E, -1), worker_edge(n_workers, -1), seen(E, -1);
    // iterative augmenting path search from worker `root`
    auto augment = [&](int root) {
        std::vector<int> stack_w{root}, stack_pos{0}, via;     // via[d]: edge taken at depth d
        while (!stack_w.empty()) {
            const int w = stack_w.back();
            int& pos = stack_pos.back();
            if (pos >= static_cast<int>(incident[w].size())) {
                stack_w.pop_back();
                stack_pos.pop_back();
                if (!via.empty()) via.pop_back();
                continue;
            }
            const int e = incident[w][pos++];
            if (seen[e] == root) continue;
            seen[e] = root;
            if (edge_owner[e] < 0) {                           // free edge: flip the path
                via.push_back(e);
                for (size_t d = 0; d < via.size(); ++d) {
                    edge_owner[via[d]] = stack_w[d];
                    worker_edge[stack_w[d]] = via[d];
                }
                return true;
            }
            via.push_back(e);
            stack_w.push_back(edge_owner[e]);
            stack_pos.push_back(0);
        }
        return false;
    };
    bool single = true;
    for (int w = 0; w < n_workers; ++w)
        if (!incident[w].empty() && !augment(w)) single = false;
    own.assign(E, 0);
    for (int w = 0; w < n_workers; ++w) {
        if (incident[w].empty()) continue;
        const int e = worker_edge[w] >= 0 ? worker_edge[w] : incident[w][0];
        own[e] |= edges[e].i == w ? 1 : 2;
    }
    for (int e = 0; e < E; ++e)
        if (own[e] == 3) single = false;
    return single;
}

constexpr int kSmCount = 148;        // SMs of the one GPU this library is built for

int make_layout(const pg::Topology& topo, const pg_layer_shape* shapes, int n_layers, int rank,
                Layout& lay, bool query_device = false) {
    if (!shapes || n_layers < 1 || n_layers > 4096) return PG_ERR_INVALID;
    if (rank < 1 || rank > PG_MAX_RANK) return PG_ERR_INVALID;
    if (!pg::topology_bounds(topo, &lay.max_edges, &lay.max_degree)) return PG_ERR_INVALID;
    if (lay.max_degree * rank > PG_MAX_SLOTS) return PG_ERR_INVALID;
    const int N = topo.n_workers;
    const int slots = lay.max_degree * rank;
    lay.n_pairs = topo.kind == PG_MATCHING ? static_cast<long long>(N) * (N - 1) / 2 : lay.max_edges;
    if (lay.n_pairs > INT_MAX / 2) return PG_ERR_INVALID;

    // The pair sweep reads both ends of an edge in one pass.  On a perfect matching a
    // row has one reader, so it is corrected in place.  On a static graph of degree 2
    // with no isolated worker (a ring, a path) a row has up to two readers: the edge in
    // the worker's slot 0 writes the corrected row to a second copy of X, which becomes
    // the current one after the sweep.  (Degree 4 was tried and is slower than the three
    // sweeps: every row pair then needs eight corrections, applied by four CTAs each.)
    lay.pair_mode = false;
    lay.pend_slots = 1;
    lay.two_copies = false;
    lay.single_owner = false;
    if (rank <= 2 && pair_sweep_allowed()) {
        if (lay.max_degree == 1) {
            lay.pair_mode = rank == 1;
        } else if (topo.kind != PG_MATCHING && lay.max_degree == 2) {
            // Rows with two readers (a ring, a path): the edge that owns a worker writes its corrected
            // rows to the second copy of X.  (Degree 4 was tried twice - every reader applying all eight
            // corrections of a row pair, and the raw form below with one owner per worker - and both are
            // slower than the three sweeps: a row then passes through four CTAs.)
            std::vector<Edge> edges;
            if (!pg::build_edges(topo, 0, 0, edges)) return PG_ERR_INVALID;
            std::vector<int> degree(N, 0), own;
            for (const Edge& ed : edges) {
                degree[ed.i] += 1;
                degree[ed.j] += 1;
            }
            const bool single = assign_owners(N, edges, own);
            if (*std::min_element(degree.begin(), degree.end()) >= 1) {
                lay.pair_mode = true;
                lay.pend_slots = lay.max_degree;
                lay.two_copies = true;
                lay.single_owner = single;
            }
        }
    }
    lay.layers.resize(n_layers);
    // aim for about 4096 tiles per sweep, each between 128 KB and 512 KB of X
    long long total_elems = 0;
    for (int l = 0; l < n_layers; ++l)
        if (shapes[l].rows > 0 && shapes[l].cols > 0)
            total_elems += static_cast<long long>(N) * shapes[l].rows * round_up(shapes[l].cols, 4);
    long long tile_elems = std::min<long long>(std::max<long long>(total_elems / 4096, 32 * 1024), 128 * 1024);
    const bool small_stack = total_elems * 4 <= 48LL * 1024 * 1024;
    lay.small_stack = small_stack;
    // Which sweep a layer takes.  A row per warp up to kPairMaxLd floats, per CTA up to kPairMidMaxLd,
    // per cluster beyond.  With two readers per row the pair sweep pays off in two regimes: a stack small
    // enough to live in L2, where it halves the launches of a step, and layers large enough to keep every
    // SM busy for many rows; other layers take the three sweeps.  Rank 2 (rings and paths only): the
    // CTA-per-row sweep has a two-column form for rows its registers hold; everything else takes the
    // three sweeps.
    auto pair_mode_of = [&](int rows, int ld) {
        int mode = !lay.pair_mode ? 0
                   : ld <= pg::kPairMaxLd ? 1
                   : ld <= pg::kPairMidMaxLd ? 3
                   : ld <= pg::kPairWideMaxLd ? 2 : 0;
        const bool large_layer = rows >= 256 && static_cast<long long>(rows) * ld >= (1LL << 20);
        if (lay.two_copies && !small_stack && !large_layer) mode = 0;
        if (rank == 2 && !(mode == 3 && large_layer && ld <= pg::kPairMid2MaxLd)) mode = 0;
        return mode;
    };
    // the raw form (see LayerGeom::raw) exists for the TMA-fed CTA-per-row kernels: at rank 1, and at rank 2
    // where no edge owns both of its ends
    auto raw_of = [&](int mode, int ld) {
        return lay.two_copies && mode == 3 && ld <= 5 * 1024 && (rank == 1 || (rank == 2 && lay.single_owner)) ? 1 : 0;
    };
    // rows the CTA-per-row sweep covers on a large stack with two readers per row (their tiles are sized together)
    long long shared_launch_rows = 0;
    if (lay.two_copies && !small_stack)
        for (int l = 0; l < n_layers; ++l)
            if (shapes[l].rows > 0 && shapes[l].cols > 0 &&
                pair_mode_of(shapes[l].rows, static_cast<int>(round_up(shapes[l].cols, 4))) == 3)
                shared_launch_rows += shapes[l].rows;
    long long x = 0, q = 0, y = 0, ph = 0, z = 0, up = 0, sp = 0;
    lay.n_row_tiles = lay.n_col_tiles = lay.n_pair_tiles = lay.n_flush_tiles = 0;
    lay.row_tile_cap = lay.col_tile_cap = 0;
    for (int l = 0; l < n_layers; ++l) {
        LayerGeom& g = lay.layers[l];
        if (shapes[l].rows < 1 || shapes[l].cols < 1) return PG_ERR_INVALID;
        if (static_cast<long long>(shapes[l].rows) * shapes[l].cols > (1LL << 40)) return PG_ERR_INVALID;
        g.n = shapes[l].rows;
        g.m = shapes[l].cols;
        g.ld = static_cast<int>(round_up(g.m, 4));
        g.npad = static_cast<int>(round_up(g.n, 4));
        // row sweeps: 32 or 64 rows by up to 2048 columns
        g.f_rows = tile_elems >= 64 * 1024 ? pg::kRowTileRowsMax : 32;
        const long long want_cols = std::min<long long>(std::max<long long>(tile_elems / g.f_rows, 128), pg::kRowTileColsMax);
        g.f_rtiles = (g.n + g.f_rows - 1) / g.f_rows;
        g.f_csplit = static_cast<int>((g.ld + want_cols - 1) / want_cols);
        g.f_chunk = static_cast<int>(round_up((g.ld + g.f_csplit - 1) / g.f_csplit, 128));
        g.f_csplit = (g.ld + g.f_chunk - 1) / g.f_chunk;
        // transposed sweep: 64, 128 or 256 rows by 256 columns
        g.t_rows = tile_elems >= 64 * 1024 ? pg::kColTileRowsMax : (tile_elems >= 32 * 1024 ? 128 : 64);
        g.t_rtiles = (g.n + g.t_rows - 1) / g.t_rows;
        g.t_ctiles = (g.ld + pg::kColTileCols - 1) / pg::kColTileCols;
        g.x_off = x;
        g.q_off = q;
        g.y_off = y;
        g.ph_off = ph;
        g.z_off = z;
        x += round_up(static_cast<long long>(g.n) * g.ld, 64);
        q += round_up(static_cast<long long>(rank) * g.ld, 64);
        y += round_up(static_cast<long long>(slots) * g.f_csplit * g.npad, 64);
        ph += round_up(static_cast<long long>(rank) * g.npad, 64);
        z += round_up(static_cast<long long>(slots) * g.t_rtiles * g.ld, 64);
        g.pair_mode = pair_mode_of(g.n, g.ld);
        g.raw = raw_of(g.pair_mode, g.ld);
        g.p_slice = static_cast<int>(round_up((g.ld + pg::kPairCluster - 1) / pg::kPairCluster, 4));
        {   // equal tiles of at most kPairTileRows rows (a multiple of 8: one row per warp and stage);
            // on graphs of degree 2 short matrices are cut finer, down to 16 rows, so that a layer gives
            // about two CTAs per SM
            const int by_height = (g.n + pg::kPairTileRows - 1) / pg::kPairTileRows;
            const int by_count = std::min((296 + lay.max_edges - 1) / lay.max_edges, std::max(g.n / 16, 1));
            // (on a matching every layer of the stack shares one launch, which has tiles enough)
            int parts = lay.two_copies ? std::max(by_height, by_count) : by_height;
            if (g.pair_mode == 3 && shared_launch_rows > 0) {
                // The large layers of such a stack run as two chains of launches side by side (see
                // pg_ctx::chain): tall tiles, about four for every three SMs over both chains.  A tile's
                // prologue (the pending terms' products, the vectors into registers) is hidden by nothing
                // with one CTA per SM, and an SM left without a tile costs as much: measured on the VGG-shaped
                // ring of 16 at rank 1 / rank 2, tiles of 256 rows (192 tiles) 0.732 / 0.904 ms per round,
                // 176 rows (288 tiles) 0.760 / 0.933 ms; one chain with 176 rows 0.777 / 0.934 ms.
                const long long target = std::max<long long>(16, shared_launch_rows * lay.max_edges * 3 / (4 * kSmCount));
                parts = std::max<int>(by_height, static_cast<int>(std::max<long long>(1, (g.n + target / 2) / target)));
            }
            g.p_rows = static_cast<int>(round_up((g.n + parts - 1) / parts, 8));
        }
        if (g.pair_mode == 2) {
            const int resident = query_device
                ? pg::pair_wide_resident_clusters((g.p_slice / 4 + 255) / 256, g.p_slice, lay.pend_slots) : 0;
            g.p_rows = wide_tile_rows(g.n, lay.max_edges, resident);
            if ((g.n + g.p_rows - 1) / g.p_rows > pg::kPairWideMaxTiles)
                g.p_rows = static_cast<int>(round_up((g.n + pg::kPairWideMaxTiles - 1) / pg::kPairWideMaxTiles,
                                                     pg::kPairWideStep));
        }
        g.p_rtiles = (g.n + g.p_rows - 1) / g.p_rows;
        {   // pair edge step: about 2048 partial sums or rows per CTA
            const int max_tiles = g.pair_mode == 2 ? pg::kPairWideMaxTiles : g.p_rtiles;
            const long long work = static_cast<long long>(max_tiles) * g.ld + g.npad;
            // (on a large ring every (edge, layer) of a step is in one launch: larger shares keep it to one wave;
            //  VGG-shaped ring 0.877 -> 0.858 ms per round at rank 1, 1.237 -> 1.195 ms at rank 2)
            const long long per_cta = (lay.two_copies && !small_stack) ? 8192 : 2048;
            g.e_chunks = static_cast<int>(std::min<long long>(std::max<long long>((work + per_cta - 1) / per_cta, 1), pg::kEdgeChunks));
        }
        g.up_off = up;
        g.sp_off = sp;
        lay.row_tile_cap += static_cast<long long>(N) * g.f_rtiles * g.f_csplit;
        lay.col_tile_cap += static_cast<long long>(N) * g.t_rtiles * g.t_ctiles;
        if (g.pair_mode != 0) {
            // wide layers: room for any tile count the device query may choose
            const int max_tiles = g.pair_mode == 2 ? pg::kPairWideMaxTiles : g.p_rtiles;
            // per tile: `rank` vectors of D^T P, and kSpPerTile scalars (||p||^2 or P^T P, the pending terms' products)
            up += round_up(static_cast<long long>(max_tiles) * rank * g.ld, 64);
            sp += static_cast<long long>(max_tiles) * pg::kSpPerTile;
            lay.n_pair_tiles += static_cast<long long>(lay.max_edges) * max_tiles;
            lay.n_flush_tiles += static_cast<long long>(N) * g.f_rtiles * g.f_csplit;
        } else {
            lay.n_row_tiles += static_cast<long long>(N) * g.f_rtiles * g.f_csplit;
            lay.n_col_tiles += static_cast<long long>(N) * g.t_rtiles * g.t_ctiles;
        }
    }
    if (lay.two_copies && lay.n_pair_tiles == 0) {   // no layer for the pair sweep: plain three-sweep context
        lay.pair_mode = false;
        lay.pend_slots = 1;
        lay.two_copies = false;
    }
    lay.up_stride = up;
    lay.sp_stride = sp;
    lay.n_pair_tiles_cap = lay.n_pair_tiles;
    lay.n_flush_tiles_cap = lay.n_flush_tiles;
    if (lay.row_tile_cap > INT_MAX || lay.col_tile_cap > INT_MAX) return PG_ERR_INVALID;
    lay.x_stride = x;
    lay.q_stride = q;
    lay.y_stride = y;
    lay.ph_stride = ph;
    lay.z_stride = z;

    TabLayout& t = lay.tab;
    t.max_edges = lay.max_edges;
    t.n_workers = N;
    t.max_degree = lay.max_degree;
    int o = 0;
    t.off_n_edges = o; o += 4;
    t.off_edge_i = o; o += lay.max_edges;
    t.off_edge_j = o; o += lay.max_edges;
    t.off_pair = o; o += lay.max_edges;
    t.off_w = o; o += lay.max_edges;
    t.off_slot_i = o; o += lay.max_edges;
    t.off_slot_j = o; o += lay.max_edges;
    t.off_degree = o; o += N;
    t.off_slot_edge = o; o += N * lay.max_degree;
    t.off_slot_coef = o; o += N * lay.max_degree;
    t.off_own = o; o += lay.max_edges;
    t.total_ints = static_cast<int>(round_up(o, 64));

    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t at = off;
        off = static_cast<size_t>(round_up(static_cast<long long>(off + bytes), kAlign));
        return at;
    };
    lay.off_X = take(sizeof(float) * static_cast<size_t>(N) * lay.x_stride * (lay.two_copies ? 2 : 1));
    lay.off_Q = take(sizeof(float) * static_cast<size_t>(lay.n_pairs) * lay.q_stride);
    lay.off_Q2 = take(lay.two_copies ? sizeof(float) * static_cast<size_t>(lay.n_pairs) * lay.q_stride : 0);
    lay.off_Qinv = take(sizeof(float) * static_cast<size_t>(lay.n_pairs) * n_layers * rank);
    lay.off_Qn2 = take(sizeof(double) * static_cast<size_t>(lay.n_pairs) * n_layers * rank * pg::kEdgeChunks);
    lay.off_Pn = take(sizeof(float) * static_cast<size_t>(lay.max_edges) * n_layers);
    lay.off_Y = take(sizeof(float) * static_cast<size_t>(N) * lay.y_stride);
    lay.off_Ph = take(sizeof(float) * 2 * static_cast<size_t>(lay.max_edges) * lay.ph_stride);  // two buffers
    lay.off_Up = take(sizeof(float) * static_cast<size_t>(lay.max_edges) * lay.up_stride);
    lay.off_Sp = take(sizeof(double) * static_cast<size_t>(lay.max_edges) * lay.sp_stride);
    lay.off_Z = take(sizeof(float) * static_cast<size_t>(N) * lay.z_stride);
    lay.off_live = take(sizeof(int) * static_cast<size_t>(lay.max_edges) * n_layers * rank);
    lay.off_status = take(sizeof(int) * 64);   // [0] status word, [16..17] grid barrier of the persistent kernel
    lay.stage_elems = 0;
    for (const LayerGeom& g : lay.layers)
        if (g.ld != g.m) lay.stage_elems = std::max(lay.stage_elems, static_cast<long long>(g.n) * g.m);
    lay.off_stage = take(sizeof(float) * static_cast<size_t>(lay.stage_elems));
    lay.off_layers = take(sizeof(LayerGeom) * static_cast<size_t>(n_layers));
    lay.off_edge_tab = take(sizeof(int) * 2 * static_cast<size_t>(n_layers) * pg::kEdgeChunks);
    lay.off_tabs = take(sizeof(int) * static_cast<size_t>(kTabRing + 1) * t.total_ints);   // + one table of an empty graph
    lay.off_row_tiles = take(sizeof(Tile) * static_cast<size_t>(lay.row_tile_cap));
    lay.off_col_tiles = take(sizeof(Tile) * static_cast<size_t>(lay.col_tile_cap));
    lay.off_pair_tiles = take(sizeof(Tile) * static_cast<size_t>(lay.n_pair_tiles_cap));
    lay.off_flush_tiles = take(sizeof(Tile) * static_cast<size_t>(lay.n_flush_tiles_cap));
    lay.total = off;
    return PG_OK;
}

}  // namespace

struct pg_ctx {
    pg::Topology topo;
    pg::PairIndex pairs;
    Layout lay;
    DevState st{};
    uint64_t seed = 0;
    int rank = 1, power_steps = 1, n_layers = 0;
    int64_t round = 0;
    bool y_valid = false;       // Y already holds X Qh for the upcoming round
    // pair sweep: the correction of the last step has not been applied to X yet
    bool pending = false;
    int64_t pending_key = 0;    // round whose table describes the pending correction
    int xbuf = 0;               // which copy of X is current (always 0 unless a correction is pending)
    // Layers are independent of each other, and a power step is a chain of kernels with a short
    // vector-only step between two sweeps over X, during which memory idles.  On large stacks the
    // layers are therefore spread over several chains, each on a stream of the library's own: while
    // one chain is between sweeps another one streams.  chain[0] takes the layers on the three
    // sweeps, chain[1..] the pair-sweep layers.  The chains are forked from the caller's stream
    // (everything enqueued there so far is waited for) and the caller's stream is made to wait for
    // all of them at the end of every call; consecutive rounds on the same stream, with no other call
    // on this context in between, continue the chains without a new fork, so a chain never waits
    // for another one.
    static constexpr int kMaxChains = 4;
    cudaStream_t chain[kMaxChains] = {};
    cudaEvent_t ev_fork = nullptr, ev_join[kMaxChains] = {};
    int n_pair_chains = 0;               // chains the pair-sweep layers are spread over (0: caller's stream)
    bool use_chains = false;
    bool chains_open = false;            // the chains are ordered after all earlier work on chain_origin
    cudaStream_t chain_origin = nullptr;
    int edge_first[kMaxChains] = {}, edge_count[kMaxChains] = {};   // CTAs per edge of a chain's pair edge step
    // pg_rounds on a static graph: two steady-state rounds captured once as a CUDA graph and replayed
    cudaStream_t cap = nullptr;          // origin stream of the capture
    cudaGraphExec_t loop_exec = nullptr;
    int loop_key = -1;                   // buffer parities the captured rounds start from
    int64_t loop_launches = 0;           // kernels in the captured pair of rounds
    bool loop_failed = false;
    int64_t step = 0;           // power steps enqueued so far (selects the P-hat buffer)
    float* ph_buf[2] = {nullptr, nullptr};
    // pair-sweep layers whose rows have several readers: step s reads the pair vectors in q_buf[s & 1]
    // and writes the new ones to the other copy (both point at the one copy otherwise)
    float* q_buf[2] = {nullptr, nullptr};
    Tile* d_pair_tiles = nullptr;
    Tile* d_flush_tiles = nullptr;
    // slice: widest per-CTA column slice (mode 2) or widest padded row (mode 3) in the group
    struct PairGroup { int mode; int nv; int slice; int first; int count; double bytes; bool raw; int max_rows; int chain; };
    std::vector<PairGroup> pair_groups;   // pair tiles grouped by float4 per lane
    int64_t launches = 0;
    char* ws = nullptr;
    int* d_tabs = nullptr;
    int* h_tabs = nullptr;      // pinned staging, kTabRing tables
    cudaEvent_t tab_event[kTabRing] = {};
    int64_t tab_round[kTabRing];
    bool tab_used[kTabRing];
    Tile* d_row_tiles = nullptr;
    Tile* d_col_tiles = nullptr;
    // Algorithm 2 read literally: one mat-vec and one update per iteration
    bool half_step = false;
    int64_t iteration = 0;      // Algorithm 2's counter k
    bool half_pending = false;  // an odd iteration's update has not been applied to X yet
    int random_proj = 0;        // 0 power iteration, 1 random right projections, 2 random left projections
    bool static_graph = true;
    bool failed = false;        // a bounded device-side wait gave up: the state on the device is not trustworthy
    bool coop_ok = false;       // the device supports cooperative launches
    int device = 0;
    // optional per-kernel timing: one event pair per launch while enabled
    bool timing = false;
    struct Span { int kind; double bytes; cudaEvent_t a, b; };
    double normal_param_bytes = 0.0;   // 4 B x parameters handled by the three-sweep path
    double pair_param_bytes = 0.0;     // 4 B x parameters handled by the pair sweep
    std::vector<Span> spans;
};

namespace {

// Fill the pinned copy of round `round`'s table.
int fill_table(pg_ctx* c, int64_t round, int* tab) {
    std::vector<Edge> edges;
    std::vector<float> w;
    if (!pg::build_edges(c->topo, c->seed, round, edges)) return PG_ERR_INVALID;
    if (!pg::edge_weights(c->topo, edges, w)) return PG_ERR_INVALID;
    if (static_cast<int>(edges.size()) > c->lay.max_edges) return PG_ERR_INVALID;
    pg::RoundSlots slots;
    pg::build_slots(c->topo.n_workers, edges, slots);
    const TabLayout& t = c->lay.tab;
    std::memset(tab, 0, sizeof(int) * static_cast<size_t>(t.total_ints));
    tab[t.off_n_edges] = static_cast<int>(edges.size());
    for (size_t e = 0; e < edges.size(); ++e) {
        const int64_t pair = c->pairs.of(edges[e].i, edges[e].j);
        if (pair < 0) return PG_ERR_INVALID;
        tab[t.off_edge_i + e] = edges[e].i;
        tab[t.off_edge_j + e] = edges[e].j;
        tab[t.off_pair + e] = static_cast<int>(pair);
        std::memcpy(&tab[t.off_w + e], &w[e], sizeof(float));
        tab[t.off_slot_i + e] = slots.slot_at_i[e];
        tab[t.off_slot_j + e] = slots.slot_at_j[e];
    }
    {
        // who writes a worker's corrected rows in the pair sweep: on a matching the one edge of either
        // end; elsewhere an assignment of workers to incident edges, spread over the edges where possible
        std::vector<int> own(edges.size(), 3);
        if (c->lay.two_copies) assign_owners(c->topo.n_workers, edges, own);
        for (size_t e = 0; e < edges.size(); ++e) tab[t.off_own + e] = own[e];
    }
    for (int v = 0; v < c->topo.n_workers; ++v) {
        if (slots.degree[v] > t.max_degree) return PG_ERR_INVALID;
        tab[t.off_degree + v] = slots.degree[v];
        for (int s = 0; s < slots.degree[v]; ++s) {
            const int e = slots.slot_edge[v][s];
            const float coef = slots.slot_sign[v][s] * w[e];
            tab[t.off_slot_edge + v * t.max_degree + s] = e;
            std::memcpy(&tab[t.off_slot_coef + v * t.max_degree + s], &coef, sizeof(float));
        }
    }
    return PG_OK;
}

// Device pointer of the table of round `round`, uploading it if needed.
int ensure_table(pg_ctx* c, int64_t round, cudaStream_t stream, const int** out) {
    const int64_t key = c->static_graph ? 0 : round;
    const int slot = static_cast<int>(((key % kTabRing) + kTabRing) % kTabRing);
    const size_t ints = static_cast<size_t>(c->lay.tab.total_ints);
    int* dev = c->d_tabs + static_cast<size_t>(slot) * ints;
    if (c->tab_used[slot] && c->tab_round[slot] == key) {
        *out = dev;
        return PG_OK;
    }
    int* host = c->h_tabs + static_cast<size_t>(slot) * ints;
    if (c->tab_used[slot] && cudaEventSynchronize(c->tab_event[slot]) != cudaSuccess) return PG_ERR_CUDA;
    const int rc = fill_table(c, key, host);
    if (rc != PG_OK) return rc;
    if (cudaMemcpyAsync(dev, host, sizeof(int) * ints, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return PG_ERR_CUDA;
    if (cudaEventRecord(c->tab_event[slot], stream) != cudaSuccess) return PG_ERR_CUDA;
    c->tab_used[slot] = true;
    c->tab_round[slot] = key;
    *out = dev;
    return PG_OK;
}

// Brackets one kernel launch with events when timing is on.
struct Timed {
    pg_ctx* c;
    cudaStream_t s;
    pg_ctx::Span span{};
    bool on;
    // `bytes`: algorithmic bytes of the launch (X read and/or written once)
    Timed(pg_ctx* ctx, int kind, cudaStream_t stream, double bytes) : c(ctx), s(stream), on(ctx->timing) {
        if (!on) return;
        span.kind = kind;
        span.bytes = bytes;
        on = cudaEventCreate(&span.a) == cudaSuccess && cudaEventCreate(&span.b) == cudaSuccess &&
             cudaEventRecord(span.a, s) == cudaSuccess;
    }
    ~Timed() {
        if (on && cudaEventRecord(span.b, s) == cudaSuccess) c->spans.push_back(span);
    }
};

// Kernels and copies go to the device that owns the workspace.
bool bind_device(const pg_ctx* c) {
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return false;
    return cur == c->device || cudaSetDevice(c->device) == cudaSuccess;
}

// Apply the correction the pair sweep left pending, so that X in memory is the
// live model (needed before X, Q or the round counter are read or overwritten).
// G, eta: the caller's gradient step, taken in the same pass (pair-sweep layers only).
int flush_pending(pg_ctx* c, cudaStream_t stream, const float* G = nullptr, float eta = 0.0f) {
    c->chains_open = false;      // whatever follows on the caller's stream must be waited for by the next round
    if (c->half_pending) {
        // the odd iteration's update p q-hat^T, with the scaled coefficients
        const int* tab = nullptr;
        const int rc = ensure_table(c, c->round, stream, &tab);
        if (rc != PG_OK) return rc;
        DevState st = c->st;
        st.Ph = c->ph_buf[0];
        st.half_odd = 1;
        Timed t(c, PG_KERNEL_UPDATE_ONLY, stream, 2.0 * c->normal_param_bytes);
        if (pg::launch_update(st, tab, c->d_row_tiles, static_cast<int>(c->lay.n_row_tiles), stream) != cudaSuccess) {
            cudaGetLastError();
            return PG_ERR_CUDA;
        }
        c->launches += 1;
        c->half_pending = false;
        c->y_valid = false;
        return PG_OK;
    }
    if (!c->pending) return PG_OK;
    const int* tab_prev = nullptr;
    const int rc = ensure_table(c, c->pending_key, stream, &tab_prev);
    if (rc != PG_OK) return rc;
    DevState st = c->st;
    st.Ph = c->ph_buf[(c->step + 1) & 1];
    st.Q = c->q_buf[c->step & 1];     // the vectors the last step stored (the flush tiles are pair-sweep layers)
    // the corrected stack always lands in the first copy of X, the one the caller sees
    st.X = c->st.X + c->xbuf * static_cast<long long>(c->topo.n_workers) * c->lay.x_stride;
    st.Xw = c->st.X;
    st.G = G;
    st.eta = eta;
    {
        Timed t(c, PG_KERNEL_UPDATE_ONLY, stream, (G ? 3.0 : 2.0) * c->pair_param_bytes);
        if (pg::launch_update(st, tab_prev, c->d_flush_tiles, static_cast<int>(c->lay.n_flush_tiles), stream) !=
            cudaSuccess) {
            cudaGetLastError();
            return PG_ERR_CUDA;
        }
    }
    c->launches += 1;
    c->pending = false;
    c->xbuf = 0;
    return PG_OK;
}

// X <- X - eta * G on the layers of `tiles` with no correction pending: the update sweep
// run against the table of an empty graph.
int gradient_only_pass(pg_ctx* c, cudaStream_t stream, const Tile* tiles, long long n_tiles, double param_bytes,
                       const float* G, float eta) {
    if (n_tiles <= 0) return PG_OK;
    DevState st = c->st;
    st.G = G;
    st.eta = eta;
    const int* empty = c->d_tabs + static_cast<size_t>(kTabRing) * c->lay.tab.total_ints;
    Timed t(c, PG_KERNEL_UPDATE_ONLY, stream, 3.0 * param_bytes);
    if (pg::launch_update(st, empty, tiles, static_cast<int>(n_tiles), stream) != cudaSuccess) {
        cudaGetLastError();
        return PG_ERR_CUDA;
    }
    c->launches += 1;
    return PG_OK;
}

// Build and upload the tile lists for the current assignment of layers to paths
// (LayerGeom::pair_mode) and refresh the counts and byte totals that go with them.
// Row and column tiles: worker-major, layers in the caller's order.  Layers on the
// pair sweep get pair tiles, grouped by kernel instantiation, and row tiles for
// flushing a pending correction.
bool upload_tile_lists(pg_ctx* c) {
    Layout& lay = c->lay;
    const int n_layers = c->n_layers;
    const int N = c->topo.n_workers;
    std::vector<Tile> rows, cols, flush, pairs;
    c->pair_groups.clear();
    c->normal_param_bytes = c->pair_param_bytes = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        const double b = 4.0 * N * static_cast<double>(lay.layers[l].n) * lay.layers[l].m;
        (lay.layers[l].pair_mode ? c->pair_param_bytes : c->normal_param_bytes) += b;
    }
    for (int v = 0; v < N; ++v)
        for (int l = 0; l < n_layers; ++l) {
            const LayerGeom& g = lay.layers[l];
            for (int rt = 0; rt < g.f_rtiles; ++rt)
                for (int ct = 0; ct < g.f_csplit; ++ct)
                    (g.pair_mode ? flush : rows).push_back(Tile{v, l, rt, ct});
            if (g.pair_mode) continue;
            for (int rt = 0; rt < g.t_rtiles; ++rt)
                for (int ct = 0; ct < g.t_ctiles; ++ct) cols.push_back(Tile{v, l, rt, ct});
        }
    // Chains (see pg_ctx::chain): on a large stack the pair-sweep layers are spread over two chains of
    // about equal size (largest layer first, each to the chain with the least so far; three chains
    // measured 2 % slower than two on the VGG-shaped ring, one chain 6 % slower).
    std::vector<int> chain_of(n_layers, 0);
    c->n_pair_chains = 0;
    c->use_chains = false;
    // (not on a time-varying graph: a round there is two long launches and a new table, and side by side
    //  they ran 5 % slower on the LSTM-shaped stack: the cluster sweep wants the GPU to itself)
    if (!lay.small_stack && c->static_graph) {
        std::vector<int> order;
        for (int l = 0; l < n_layers; ++l)
            if (lay.layers[l].pair_mode) order.push_back(l);
        const int want = std::min<int>({kPairChains, pg_ctx::kMaxChains - 1, static_cast<int>(order.size())});
        if (want >= 2 || (want >= 1 && !rows.empty())) {
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
                return static_cast<long long>(lay.layers[a].n) * lay.layers[a].ld >
                       static_cast<long long>(lay.layers[b].n) * lay.layers[b].ld;
            });
            std::vector<double> load(want, 0.0);
            for (int l : order) {
                const int k = static_cast<int>(std::min_element(load.begin(), load.end()) - load.begin());
                chain_of[l] = k;
                load[k] += static_cast<double>(lay.layers[l].n) * lay.layers[l].ld;
            }
            c->n_pair_chains = want;
            c->use_chains = true;
        }
    }
    // one launch per group of layers that share the kernel instantiation (and the chain)
    auto group_of = [&](const LayerGeom& g, int* nv, int* slice) {
        if (g.pair_mode == 1) {
            *nv = (g.ld + 127) / 128;
            *slice = 0;
        } else if (g.pair_mode == 3) {
            *nv = (g.ld + 1023) / 1024;
            *slice = g.ld;
        } else {
            *nv = (g.p_slice / 4 + 255) / 256;
            *slice = g.p_slice;
        }
    };
    std::vector<char> done(n_layers, 0);
    for (int l0 = 0; l0 < n_layers; ++l0) {
        if (!lay.layers[l0].pair_mode || done[l0]) continue;
        int nv0 = 0, slice0 = 0;
        group_of(lay.layers[l0], &nv0, &slice0);
        const int first = static_cast<int>(pairs.size());
        double bytes = 0.0;   // every worker's rows read from memory once and written once
        int max_rows = 0;     // tallest tile of the group
        for (int l = l0; l < n_layers; ++l) {
            const LayerGeom& g = lay.layers[l];
            int nv = 0, slice = 0;
            if (!g.pair_mode || done[l] || g.pair_mode != lay.layers[l0].pair_mode || g.raw != lay.layers[l0].raw ||
                chain_of[l] != chain_of[l0])
                continue;
            group_of(g, &nv, &slice);
            if (nv != nv0) continue;
            slice0 = std::max(slice0, slice);     // sizes the shared-memory vectors of the launch
            max_rows = std::max(max_rows, g.p_rows);
            done[l] = 1;
            if (lay.two_copies) {
                // the readers of a row block run next to each other, so the second one finds it in L2
                for (int rt = 0; rt < g.p_rtiles; ++rt)
                    for (int e = 0; e < lay.max_edges; ++e) pairs.push_back(Tile{e, l, rt, 0});
            } else {
                for (int e = 0; e < lay.max_edges; ++e)
                    for (int rt = 0; rt < g.p_rtiles; ++rt) pairs.push_back(Tile{e, l, rt, 0});
            }
            bytes += 8.0 * N * static_cast<double>(g.n) * g.m;
        }
        const int count = static_cast<int>(pairs.size()) - first;
        c->pair_groups.push_back(pg_ctx::PairGroup{lay.layers[l0].pair_mode, nv0, slice0, first, count, bytes,
                                                   lay.layers[l0].raw != 0, max_rows, chain_of[l0]});
    }
    // Launch order: longest rows first (the costliest tiles start first, the cheaper ones fill the end of
    // the launch).  A group with fewer than two tiles per SM joins the group before it, of its kind with
    // longer rows (the kernels take any row up to their template's width): fewer, fuller launches.
    {
        std::vector<pg_ctx::PairGroup>& gr = c->pair_groups;
        std::stable_sort(gr.begin(), gr.end(), [](const pg_ctx::PairGroup& a, const pg_ctx::PairGroup& b) {
            if (a.chain != b.chain) return a.chain < b.chain;
            return a.mode != b.mode ? a.mode < b.mode : (a.raw != b.raw ? a.raw < b.raw : a.nv > b.nv);
        });
        std::vector<Tile> merged;
        std::vector<pg_ctx::PairGroup> out;
        merged.reserve(pairs.size());
        for (size_t i = 0; i < gr.size(); ++i) {
            const pg_ctx::PairGroup& cur = gr[i];
            const int first = static_cast<int>(merged.size());
            merged.insert(merged.end(), pairs.begin() + cur.first, pairs.begin() + cur.first + cur.count);
            if (!out.empty() && cur.mode != 2 && cur.count < 2 * kSmCount && out.back().mode == cur.mode &&
                out.back().raw == cur.raw && out.back().chain == cur.chain) {
                pg_ctx::PairGroup& prev = out.back();       // its tiles end where these begin
                prev.slice = std::max(prev.slice, cur.slice);
                prev.count += cur.count;
                prev.bytes += cur.bytes;
                prev.max_rows = std::max(prev.max_rows, cur.max_rows);
            } else {
                out.push_back(cur);
                out.back().first = first;
            }
        }
        pairs.swap(merged);
        gr.swap(out);
    }
    // serpentine: the transposed sweep walks the stack in the opposite direction to the row
    // sweeps that run before and after it, so each sweep starts on what is still in L2
    std::reverse(cols.begin(), cols.end());
    if (static_cast<long long>(rows.size()) > lay.row_tile_cap || static_cast<long long>(cols.size()) > lay.col_tile_cap ||
        static_cast<long long>(pairs.size()) > lay.n_pair_tiles_cap || static_cast<long long>(flush.size()) > lay.n_flush_tiles_cap)
        return false;
    lay.n_row_tiles = static_cast<long long>(rows.size());
    lay.n_col_tiles = static_cast<long long>(cols.size());
    lay.n_pair_tiles = static_cast<long long>(pairs.size());
    lay.n_flush_tiles = static_cast<long long>(flush.size());
    auto put = [](Tile* dst, const std::vector<Tile>& v) {
        return v.empty() || cudaMemcpy(dst, v.data(), sizeof(Tile) * v.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    };
    // the CTAs of the pair edge step of one edge, chain by chain: (layer, chunk)
    std::vector<int> edge_tab;
    for (int k = 0; k < std::max(c->n_pair_chains, 1); ++k) {
        c->edge_first[k] = static_cast<int>(edge_tab.size() / 2);
        for (int l = 0; l < n_layers; ++l)
            if (lay.layers[l].pair_mode && chain_of[l] == k)
                for (int ch = 0; ch < lay.layers[l].e_chunks; ++ch) {
                    edge_tab.push_back(l);
                    edge_tab.push_back(ch);
                }
        c->edge_count[k] = static_cast<int>(edge_tab.size() / 2) - c->edge_first[k];
    }
    c->st.e_total = static_cast<int>(edge_tab.size() / 2);
    if (!edge_tab.empty() && cudaMemcpy(c->ws + lay.off_edge_tab, edge_tab.data(), sizeof(int) * edge_tab.size(),
                                        cudaMemcpyHostToDevice) != cudaSuccess)
        return false;
    // kernels that share the GPU with another chain's are launched plainly
    c->st.dep_launch = dependent_launch_mask(lay.small_stack, c->use_chains);
    return cudaMemcpy(c->ws + lay.off_layers, lay.layers.data(), sizeof(LayerGeom) * n_layers, cudaMemcpyHostToDevice) ==
               cudaSuccess &&
           put(c->d_row_tiles, rows) && put(c->d_col_tiles, cols) && put(c->d_pair_tiles, pairs) &&
           put(c->d_flush_tiles, flush);
}

// Move every layer to the three-sweep path (the modes that have no pair-sweep form
// need it).  Only before the first round, with nothing pending.
bool leave_pair_mode(pg_ctx* c) {
    if (c->lay.n_pair_tiles == 0) return true;
    for (LayerGeom& g : c->lay.layers) g.pair_mode = g.raw = 0;
    if (c->loop_exec) {
        cudaGraphExecDestroy(c->loop_exec);
        c->loop_exec = nullptr;
    }
    return upload_tile_lists(c);
}

int check_worker_layer(const pg_ctx* c, int worker, int layer) {
    if (!c) return PG_ERR_INVALID;
    if (worker < 0 || worker >= c->topo.n_workers || layer < 0 || layer >= c->n_layers) return PG_ERR_INVALID;
    return PG_OK;
}

int device_status(pg_ctx* c, cudaStream_t stream) {
    int word = 0;
    if (cudaMemcpyAsync(&word, c->st.status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return PG_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return PG_ERR_CUDA;
    if (word & (1 << PG_ERR_TIMEOUT)) {
        // a kernel left in the middle of a step: X, Q and the cached products no longer belong
        // together.  No further round runs on this context.
        c->failed = true;
        c->y_valid = false;
        if (c->loop_exec) {
            cudaGraphExecDestroy(c->loop_exec);
            c->loop_exec = nullptr;
        }
        return PG_ERR_TIMEOUT;
    }
    if (word & (1 << PG_ERR_BOUNDS)) return PG_ERR_BOUNDS;
    if (word & (1 << PG_ERR_NUMERIC)) return PG_ERR_NUMERIC;
    return word == 0 ? PG_OK : PG_ERR_STATE;
}

}  // namespace

extern "C" {

int pg_workspace_bytes(const pg_topology* topo, const pg_layer_shape* shapes, int32_t n_layers,
                       int32_t rank, size_t* bytes_out) {
    if (!bytes_out) return PG_ERR_INVALID;
    pg::Topology t;
    // the explicit matrix does not change the size: validate the graph only
    pg_topology probe;
    if (!topo) return PG_ERR_INVALID;
    probe = *topo;
    if (probe.kind != PG_MATCHING && probe.weight_rule == PG_W_EXPLICIT) probe.weight_rule = PG_W_METROPOLIS;
    int rc = make_topology(&probe, nullptr, t);
    if (rc != PG_OK) return rc;
    Layout lay;
    rc = make_layout(t, shapes, n_layers, rank, lay);
    if (rc != PG_OK) return rc;
    *bytes_out = lay.total;
    return PG_OK;
}

int pg_create(const pg_topology* topo, const float* W_host, const pg_layer_shape* shapes,
              int32_t n_layers, int32_t rank, int32_t power_steps, uint64_t seed,
              void* dev_workspace, size_t workspace_bytes, pg_ctx** ctx_out) {
    if (!ctx_out || power_steps < 1) return PG_ERR_INVALID;
    pg_ctx* c = new (std::nothrow) pg_ctx();
    if (!c) return PG_ERR_INVALID;
    int rc = make_topology(topo, W_host, c->topo);
    if (rc == PG_OK) rc = make_layout(c->topo, shapes, n_layers, rank, c->lay);
    std::vector<Edge> edges0;
    std::vector<float> w0;
    if (rc == PG_OK && !pg::build_edges(c->topo, seed, 0, edges0)) rc = PG_ERR_INVALID;
    if (rc == PG_OK && !pg::edge_weights(c->topo, edges0, w0)) rc = PG_ERR_INVALID;
    if (rc == PG_OK) {
        // workspace: present, aligned, large enough and device memory
        cudaPointerAttributes attr{};
        if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) % kAlign) != 0 ||
            workspace_bytes < c->lay.total) {
            rc = PG_ERR_WORKSPACE;
        } else if (cudaPointerGetAttributes(&attr, dev_workspace) != cudaSuccess ||
                   attr.type != cudaMemoryTypeDevice) {
            cudaGetLastError();
            rc = PG_ERR_WORKSPACE;
        } else {
            c->device = attr.device;
            if (!bind_device(c)) rc = PG_ERR_CUDA;
        }
    }
    if (rc == PG_OK) {
        // same sections and sizes as the sizing pass; tile shapes tuned to this device
        const size_t need = c->lay.total;
        rc = make_layout(c->topo, shapes, n_layers, rank, c->lay, true);
        if (rc == PG_OK && c->lay.total != need) rc = PG_ERR_STATE;
    }
    if (rc != PG_OK) {
        delete c;
        return rc;
    }
    c->seed = seed;
    c->rank = rank;
    c->power_steps = power_steps;
    c->n_layers = n_layers;
    c->static_graph = c->topo.kind != PG_MATCHING;
    {
        int coop = 0;
        c->coop_ok = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) == cudaSuccess && coop != 0;
    }
    c->pairs.triangular = !c->static_graph;
    c->pairs.n_workers = c->topo.n_workers;
    if (c->static_graph) c->pairs.static_edges = edges0;
    c->ws = static_cast<char*>(dev_workspace);
    for (int s = 0; s < kTabRing; ++s) {
        c->tab_used[s] = false;
        c->tab_round[s] = -1;
    }

    const Layout& lay = c->lay;
    DevState& st = c->st;
    st.X = reinterpret_cast<float*>(c->ws + lay.off_X);
    st.Xw = st.X;
    st.Q = reinterpret_cast<float*>(c->ws + lay.off_Q);
    st.Qr = st.Qw = st.Q;
    st.raw_pending = 0;
    c->q_buf[0] = st.Q;
    c->q_buf[1] = lay.two_copies ? reinterpret_cast<float*>(c->ws + lay.off_Q2) : st.Q;
    st.Qinv = reinterpret_cast<float*>(c->ws + lay.off_Qinv);
    st.Qn2 = reinterpret_cast<double*>(c->ws + lay.off_Qn2);
    st.Pn = reinterpret_cast<float*>(c->ws + lay.off_Pn);
    st.half_odd = 0;
    st.Y = reinterpret_cast<float*>(c->ws + lay.off_Y);
    st.Ph = reinterpret_cast<float*>(c->ws + lay.off_Ph);
    st.PhNext = st.Ph + static_cast<long long>(lay.max_edges) * lay.ph_stride;
    c->ph_buf[0] = st.Ph;
    c->ph_buf[1] = st.PhNext;
    st.Up = reinterpret_cast<float*>(c->ws + lay.off_Up);
    st.Sp = reinterpret_cast<double*>(c->ws + lay.off_Sp);
    st.up_stride = lay.up_stride;
    st.sp_stride = lay.sp_stride;
    c->d_pair_tiles = reinterpret_cast<Tile*>(c->ws + lay.off_pair_tiles);
    c->d_flush_tiles = reinterpret_cast<Tile*>(c->ws + lay.off_flush_tiles);
    st.Z = reinterpret_cast<float*>(c->ws + lay.off_Z);
    st.live = reinterpret_cast<int*>(c->ws + lay.off_live);
    st.status = reinterpret_cast<int*>(c->ws + lay.off_status);
    st.layers = reinterpret_cast<const LayerGeom*>(c->ws + lay.off_layers);
    st.edge_tab = reinterpret_cast<const int*>(c->ws + lay.off_edge_tab);
    st.e_total = 0;
    st.x_stride = lay.x_stride;
    st.q_stride = lay.q_stride;
    st.y_stride = lay.y_stride;
    st.ph_stride = lay.ph_stride;
    st.z_stride = lay.z_stride;
    st.n_layers = n_layers;
    st.rank = rank;
    st.n_workers = c->topo.n_workers;
    st.max_degree = lay.max_degree;
    st.f_chunk_max = st.f_rows_max = 0;
    for (const LayerGeom& g : lay.layers) {
        st.f_chunk_max = std::max(st.f_chunk_max, g.f_chunk);
        st.f_rows_max = std::max(st.f_rows_max, g.f_rows);
    }
    st.tab = lay.tab;
#ifdef PG_BOUNDS_CHECK
    {   // section bounds for the bounds-checked build
        auto sec = [&](int id, size_t lo, size_t bytes) {
            st.sec_lo[id] = c->ws + lo;
            st.sec_hi[id] = c->ws + lo + bytes;
        };
        const size_t N = static_cast<size_t>(c->topo.n_workers), E = static_cast<size_t>(lay.max_edges);
        const size_t P = static_cast<size_t>(lay.n_pairs), L = static_cast<size_t>(n_layers);
        sec(pg::kSecX, lay.off_X, sizeof(float) * N * lay.x_stride * (lay.two_copies ? 2 : 1));
        sec(pg::kSecQ, lay.off_Q, (lay.two_copies ? lay.off_Q2 - lay.off_Q : 0) + sizeof(float) * P * lay.q_stride);
        sec(pg::kSecQinv, lay.off_Qinv, sizeof(float) * P * L * rank);
        sec(pg::kSecQn2, lay.off_Qn2, sizeof(double) * P * L * rank * pg::kEdgeChunks);
        sec(pg::kSecPn, lay.off_Pn, sizeof(float) * E * L);
        sec(pg::kSecY, lay.off_Y, sizeof(float) * N * lay.y_stride);
        sec(pg::kSecPh, lay.off_Ph, sizeof(float) * 2 * E * lay.ph_stride);
        sec(pg::kSecUp, lay.off_Up, sizeof(float) * E * lay.up_stride);
        sec(pg::kSecSp, lay.off_Sp, sizeof(double) * E * lay.sp_stride);
        sec(pg::kSecZ, lay.off_Z, sizeof(float) * N * lay.z_stride);
        sec(pg::kSecLive, lay.off_live, sizeof(int) * E * L * rank);
        sec(pg::kSecTabs, lay.off_tabs, sizeof(int) * static_cast<size_t>(kTabRing + 1) * lay.tab.total_ints);
        sec(pg::kSecTiles, lay.off_row_tiles, lay.total - lay.off_row_tiles);
        sec(pg::kSecLayers, lay.off_layers, sizeof(LayerGeom) * L);
    }
#endif
    c->d_tabs = reinterpret_cast<int*>(c->ws + lay.off_tabs);
    c->d_row_tiles = reinterpret_cast<Tile*>(c->ws + lay.off_row_tiles);
    c->d_col_tiles = reinterpret_cast<Tile*>(c->ws + lay.off_col_tiles);

    bool ok = cudaMemset(c->ws, 0, lay.total) == cudaSuccess;
    ok = ok && upload_tile_lists(c);
    // Algorithm 2, initialisation: one standard-normal vector per pair, layer, column
    if (ok) {
        std::vector<Edge> all_pairs;
        if (c->static_graph) {
            all_pairs = edges0;
        } else {
            for (int a = 0; a < c->topo.n_workers; ++a)
                for (int b = a + 1; b < c->topo.n_workers; ++b) all_pairs.push_back(Edge{a, b});
        }
        std::vector<float> block(static_cast<size_t>(lay.q_stride), 0.0f);
        for (size_t p = 0; p < all_pairs.size() && ok; ++p) {
            for (int l = 0; l < n_layers; ++l)
                for (int k = 0; k < rank; ++k)
                    pg::init_q_column(seed, all_pairs[p].i, all_pairs[p].j, l, k, lay.layers[l].m,
                                      block.data() + lay.layers[l].q_off + static_cast<long long>(k) * lay.layers[l].ld);
            ok = cudaMemcpy(st.Q + static_cast<long long>(p) * lay.q_stride, block.data(),
                            sizeof(float) * block.size(), cudaMemcpyHostToDevice) == cudaSuccess;
        }
    }
    ok = ok && cudaMallocHost(&c->h_tabs, sizeof(int) * static_cast<size_t>(kTabRing) * lay.tab.total_ints) == cudaSuccess;
    for (int s = 0; s < kTabRing && ok; ++s)
        ok = cudaEventCreateWithFlags(&c->tab_event[s], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->cap, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    for (int k = 0; k < pg_ctx::kMaxChains && ok; ++k)
        ok = cudaStreamCreateWithFlags(&c->chain[k], cudaStreamNonBlocking) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->ev_join[k], cudaEventDisableTiming) == cudaSuccess;
    if (ok) {
        ok = pg::launch_column_norms(st, lay.n_pairs, nullptr) == cudaSuccess;
        c->launches += 1;
        ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        pg_destroy(c);
        return PG_ERR_CUDA;
    }
    *ctx_out = c;
    return PG_OK;
}

void pg_destroy(pg_ctx* c) {
    if (!c) return;
    for (auto& sp : c->spans) {
        cudaEventDestroy(sp.a);
        cudaEventDestroy(sp.b);
    }
    for (int s = 0; s < kTabRing; ++s)
        if (c->tab_event[s]) cudaEventDestroy(c->tab_event[s]);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    for (int k = 0; k < pg_ctx::kMaxChains; ++k) {
        if (c->ev_join[k]) cudaEventDestroy(c->ev_join[k]);
        if (c->chain[k]) cudaStreamDestroy(c->chain[k]);
    }
    if (c->loop_exec) cudaGraphExecDestroy(c->loop_exec);
    if (c->cap) cudaStreamDestroy(c->cap);
    if (c->h_tabs) cudaFreeHost(c->h_tabs);
    delete c;
}

int pg_write_params(pg_ctx* c, int32_t worker, int32_t layer, const float* host_src, void* stream) {
    int rc = check_worker_layer(c, worker, layer);
    if (rc != PG_OK || !host_src) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    rc = flush_pending(c, static_cast<cudaStream_t>(stream));
    if (rc != PG_OK) return rc;
    const LayerGeom& g = c->lay.layers[layer];
    float* dst = c->st.X + static_cast<long long>(worker) * c->st.x_stride + g.x_off;
    c->y_valid = false;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t dense = sizeof(float) * static_cast<size_t>(g.n) * g.m;
    if (g.ld == g.m) {
        if (cudaMemcpyAsync(dst, host_src, dense, cudaMemcpyHostToDevice, s) != cudaSuccess) return PG_ERR_CUDA;
        return PG_OK;
    }
    // Rows that need padding: one contiguous copy into a staging area, then a kernel spreads the
    // rows (a strided host-to-device copy of narrow rows runs at half the link rate).  The staging
    // area is reused in stream order, like everything else in a context.
    float* stage = reinterpret_cast<float*>(c->ws + c->lay.off_stage);
    if (cudaMemcpyAsync(stage, host_src, dense, cudaMemcpyHostToDevice, s) != cudaSuccess ||
        pg::launch_unpack_rows(dst, g.ld, stage, g.n, g.m, s) != cudaSuccess) {
        cudaGetLastError();
        return PG_ERR_CUDA;
    }
    return PG_OK;
}

int pg_read_params_async(pg_ctx* c, int32_t worker, int32_t layer, float* host_dst, void* stream) {
    int rc = check_worker_layer(c, worker, layer);
    if (rc != PG_OK || !host_dst) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    rc = flush_pending(c, static_cast<cudaStream_t>(stream));
    if (rc != PG_OK) return rc;
    const LayerGeom& g = c->lay.layers[layer];
    const float* src = c->st.X + static_cast<long long>(worker) * c->st.x_stride + g.x_off;
    if (cudaMemcpy2DAsync(host_dst, sizeof(float) * g.m, src, sizeof(float) * g.ld, sizeof(float) * g.m,
                          g.n, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return PG_ERR_CUDA;
    return PG_OK;
}

int pg_read_params(pg_ctx* c, int32_t worker, int32_t layer, float* host_dst, void* stream) {
    const int rc = pg_read_params_async(c, worker, layer, host_dst, stream);
    if (rc != PG_OK) return rc;
    return device_status(c, static_cast<cudaStream_t>(stream));
}

int pg_params_device(pg_ctx* c, int32_t worker, int32_t layer, void* stream, float** dev_ptr_out,
                     int64_t* ld_out) {
    int rc = check_worker_layer(c, worker, layer);
    if (rc != PG_OK || !dev_ptr_out || !ld_out) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    rc = flush_pending(c, static_cast<cudaStream_t>(stream));
    if (rc != PG_OK) return rc;
    const LayerGeom& g = c->lay.layers[layer];
    *dev_ptr_out = c->st.X + static_cast<long long>(worker) * c->st.x_stride + g.x_off;
    *ld_out = g.ld;
    c->y_valid = false;     // the caller is about to change X
    return PG_OK;
}

int pg_device_status(pg_ctx* c, void* stream) {
    if (!c) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    return device_status(c, static_cast<cudaStream_t>(stream));
}

// One round; with G, X also loses eta * G with the round's last update (Algorithm 1, line 6)
// and is left fully updated in memory.
static int round_impl(pg_ctx* c, void* stream_v, const float* G, float eta) {
    if (!c) return PG_ERR_INVALID;
    if (c->failed) return PG_ERR_STATE;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int* tab = nullptr;
    const int* tab_next = nullptr;
    int rc = ensure_table(c, c->round, stream, &tab);
    if (rc == PG_OK) rc = ensure_table(c, c->round + 1, stream, &tab_next);
    if (rc != PG_OK) return rc;
    const int n_rows = static_cast<int>(c->lay.n_row_tiles), n_cols = static_cast<int>(c->lay.n_col_tiles);
    const bool has_pair = c->lay.n_pair_tiles > 0;
    bool ok = true;
    if (c->random_proj) {
        // fresh orthonormal directions, one product, the raw difference, the update
        DevState st = c->st;
        st.Ph = c->ph_buf[0];
        for (int p = 0; p < c->power_steps && ok; ++p) {
            const uint64_t t1 = static_cast<uint64_t>(c->step) + 1u;
            const uint64_t key = c->seed ^ (t1 & 0xFFFFFFFFu) ^ (((t1 >> 32) ^ 0x52503031u) << 32);
            const unsigned klo = static_cast<unsigned>(key), khi = static_cast<unsigned>(key >> 32);
            {
                Timed t(c, PG_KERNEL_EDGE_LEFT, stream, 0.0);
                ok = ok && pg::launch_random_directions(st, tab, c->lay.max_edges, klo, khi,
                                                        c->random_proj == 1 ? 0 : 1, stream) == cudaSuccess;
            }
            if (c->random_proj == 1) {
                {
                    Timed t(c, PG_KERNEL_FORWARD, stream, c->normal_param_bytes);
                    ok = ok && pg::launch_forward(st, tab, c->d_row_tiles, n_rows, stream) == cudaSuccess;
                }
                Timed t(c, PG_KERNEL_EDGE_RIGHT, stream, 0.0);
                ok = ok && pg::launch_edge_raw(st, tab, c->lay.max_edges, stream) == cudaSuccess;
            } else {
                {
                    Timed t(c, PG_KERNEL_TRANSPOSED, stream, c->normal_param_bytes);
                    ok = ok && pg::launch_transposed(st, tab, c->d_col_tiles, n_cols, stream) == cudaSuccess;
                }
                Timed t(c, PG_KERNEL_EDGE_RIGHT, stream, 0.0);
                ok = ok && pg::launch_edge_right(st, tab, c->lay.max_edges, stream) == cudaSuccess;
            }
            {
                Timed t(c, PG_KERNEL_UPDATE_ONLY, stream, 2.0 * c->normal_param_bytes);
                ok = ok && pg::launch_update(st, tab, c->d_row_tiles, n_rows, stream) == cudaSuccess;
            }
            c->launches += 4;
            c->step += 1;
        }
        c->y_valid = false;
        if (!ok) {
            cudaGetLastError();
            return PG_ERR_CUDA;
        }
        if (G) {
            rc = gradient_only_pass(c, stream, c->d_row_tiles, n_rows, c->normal_param_bytes, G, eta);
            if (rc != PG_OK) return rc;
        }
        c->round += 1;
        return PG_OK;
    }
    if (c->half_step) {
        // `power_steps` iterations of Algorithm 2.  Odd: X q-hat -> p; its update stays
        // pending and is applied by the even iteration's transposed sweep.  Even:
        // X^T p-hat -> q; its update is fused with the next odd iteration's X q-hat.
        DevState st = c->st;
        st.Ph = c->ph_buf[0];
        for (int it = 0; it < c->power_steps && ok; ++it) {
            c->iteration += 1;
            if (c->iteration % 2 == 1) {
                if (!c->y_valid) {
                    Timed t(c, PG_KERNEL_FORWARD, stream, c->normal_param_bytes);
                    ok = ok && pg::launch_forward(st, tab, c->d_row_tiles, n_rows, stream) == cudaSuccess;
                    c->launches += 1;
                }
                {
                    Timed t(c, PG_KERNEL_EDGE_LEFT, stream, 0.0);
                    ok = ok && pg::launch_edge_odd(st, tab, c->lay.max_edges, stream) == cudaSuccess;
                }
                c->launches += 1;
                c->half_pending = true;
                c->y_valid = false;
            } else {
                if (c->half_pending) {
                    Timed t(c, PG_KERNEL_TRANSPOSED, stream, 2.0 * c->normal_param_bytes);
                    ok = ok && pg::launch_transposed_update(st, tab, c->d_col_tiles, n_cols, stream) == cudaSuccess;
                } else {
                    Timed t(c, PG_KERNEL_TRANSPOSED, stream, c->normal_param_bytes);
                    ok = ok && pg::launch_transposed(st, tab, c->d_col_tiles, n_cols, stream) == cudaSuccess;
                }
                c->half_pending = false;
                {
                    Timed t(c, PG_KERNEL_EDGE_RIGHT, stream, 0.0);
                    ok = ok && pg::launch_edge_right(st, tab, c->lay.max_edges, stream) == cudaSuccess;
                }
                {
                    Timed t(c, PG_KERNEL_UPDATE_FORWARD, stream, 2.0 * c->normal_param_bytes);
                    ok = ok && pg::launch_update_forward(st, tab, tab, c->d_row_tiles, n_rows, stream) == cudaSuccess;
                }
                c->launches += 3;
                c->y_valid = true;
            }
        }
        if (!ok) {
            cudaGetLastError();
            c->y_valid = false;
            return PG_ERR_CUDA;
        }
        c->round += 1;
        if (G) {
            // apply what is pending, then the gradient step in a pass of its own
            rc = flush_pending(c, stream);
            if (rc == PG_OK)
                rc = gradient_only_pass(c, stream, c->d_row_tiles, n_rows, c->normal_param_bytes, G, eta);
            c->y_valid = false;
            if (rc != PG_OK) return rc;
        }
        return PG_OK;
    }
    // Large stacks: the layers' chains of kernels go to the library's streams (see pg_ctx::chain)
    const bool chained = c->use_chains;
    cudaStream_t s3 = stream;                       // the three sweeps
    if (chained) {
        if (!c->chains_open || c->chain_origin != stream || !c->static_graph) {
            // fork: every chain waits for what the caller's stream holds now (uploads, this round's table)
            ok = cudaEventRecord(c->ev_fork, stream) == cudaSuccess;
            for (int k = 0; k <= c->n_pair_chains && ok; ++k)
                ok = cudaStreamWaitEvent(c->chain[k], c->ev_fork, 0) == cudaSuccess;
            c->chains_open = true;
            c->chain_origin = stream;
        }
        s3 = c->chain[0];
    }
    auto pair_stream = [&](int chain) { return chained ? c->chain[1 + chain] : stream; };
    if (n_rows > 0 && !c->y_valid) {
        Timed t(c, PG_KERNEL_FORWARD, s3, c->normal_param_bytes);
        ok = ok && pg::launch_forward(c->st, tab, c->d_row_tiles, n_rows, s3) == cudaSuccess;
        c->launches += 1;
    }
    for (int p = 0; p < c->power_steps && ok; ++p) {
        const int* tab_fwd = (p + 1 < c->power_steps) ? tab : tab_next;
        float* const ph_cur = c->ph_buf[c->step & 1];        // this step's P-hat
        float* const ph_prev = c->ph_buf[(c->step + 1) & 1]; // last step's (pending correction)
        if (n_rows > 0) {
            DevState st = c->st;
            st.Ph = ph_cur;
            {
                Timed t(c, PG_KERNEL_EDGE_LEFT, s3, 0.0);
                ok = ok && pg::launch_edge_left(st, tab, c->lay.max_edges, s3) == cudaSuccess;
            }
            {
                Timed t(c, PG_KERNEL_TRANSPOSED, s3, c->normal_param_bytes);
                ok = ok && pg::launch_transposed(st, tab, c->d_col_tiles, n_cols, s3) == cudaSuccess;
            }
            {
                Timed t(c, PG_KERNEL_EDGE_RIGHT, s3, 0.0);
                ok = ok && pg::launch_edge_right(st, tab, c->lay.max_edges, s3) == cudaSuccess;
            }
            {
                // the round's last update also takes the gradient step; the product for the
                // next round is formed from the rows it has just written
                const bool with_g = G && p + 1 == c->power_steps;
                st.G = with_g ? G : nullptr;
                st.eta = eta;
                Timed t(c, PG_KERNEL_UPDATE_FORWARD, s3, (with_g ? 3.0 : 2.0) * c->normal_param_bytes);
                ok = ok && pg::launch_update_forward(st, tab, tab_fwd, c->d_row_tiles, n_rows, s3) == cudaSuccess;
            }
            c->launches += 4;
        }
        if (has_pair && ok) {
            // one read of both ends of every edge: apply the correction pending from the
            // last step, form p and this step's share of D^T p; then the scalar edge step
            const int* tab_prev = tab;
            if (c->pending) ok = ensure_table(c, c->pending_key, stream, &tab_prev) == PG_OK;
            DevState st = c->st;
            st.Ph = ph_prev;
            st.PhNext = ph_cur;
            st.Qr = c->q_buf[c->step & 1];
            st.Qw = c->q_buf[(c->step + 1) & 1];
            st.raw_pending = c->pending ? 1 : 0;
            // rows with several readers: read the current copy of X, write the corrected rows to the other
            const long long copy_elems = static_cast<long long>(c->topo.n_workers) * c->lay.x_stride;
            const bool flip = c->lay.two_copies && c->pending;
            st.X = c->st.X + c->xbuf * copy_elems;
            st.Xw = flip ? c->st.X + (c->xbuf ^ 1) * copy_elems : st.X;
            const int n_chains = std::max(c->n_pair_chains, 1);
            for (int k = 0; k < n_chains && ok; ++k) {
                cudaStream_t sp = pair_stream(k);
                for (const auto& grp : c->pair_groups) {
                    if (grp.chain != k) continue;
                    // without a pending correction the sweep only reads
                    Timed t(c, PG_KERNEL_PAIR_SWEEP, sp, c->pending ? grp.bytes : 0.5 * grp.bytes);
                    if (grp.mode == 1)
                        ok = ok && pg::launch_pair_sweep(st, tab_prev, tab, c->pending, c->d_pair_tiles + grp.first,
                                                         grp.count, grp.nv, c->lay.pend_slots, sp) == cudaSuccess;
                    else if (grp.mode == 3)
                        ok = ok && pg::launch_pair_sweep_mid(st, tab_prev, tab, c->pending,
                                                             c->d_pair_tiles + grp.first, grp.count, grp.nv,
                                                             static_cast<int>(round_up(grp.slice, 4)),
                                                             c->lay.pend_slots, grp.raw, c->lay.single_owner,
                                                             grp.max_rows, sp) == cudaSuccess;
                    else
                        ok = ok && pg::launch_pair_sweep_wide(st, tab_prev, tab, c->pending,
                                                              c->d_pair_tiles + grp.first, grp.count, grp.nv, grp.slice,
                                                              c->lay.pend_slots, sp) == cudaSuccess;
                    c->launches += 1;
                }
                if (c->edge_count[k] > 0) {     // the pair edge step of this chain's layers
                    DevState se = st;
                    se.edge_tab = c->st.edge_tab + 2 * c->edge_first[k];
                    se.e_total = c->edge_count[k];
                    Timed t(c, PG_KERNEL_PAIR_EDGE, sp, 0.0);
                    ok = ok && pg::launch_pair_edge(se, tab, c->lay.max_edges, sp) == cudaSuccess;
                    c->launches += 1;
                }
            }
            if (flip) c->xbuf ^= 1;
            c->pending = true;
            c->pending_key = c->static_graph ? 0 : c->round;
        }
        c->step += 1;
    }
    if (chained)   // join even after a failed launch, so the caller's stream stays ordered after the chains
        for (int k = 0; k <= c->n_pair_chains; ++k)
            ok = (cudaEventRecord(c->ev_join[k], c->chain[k]) == cudaSuccess &&
                  cudaStreamWaitEvent(stream, c->ev_join[k], 0) == cudaSuccess) && ok;
    if (!ok) {
        cudaGetLastError();
        c->y_valid = false;
        c->chains_open = false;
        return PG_ERR_CUDA;
    }
    c->y_valid = true;
    c->round += 1;
    // pair-sweep layers: the pending correction and the gradient step in one pass
    if (G && has_pair) return flush_pending(c, stream, G, eta);
    return PG_OK;
}

int pg_round(pg_ctx* c, void* stream) { return round_impl(c, stream, nullptr, 0.0f); }

int pg_round_sgd(pg_ctx* c, const float* G_dev, float eta, void* stream) {
    if (!c || !G_dev || !std::isfinite(eta)) return PG_ERR_INVALID;
    if (reinterpret_cast<uintptr_t>(G_dev) % 16 != 0) return PG_ERR_INVALID;
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, G_dev) != cudaSuccess || attr.type != cudaMemoryTypeDevice ||
        attr.device != c->device) {
        cudaGetLastError();
        return PG_ERR_INVALID;
    }
    return round_impl(c, stream, G_dev, eta);
}

int pg_stack_elems(pg_ctx* c, int64_t* elems_out) {
    if (!c || !elems_out) return PG_ERR_INVALID;
    *elems_out = static_cast<int64_t>(c->topo.n_workers) * c->lay.x_stride;
    return PG_OK;
}

int pg_stack_offset(pg_ctx* c, int32_t worker, int32_t layer, int64_t* offset_out, int64_t* ld_out) {
    const int rc = check_worker_layer(c, worker, layer);
    if (rc != PG_OK || !offset_out || !ld_out) return PG_ERR_INVALID;
    *offset_out = static_cast<int64_t>(worker) * c->lay.x_stride + c->lay.layers[layer].x_off;
    *ld_out = c->lay.layers[layer].ld;
    return PG_OK;
}

int pg_set_half_step(pg_ctx* c, int32_t on) {
    if (!c) return PG_ERR_INVALID;
    if (c->round != 0 || c->pending || c->y_valid) return PG_ERR_STATE;
    if (on && (c->rank != 1 || !c->static_graph || c->random_proj)) return PG_ERR_INVALID;
    // the pair sweep has no half-step form: every layer goes to the three-sweep path
    if (on && (!bind_device(c) || !leave_pair_mode(c))) return PG_ERR_CUDA;
    c->half_step = on != 0;
    c->iteration = 0;
    return PG_OK;
}

int pg_set_random_projection(pg_ctx* c, int32_t mode) {
    if (!c || mode < 0 || mode > 2) return PG_ERR_INVALID;
    if (c->round != 0 || c->pending || c->y_valid || c->half_step) return PG_ERR_STATE;
    // the pair sweep has no random-projection form: every layer goes to the three-sweep path
    if (mode != 0 && !c->static_graph) return PG_ERR_INVALID;
    if (mode != 0 && (!bind_device(c) || !leave_pair_mode(c))) return PG_ERR_CUDA;
    c->random_proj = mode;
    return PG_OK;
}

// Steady state of a static graph: the table is on the device, the pair sweep has a correction
// pending and the three sweeps have their forward product cached, so every round enqueues the
// same kernels with the same arguments up to the parity of the double buffers.
static bool rounds_are_periodic(const pg_ctx* c) {
    return c->static_graph && c->tab_used[0] && c->tab_round[0] == 0 &&
           (c->lay.n_pair_tiles == 0 || c->pending) && (c->lay.n_row_tiles == 0 || c->y_valid);
}

// Capture two rounds (an even number of power steps: the buffer parities return) on the
// library's own stream and instantiate them.  Nothing runs; the host state is put back.
static void capture_two_rounds(pg_ctx* c, int key) {
    const int64_t round = c->round, step = c->step, launches = c->launches, pending_key = c->pending_key;
    const int xbuf = c->xbuf;
    const bool pending = c->pending, y_valid = c->y_valid;
    c->chains_open = false;              // the captured rounds fork the chains from the capturing stream
    if (cudaStreamBeginCapture(c->cap, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        c->loop_failed = true;
        return;
    }
    // plain launches inside the graph: replay has no launch gaps to hide, and dependent
    // launches measured equal or slower there
    const int dep_launch = c->st.dep_launch;
    c->st.dep_launch = 0;
    int rc = round_impl(c, c->cap, nullptr, 0.0f);
    if (rc == PG_OK) rc = round_impl(c, c->cap, nullptr, 0.0f);
    c->st.dep_launch = dep_launch;
    cudaGraph_t graph = nullptr;
    const cudaError_t end = cudaStreamEndCapture(c->cap, &graph);
    c->loop_launches = c->launches - launches;
    c->round = round; c->step = step; c->launches = launches; c->pending_key = pending_key;
    c->xbuf = xbuf; c->pending = pending; c->y_valid = y_valid;
    c->chains_open = false;
    if (c->loop_exec) {
        cudaGraphExecDestroy(c->loop_exec);
        c->loop_exec = nullptr;
    }
    if (rc != PG_OK || end != cudaSuccess || !graph ||
        cudaGraphInstantiate(&c->loop_exec, graph, 0) != cudaSuccess) {
        cudaGetLastError();
        c->loop_exec = nullptr;
        c->loop_failed = true;
    }
    if (graph) cudaGraphDestroy(graph);
    c->loop_key = key;
}

int pg_rounds(pg_ctx* c, int32_t n_rounds, void* stream_v) {
    if (!c || n_rounds < 0) return PG_ERR_INVALID;
    if (c->failed) return PG_ERR_STATE;
    if (n_rounds == 0) return PG_OK;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    // One cooperative launch when the graph is static, no layer uses the pair sweep and the
    // whole stack stays in L2; otherwise the rounds are enqueued one by one.
    const double x_bytes = c->normal_param_bytes;
    const bool persistent = c->static_graph && !c->half_step && !c->random_proj && c->lay.n_pair_tiles == 0 && c->coop_ok &&
                            x_bytes <= 64.0 * 1024 * 1024 && !c->timing;
    if (!persistent) {
        int done = 0;
        // launch-bound loops on a static graph: replay a captured pair of rounds
        bool replay = c->static_graph && !c->half_step && !c->random_proj && !c->timing && !c->loop_failed &&
                      n_rounds >= 4;
        if (replay) {
            cudaStreamCaptureStatus busy = cudaStreamCaptureStatusNone;
            if (cudaStreamIsCapturing(stream, &busy) != cudaSuccess || busy != cudaStreamCaptureStatusNone) {
                cudaGetLastError();
                replay = false;      // the caller is capturing: enqueue plain launches into their graph
            }
        }
        if (replay) {
            while (done < n_rounds && !rounds_are_periodic(c)) {
                const int rc = pg_round(c, stream_v);
                if (rc != PG_OK) return rc;
                ++done;
            }
            const int pairs_left = (n_rounds - done) / 2;
            if (pairs_left > 0) {
                const int key = static_cast<int>(c->step & 1) | (c->xbuf << 1);
                if (!c->loop_exec || c->loop_key != key) capture_two_rounds(c, key);
                if (c->loop_exec) {
                    for (int r = 0; r < pairs_left; ++r)
                        if (cudaGraphLaunch(c->loop_exec, stream) != cudaSuccess) {
                            cudaGetLastError();
                            return PG_ERR_CUDA;
                        }
                    c->chains_open = false;
                    c->round += 2LL * pairs_left;
                    c->step += 2LL * pairs_left * c->power_steps;
                    c->launches += c->loop_launches * pairs_left;
                    done += 2 * pairs_left;
                }
            }
        }
        for (; done < n_rounds; ++done) {
            const int rc = pg_round(c, stream_v);
            if (rc != PG_OK) return rc;
        }
        return PG_OK;
    }
    const int* tab = nullptr;
    int rc = ensure_table(c, c->round, stream, &tab);
    if (rc != PG_OK) return rc;
    DevState st = c->st;
    st.Ph = c->ph_buf[0];
    const long long steps = static_cast<long long>(n_rounds) * c->power_steps;
    if (steps > INT_MAX) return PG_ERR_INVALID;
    int* bar = c->st.status + 16;
    if (pg::launch_persistent(st, tab, c->d_row_tiles, static_cast<int>(c->lay.n_row_tiles), c->d_col_tiles,
                              static_cast<int>(c->lay.n_col_tiles), static_cast<int>(steps), !c->y_valid, bar,
                              stream) != cudaSuccess) {
        cudaGetLastError();
        c->y_valid = false;
        return PG_ERR_CUDA;
    }
    c->launches += 1;
    c->y_valid = true;
    c->step += steps;
    c->round += n_rounds;
    return PG_OK;
}

int pg_selftest_barrier_timeout(pg_ctx* c, void* stream_v) {
    if (!c) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    if (pg::launch_barrier_timeout_probe(c->st.status + 16, c->st.status, stream) != cudaSuccess) {
        cudaGetLastError();
        return PG_ERR_CUDA;
    }
    c->launches += 1;
    return device_status(c, stream);
}

int pg_selftest_bounds_check(pg_ctx* c, void* stream_v) {
    if (!c) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    if (pg::launch_bounds_probe(c->st, stream) != cudaSuccess) {
        cudaGetLastError();
        return PG_ERR_CUDA;
    }
    c->launches += 1;
    return device_status(c, stream);
}

int pg_max_edges(pg_ctx* c, int32_t* max_edges_out) {
    if (!c || !max_edges_out) return PG_ERR_INVALID;
    *max_edges_out = c->lay.max_edges;
    return PG_OK;
}

int pg_get_schedule(pg_ctx* c, int64_t round, int32_t* edges_out, float* w_out, int32_t* n_edges_out) {
    if (!c || !edges_out || !n_edges_out || round < 0) return PG_ERR_INVALID;
    std::vector<Edge> edges;
    std::vector<float> w;
    if (!pg::build_edges(c->topo, c->seed, round, edges)) return PG_ERR_INVALID;
    if (!pg::edge_weights(c->topo, edges, w)) return PG_ERR_INVALID;
    for (size_t e = 0; e < edges.size(); ++e) {
        edges_out[2 * e] = edges[e].i;
        edges_out[2 * e + 1] = edges[e].j;
        if (w_out) w_out[e] = w[e];
    }
    *n_edges_out = static_cast<int32_t>(edges.size());
    return PG_OK;
}

int pg_read_q(pg_ctx* c, int32_t i, int32_t j, int32_t layer, float* host_dst, void* stream_v) {
    if (!c || !host_dst || layer < 0 || layer >= c->n_layers) return PG_ERR_INVALID;
    const int64_t pair = c->pairs.of(i, j);
    if (pair < 0) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const LayerGeom& g = c->lay.layers[layer];
    const float* src = (g.pair_mode ? c->q_buf[c->step & 1] : c->st.Q) + pair * c->st.q_stride + g.q_off;
    if (cudaMemcpy2DAsync(host_dst, sizeof(float) * g.m, src, sizeof(float) * g.ld, sizeof(float) * g.m,
                          c->rank, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return PG_ERR_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? PG_OK : PG_ERR_CUDA;
}

int pg_write_q(pg_ctx* c, int32_t i, int32_t j, int32_t layer, const float* host_src, void* stream_v) {
    if (!c || !host_src || layer < 0 || layer >= c->n_layers) return PG_ERR_INVALID;
    const int64_t pair = c->pairs.of(i, j);
    if (pair < 0) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const LayerGeom& g = c->lay.layers[layer];
    float* dst = (g.pair_mode ? c->q_buf[c->step & 1] : c->st.Q) + pair * c->st.q_stride + g.q_off;
    const int frc = flush_pending(c, stream);     // the pending correction uses the stored vectors
    if (frc != PG_OK) return frc;
    c->y_valid = false;
    if (cudaMemcpy2DAsync(dst, sizeof(float) * g.ld, host_src, sizeof(float) * g.m, sizeof(float) * g.m,
                          c->rank, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return PG_ERR_CUDA;
    {
        DevState st = c->st;
        st.Qr = c->q_buf[c->step & 1];
        if (pg::launch_column_norms(st, c->lay.n_pairs, stream) != cudaSuccess) return PG_ERR_CUDA;
    }
    c->launches += 1;
    return cudaStreamSynchronize(stream) == cudaSuccess ? PG_OK : PG_ERR_CUDA;
}

int pg_build_schedule(const pg_topology* topo, const float* W_host, uint64_t seed, int64_t round,
                      int32_t* edges_out, float* w_out, int32_t capacity, int32_t* n_edges_out) {
    if (!edges_out || !n_edges_out || round < 0) return PG_ERR_INVALID;
    pg::Topology t;
    const int rc = make_topology(topo, W_host, t);
    if (rc != PG_OK) return rc;
    std::vector<Edge> edges;
    std::vector<float> w;
    if (!pg::build_edges(t, seed, round, edges)) return PG_ERR_INVALID;
    if (!pg::edge_weights(t, edges, w)) return PG_ERR_INVALID;
    if (static_cast<int64_t>(edges.size()) > capacity) return PG_ERR_INVALID;
    for (size_t e = 0; e < edges.size(); ++e) {
        edges_out[2 * e] = edges[e].i;
        edges_out[2 * e + 1] = edges[e].j;
        if (w_out) w_out[e] = w[e];
    }
    *n_edges_out = static_cast<int32_t>(edges.size());
    return PG_OK;
}

int pg_initial_vector(uint64_t seed, int32_t i, int32_t j, int32_t layer, int32_t col, int32_t m,
                      float* host_dst) {
    if (!host_dst || i < 0 || j <= i || layer < 0 || col < 0 || col >= 256 || m < 1) return PG_ERR_INVALID;
    pg::init_q_column(seed, i, j, layer, col, m, host_dst);
    return PG_OK;
}

int pg_comm_floats(const pg_layer_shape* shapes, int32_t n_layers, int32_t rank, int64_t first_iteration,
                   int64_t iterations, int64_t* floats_out, int64_t* dense_out) {
    if (!shapes || n_layers < 1 || rank < 1 || first_iteration < 1 || iterations < 0 || !floats_out)
        return PG_ERR_INVALID;
    int64_t rows = 0, cols = 0, dense = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (shapes[l].rows < 1 || shapes[l].cols < 1) return PG_ERR_INVALID;
        rows += shapes[l].rows;
        cols += shapes[l].cols;
        dense += static_cast<int64_t>(shapes[l].rows) * shapes[l].cols;
    }
    // odd counters among first_iteration .. first_iteration + iterations - 1
    const int64_t last = first_iteration + iterations - 1;
    const int64_t n_odd = (last + 1) / 2 - first_iteration / 2;
    const int64_t n_even = iterations - n_odd;
    *floats_out = rank * (n_odd * rows + n_even * cols);
    if (dense_out) *dense_out = dense;
    return PG_OK;
}

int pg_comm_floats_round(pg_ctx* c, int64_t round, int64_t* floats_out, int64_t* dense_out) {
    if (!c || round < 0 || !floats_out) return PG_ERR_INVALID;
    std::vector<Edge> edges;
    if (!pg::build_edges(c->topo, c->seed, round, edges)) return PG_ERR_INVALID;
    std::vector<pg_layer_shape> shapes(c->n_layers);
    for (int l = 0; l < c->n_layers; ++l) shapes[l] = pg_layer_shape{c->lay.layers[l].n, c->lay.layers[l].m};
    int64_t per_end = 0, dense = 0;
    int rc;
    if (c->random_proj) {
        // one product per step: an "odd" iteration for right projections, an "even" one for left
        rc = pg_comm_floats(shapes.data(), c->n_layers, c->rank, c->random_proj == 1 ? 1 : 2, 1, &per_end, &dense);
        per_end *= c->power_steps;
    } else if (c->half_step) {
        rc = pg_comm_floats(shapes.data(), c->n_layers, c->rank, round * c->power_steps + 1, c->power_steps,
                            &per_end, &dense);
    } else {
        rc = pg_comm_floats(shapes.data(), c->n_layers, c->rank, 1, 2LL * c->power_steps, &per_end, &dense);
    }
    if (rc != PG_OK) return rc;
    const int64_t ends = 2 * static_cast<int64_t>(edges.size());
    *floats_out = ends * per_end;
    if (dense_out) *dense_out = ends * dense;
    return PG_OK;
}

int pg_get_round(pg_ctx* c, int64_t* round_out) {
    if (!c || !round_out) return PG_ERR_INVALID;
    *round_out = c->round;
    return PG_OK;
}

int pg_set_round(pg_ctx* c, int64_t round, void* stream_v) {
    if (!c || round < 0) return PG_ERR_INVALID;
    if (c->failed) return PG_ERR_STATE;
    c->chains_open = false;
    if (c->pending || c->half_pending) {
        // the pending correction belongs to the old round's graph: apply it first, on the
        // stream the rounds were enqueued on
        if (!bind_device(c)) return PG_ERR_CUDA;
        const int rc = flush_pending(c, static_cast<cudaStream_t>(stream_v));
        if (rc != PG_OK) return rc;
    }
    c->round = round;
    c->y_valid = false;
    return PG_OK;
}

int pg_round_bytes(pg_ctx* c, double* bytes_out, double* pair_fraction_out) {
    if (!c || !bytes_out) return PG_ERR_INVALID;
    // normal_param_bytes / pair_param_bytes: 4 B x the parameters on either path
    const double per_step = c->half_step ? 2.0 * c->normal_param_bytes
                                         : 3.0 * c->normal_param_bytes + 2.0 * c->pair_param_bytes;
    *bytes_out = per_step * c->power_steps;
    const double all = c->normal_param_bytes + c->pair_param_bytes;
    if (pair_fraction_out) *pair_fraction_out = all > 0.0 ? c->pair_param_bytes / all : 0.0;
    return PG_OK;
}

int pg_timing_enable(pg_ctx* c, int32_t on) {
    if (!c) return PG_ERR_INVALID;
    c->timing = on != 0;
    return PG_OK;
}

int pg_timing_read(pg_ctx* c, double* ms_out, int64_t* launches_out, double* bytes_out) {
    if (!c || !ms_out || !launches_out || !bytes_out) return PG_ERR_INVALID;
    if (!bind_device(c)) return PG_ERR_CUDA;
    for (int k = 0; k < PG_KERNEL_KINDS; ++k) {
        ms_out[k] = 0.0;
        launches_out[k] = 0;
        bytes_out[k] = 0.0;
    }
    bool ok = true;
    for (auto& sp : c->spans) {
        float ms = 0.0f;
        ok = ok && cudaEventSynchronize(sp.b) == cudaSuccess && cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess;
        if (ok) {
            ms_out[sp.kind] += ms;
            launches_out[sp.kind] += 1;
            bytes_out[sp.kind] += sp.bytes;
        }
        cudaEventDestroy(sp.a);
        cudaEventDestroy(sp.b);
    }
    c->spans.clear();
    if (!ok) cudaGetLastError();
    return ok ? PG_OK : PG_ERR_CUDA;
}

int pg_kernel_launches(pg_ctx* c, int64_t* count_out) {
    if (!c || !count_out) return PG_ERR_INVALID;
    *count_out = c->launches;
    return PG_OK;
}

const char* pg_status_string(int status) {
    switch (status) {
        case PG_OK: return "ok";
        case PG_ERR_INVALID: return "invalid argument, topology or mixing matrix";
        case PG_ERR_WORKSPACE: return "workspace missing, misaligned, too small or not device memory";
        case PG_ERR_CUDA: return "a CUDA runtime call failed";
        case PG_ERR_STATE: return "call not allowed in this state";
        case PG_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case PG_ERR_NUMERIC: return "a norm was not finite";
        case PG_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the no-allocation entry point";
        case PG_ERR_BOUNDS: return "a kernel of the bounds-checked build computed an address outside its section";
        default: return "unknown status";
    }
}

}  // extern "C"
