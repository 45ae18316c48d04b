// Device-side data layout of the PowerGossip library and the launchers of its
// kernels.  Everything lives in the caller's single workspace; offsets are in
// floats from the start of a section.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

namespace pg {

constexpr int kMaxSlots = 8;   // vectors per worker per sweep: degree * rank
constexpr int kMaxRank = 4;

// Tiling limits.  The host picks the tile of every layer inside these limits so
// that each sweep has a few thousand CTAs (several waves on 148 SMs) whatever
// the size of the stack.
constexpr int kRowTileRowsMax = 64;    // rows of X per CTA in the row-oriented sweeps (32 or 64)
constexpr int kRowTileColsMax = 2048;  // most columns one CTA reduces over (multiple of 128)
constexpr int kColTileRowsMax = 256;   // rows of X per CTA in the transposed sweep (64, 128 or 256)
constexpr int kColTileCols = 256;      // columns per CTA in the transposed sweep (64 threads x float4)
constexpr int kPairTileRows = 512;     // rows of both matrices per CTA in the pair sweep
constexpr int kPairMaxLd = 1024;       // widest row a warp of the pair sweep keeps in registers
constexpr int kPairMidMaxLd = 8192;    // widest row one CTA of the pair sweep keeps in registers (8 float4 per thread)
constexpr int kPairMid2MaxLd = 5120;   // widest row of the rank-2 form of that sweep (5 float4 per thread)
constexpr int kPairCluster = 8;        // CTAs that share a row of a wider layer (thread-block cluster)
constexpr int kPairWideRows = 32;      // rows per cluster tile of a wider layer when residency is unknown
constexpr int kPairWideMaxTiles = 32;  // most row tiles per (edge, wide layer); sizes the partial-sum buffer
constexpr int kPairWideStep = 1;       // rows a cluster handles between two exchanges
constexpr int kPairWideMinBlocks = 3;  // resident CTAs per SM the cluster sweep is compiled for
constexpr int kPairWideMaxLd = 8 * 256 * 4 * kPairCluster;  // widest row the cluster variant covers
constexpr int kEdgeChunks = 32;        // CTAs that share the pair edge step of one (edge, layer)
constexpr int kSpPerTile = 16;         // doubles a pair-sweep tile leaves for the pair edge step, see DevState::Sp
constexpr int kMaxTerms = 3;           // edges whose corrections can be pending on the difference of an edge (degree 2)

// Geometry of one layer (same for every worker).
struct LayerGeom {
    int n, m;          // rows, cols of X
    int ld;            // leading dimension of X in floats: m rounded up to 4
    int npad;          // n rounded up to 4 (length of n-vectors)
    int f_rows;        // rows per tile of the row-oriented sweeps
    int t_rows;        // rows per tile of the transposed sweep
    int f_rtiles;      // row tiles of the row-oriented sweeps
    int f_csplit;      // column chunks (partial sums of X q)
    int f_chunk;       // columns per chunk (multiple of 128)
    int t_rtiles;      // row tiles of the transposed sweep (partial sums of X^T p)
    int t_ctiles;      // column tiles of the transposed sweep
    long long x_off;   // X of this layer inside a worker's parameter block
    long long q_off;   // Q of this layer inside a pair's block      (rank x ld)
    long long y_off;   // forward partials inside a worker's block   (slots x f_csplit x npad)
    long long ph_off;  // P-hat inside an edge's block               (rank x npad)
    long long z_off;   // transposed partials inside a worker's block (slots x t_rtiles x ld)
    // pair sweep (rank 1: a matching or a static graph of degree <= 2; rank 2: mode 3 on such a static graph)
    int pair_mode;     // 0: three sweeps; pair sweep with a row per 1: warp, 2: cluster, 3: CTA
    int p_rows;        // rows per tile of the pair sweep
    int p_rtiles;      // row tiles of the pair sweep
    int p_slice;       // mode 2: columns per CTA of the cluster (multiple of 4)
    long long up_off;  // partial sums of D^T p inside an edge's block (p_rtiles x rank x ld)
    long long sp_off;  // per-tile scalars for the pair edge step (p_rtiles x kSpPerTile doubles)
    int e_chunks;      // CTAs that share the pair edge step of one edge on this layer (1..kEdgeChunks)
    int raw;           // pair sweep forms D from the rows as stored and leaves the pending terms to vector
                       // algebra (graphs where a row has two readers), see raw_terms
};

// One unit of work of a sweep: a tile of one worker's layer.
struct Tile {
    int worker;
    int layer;
    int rtile;
    int ctile;
};

// Table of one round, in device memory.  Arrays follow the header; their
// offsets (in ints from the start of the table) are in TabLayout.
struct TabLayout {
    int max_edges, n_workers, max_degree;
    int off_n_edges;     // 1 int
    int off_edge_i;      // max_edges ints
    int off_edge_j;      // max_edges ints
    int off_pair;        // max_edges ints (index into per-pair state; fits int)
    int off_w;           // max_edges floats
    int off_slot_i;      // max_edges ints: slot of the edge at its smaller end
    int off_slot_j;      // max_edges ints: slot at its larger end
    int off_degree;      // n_workers ints
    int off_slot_edge;   // n_workers * max_degree ints
    int off_slot_coef;   // n_workers * max_degree floats: sign * W
    int off_own;         // max_edges ints: bit 0 / bit 1 set if the edge's CTAs write the corrected rows of
                         // its smaller / larger end in the pair sweep (every worker has exactly one such edge)
    int total_ints;
};

// Sections of the workspace, for the bounds-checked build (-DPG_BOUNDS_CHECK): every kernel checks the
// address ranges it is about to touch against the section they belong to; a range outside raises
// the bounds bit of the status word and the access is skipped (nothing traps).
enum : int { kSecX, kSecQ, kSecQinv, kSecQn2, kSecPn, kSecY, kSecPh, kSecUp, kSecSp, kSecZ, kSecLive, kSecTabs,
             kSecTiles, kSecLayers, kSecCount };

// Pointers into the workspace (device) plus sizes; passed to kernels by value.
// Kernel families for DevState::dep_launch.
enum : int { kDepSweep = 1, kDepPairRow = 2, kDepPairMid = 4, kDepPairWide = 8, kDepPairEdge = 16 };

struct DevState {
    float* X;            // [worker][x_stride]
    float* Xw;           // where corrected rows are written: X itself, or the second copy of the stack
                         // when a row has two readers in one sweep (pair sweep on graphs of degree 2)
    const float* G;      // null, or the caller's gradients laid out like X: updates also subtract eta * G
    float eta;
    float* Q;            // [pair][q_stride]     raw right factors (three-sweep layers; update sweeps)
    float* Qr;           // pair-sweep layers: the stored vectors this step reads (q and the pending q') ...
    float* Qw;           // ... and where the pair edge step writes the new ones.  Qr == Qw == Q unless rows
                         // have several readers; there the two copies of Q swap roles every step, because an
                         // edge's step still needs its neighbours' previous vectors while they write new ones
    int raw_pending;     // pair edge step: the sweep ran on rows with corrections pending (their terms apply)
    float* Qinv;         // [pair][layer][rank]  1 / column norm (0 for a zero column)
    double* Qn2;         // [pair][layer][rank][kEdgeChunks]  pair sweep layers: shares of ||Q_k||^2
    float* Y;            // [worker][y_stride]   partial sums of X q
    float* Ph;           // [edge][ph_stride]    orthonormal left factors of this step
    float* Z;            // [worker][z_stride]   partial sums of X^T p
    float* PhNext;       // same shape as Ph: where the pair sweep writes this step's p
    float* Up;           // [edge][up_stride]    pair sweep: partial sums of D^T p
    double* Sp;          // [edge][sp_stride]    pair sweep, per tile kSpPerTile doubles: [0] ||p||^2 (rank 2:
                         // [0..2] P^T P), [4 + k] sum_r p_r p-hat_k[r] for pending term k (rank 2: [4 + 2k + c])
    float* Pn;           // [edge][layer]  half-step mode: ||p|| of the last odd iteration
    int dep_launch;      // host only: kernel families (kDep*) launched with programmatic stream serialisation
    int half_odd;        // half-step mode: the update being applied is an odd iteration's,
                         // p q-hat^T = (||p|| / ||q||) p-hat q^T: scale the coefficients accordingly
    int* live;           // [edge][layer][rank]  1 if the column took part in this step
    int* status;         // device status word (bit n set = error code n was raised)
    const LayerGeom* layers;
    const int* edge_tab; // [e_total][2]  (layer, chunk) of every CTA of the pair edge step of one edge
    int e_total;
    long long x_stride, q_stride, y_stride, ph_stride, z_stride, up_stride, sp_stride;
    int n_layers, rank, n_workers, max_degree;
    int f_chunk_max, f_rows_max;   // widest column chunk and tallest tile of the row-oriented sweeps over all layers
    TabLayout tab;
#ifdef PG_BOUNDS_CHECK
    const char* sec_lo[kSecCount];   // first byte and one past the last byte of every workspace section
    const char* sec_hi[kSecCount];   // (kernel parameters: only the checked build carries them)
#endif
};

// Launchers (all asynchronous on `stream`; return the cudaError of the launch).
// `slots` = max_degree * rank of the context.
cudaError_t launch_forward(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                           cudaStream_t stream);
cudaError_t launch_edge_left(const DevState& st, const int* tab, int max_edges, cudaStream_t stream);
cudaError_t launch_transposed(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                              cudaStream_t stream);
cudaError_t launch_edge_right(const DevState& st, const int* tab, int max_edges, cudaStream_t stream);
cudaError_t launch_update_forward(const DevState& st, const int* tab_update, const int* tab_forward,
                                  const Tile* tiles, int n_tiles, cudaStream_t stream);
// half-step mode
cudaError_t launch_edge_odd(const DevState& st, const int* tab, int max_edges, cudaStream_t stream);
cudaError_t launch_transposed_update(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                                     cudaStream_t stream);
// random-projection compressors: fresh orthonormal directions per (edge, layer) into Q
// (side 0, length cols) or P-hat (side 1, length rows); raw difference of the forward products
cudaError_t launch_random_directions(const DevState& st, const int* tab, int max_edges, unsigned key_lo,
                                     unsigned key_hi, int side, cudaStream_t stream);
cudaError_t launch_edge_raw(const DevState& st, const int* tab, int max_edges, cudaStream_t stream);
cudaError_t launch_update(const DevState& st, const int* tab_update, const Tile* tiles, int n_tiles,
                          cudaStream_t stream);
// pend_slots: most corrections pending at a worker (its degree)
cudaError_t launch_pair_sweep(const DevState& st, const int* tab_prev, const int* tab_cur, bool apply_pending,
                              const Tile* tiles, int n_tiles, int nv, int pend_slots, cudaStream_t stream);
cudaError_t launch_pair_sweep_wide(const DevState& st, const int* tab_prev, const int* tab_cur,
                                   bool apply_pending, const Tile* tiles, int n_tiles, int nv, int slice,
                                   int pend_slots, cudaStream_t stream);
// `tiles`: tiles of layers whose rows one CTA holds (nv float4 per thread, rows of at most ld_pad floats)
// raw / single_owner: see LayerGeom::raw and TabLayout::off_own (single_owner: no edge writes both of its
// ends); max_rows: tallest tile in `tiles`
cudaError_t launch_pair_sweep_mid(const DevState& st, const int* tab_prev, const int* tab_cur,
                                  bool apply_pending, const Tile* tiles, int n_tiles, int nv, int ld_pad,
                                  int pend_slots, bool raw, bool single_owner, int max_rows, cudaStream_t stream);
// Clusters of the wide pair sweep that can be resident at once (0 if unknown).
int pair_wide_resident_clusters(int nv, int slice, int pend_slots);
cudaError_t launch_pair_edge(const DevState& st, const int* tab, int max_edges, cudaStream_t stream);
// dense rows x cols at `src` (device) -> rows of leading dimension ld at `dst`
cudaError_t launch_unpack_rows(float* dst, long long ld, const float* src, int rows, int cols, cudaStream_t stream);
// One cooperative launch for `n_steps` power steps of a static graph (small stacks).
cudaError_t launch_persistent(const DevState& st, const int* tab, const Tile* row_tiles, int n_rows,
                              const Tile* col_tiles, int n_cols, int n_steps, bool forward_first, int* bar,
                              cudaStream_t stream);
cudaError_t launch_barrier_timeout_probe(int* bar, int* status, cudaStream_t stream);
cudaError_t launch_bounds_probe(const DevState& st, cudaStream_t stream);
cudaError_t launch_column_norms(const DevState& st, long long n_pairs, cudaStream_t stream);

}  // namespace pg
