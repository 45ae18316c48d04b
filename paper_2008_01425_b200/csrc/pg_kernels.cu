// CUDA kernels of the PowerGossip power step (sm_100a).
//
// One power step of every edge (i<j) and layer (Algorithm 2 of the paper, two
// consecutive iterations, followed by the gossip update of Eq. 2):
//   row sweep    Y[w][v]  = X_w Qh_v          for all vectors v of worker w's edges
//   edge (left)  P = Y[i] - Y[j], orthonormalise -> Ph          (tiny, fp64)
//   col sweep    Z[w][v]  = X_w^T Ph_v
//   edge (right) Q' = Z[i] - Z[j]; Q <- Q'; 1/||Q'||            (tiny, fp64)
//   row sweep    X_w -= sum_v coef_v Ph_v Q'_v^T, and in the same pass the next
//                step's Y = X_w Qh_next
// The three sweeps stream X with 16-byte loads; each is bound by HBM bandwidth.
// Sums over column chunks / row tiles are written as partials and added in a
// fixed order by the edge kernels, so results are bit-reproducible.
#include <cooperative_groups.h>

#include <algorithm>
#include <cstdlib>

#include "pg_device.h"

namespace pg {
namespace {

constexpr int kStatusNumeric = 6;  // PG_ERR_NUMERIC
constexpr int kStatusTimeout = 5;  // PG_ERR_TIMEOUT
[[maybe_unused]] constexpr int kStatusBounds = 8;   // PG_ERR_BOUNDS (raised by the checked build only)

// Bounds-checked build (-DPG_BOUNDS_CHECK; the stand-in for a memory checker): PG_OOB(st, section,
// pointer, count) is true, and raises the bounds bit of the status word, if the `count` elements at
// `pointer` do not lie inside that section of the workspace; the caller then skips the work that
// would touch them.  In the normal build it is the constant false and costs nothing.
#ifdef PG_BOUNDS_CHECK
__device__ __noinline__ bool pg_out_of_bounds(const DevState& st, int sec, const void* p, long long bytes) {
    const char* a = static_cast<const char*>(p);
    if (bytes <= 0 || (a >= st.sec_lo[sec] && a + bytes <= st.sec_hi[sec])) return false;
    atomicOr(st.status, 1 << kStatusBounds);
    return true;
}
#define PG_OOB(st, sec, ptr, count) pg_out_of_bounds(st, sec, ptr, (long long)(count) * (long long)sizeof(*(ptr)))
#else
#define PG_OOB(st, sec, ptr, count) ((void)sizeof(ptr), (void)sizeof(count), false)   // names its operands, evaluates nothing
#endif
constexpr long long kBarrierSpinLimit = 1LL << 23;   // polls before a grid barrier gives up (a few seconds)

// Rows a warp of the row sweep works on at once, per number of vectors S.
constexpr int kRowsPerWarp1 = 4, kRowsPerWarp2 = 4, kRowsPerWarp4 = 2, kRowsPerWarp8 = 2;
// Resident CTAs per SM the row sweep is compiled for (caps its registers), per number of vectors S.
__host__ __device__ constexpr int row_min_blocks(int s) { return s <= 2 ? 4 : (s == 4 ? 3 : 2); }
// Stages of the row sweep's ring of rows in shared memory (see row_tile): 3 stages of 4 rows (128 bytes in
// flight per thread, 48 KB per CTA) or 4 stages of 2 rows (96 bytes, 32 KB).
__host__ __device__ constexpr int row_stages(int s, int rt) { return rt >= 4 ? 3 : 4; }
constexpr size_t row_ring_bytes(int s, int rt) { return (size_t)row_stages(s, rt) * rt * 256 * sizeof(float4); }

__device__ __forceinline__ float4 ld_stream(const float* p) {
    float4 v;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream(float* p, const float4& v) {
    asm volatile("st.global.L1::no_allocate.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(v.x), "f"(v.y),
                 "f"(v.z), "f"(v.w)
                 : "memory");
}

// Asynchronous 16-byte copies from global to shared memory (past L1), in groups a thread commits and
// later waits for: the bytes in flight cost no registers.  A thread reads back only what it copied
// itself, so no barrier is involved.
__device__ __forceinline__ void copy_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(smem_dst)),
                 "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void copy_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void copy_async_wait() {      // all but the N most recent groups have landed
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Programmatic dependent launch.  Every kernel of a round starts with this pair:
// the trigger lets the next kernel of the stream be scheduled while this one is
// still running (its CTAs take the slots this kernel's tail leaves free), and the
// wait returns once the previous kernel of the stream has completed and its
// writes are visible.  Nothing before the wait touches global memory.  Without
// the launch attribute both instructions do nothing.
__device__ __forceinline__ void grid_dependency_sync() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Vector / scalar loads of data that other CTAs produce.  In the multi-launch
// path a kernel boundary separates producer and consumer, so the read-only
// (L1-cached) path is fine.  COH = true is for the persistent kernel, where
// producer and consumer run in the same launch: those loads go past L1.
template <bool COH>
__device__ __forceinline__ float4 ld_vec(const float* p) {
    return COH ? __ldcg(reinterpret_cast<const float4*>(p)) : __ldg(reinterpret_cast<const float4*>(p));
}
template <bool COH>
__device__ __forceinline__ float ld_f(const float* p) {
    return COH ? __ldcg(p) : __ldg(p);
}
// Data the running kernel itself wrote earlier (never the read-only path).
template <bool COH>
__device__ __forceinline__ float ld_own(const float* p) {
    return COH ? __ldcg(p) : *p;
}
template <bool COH>
__device__ __forceinline__ int ld_i(const int* p) {
    return COH ? __ldcg(p) : *p;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of one double per thread over the whole block, returned to every thread.
__device__ double block_sum(double v, double* scratch /* >= 33 doubles of shared memory */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();  // scratch may still be read from the previous call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        double t = lane < nwarps ? scratch[lane] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// Packed fp32 arithmetic (fma.rn.f32x2: two IEEE fused multiply-adds per instruction, each
// lane rounded exactly like fmaf).  The row sweeps with four or more vectors and the two-column
// pair sweep are bound by instruction issue, and most of their instructions are these.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// x += a * v
__device__ __forceinline__ void fma4(float4& x, float a, const float4& v) {
    const unsigned long long aa = pack2(a, a);
    unpack2(fma2(aa, pack2(v.x, v.y), pack2(x.x, x.y)), x.x, x.y);
    unpack2(fma2(aa, pack2(v.z, v.w), pack2(x.z, x.w)), x.z, x.w);
}
// acc (two partial sums) += d * v, lane by lane
__device__ __forceinline__ void dot4(float2& acc, const float4& d, const float4& v) {
    unsigned long long t = pack2(acc.x, acc.y);
    t = fma2(pack2(d.x, d.y), pack2(v.x, v.y), t);
    t = fma2(pack2(d.z, d.w), pack2(v.z, v.w), t);
    unpack2(t, acc.x, acc.y);
}

// --------------------------------------------------------------------------
// Row-oriented sweep: optional rank-r update of X, optional forward product.
// A warp owns RT rows at a time; its lanes walk the columns with float4 loads.
// --------------------------------------------------------------------------
// SAME: update and forward use the same vectors (Q' of this step is the next
// step's q, as on a static graph), so each is loaded once.
template <int S>
struct RowShared {
    const float* uq[S];
    const float* up[S];
    float uc[S];
    const float* fq[S];
    float fs[S];
    int nu, nf;
};

// x += a * v and acc += x . v of one float4: packed (two lanes per instruction) where the sweep carries four or
// more vectors and is bound by instruction issue, plain where it waits on memory and the packed form's
// extra registers would spill.  The packed dot keeps even and odd column pairs in two partial sums.
template <int S>
__device__ __forceinline__ void row_axpy(float4& x, float a, const float4& v) {
    if (S >= 4) {
        fma4(x, a, v);
    } else {
        x.x = fmaf(a, v.x, x.x); x.y = fmaf(a, v.y, x.y); x.z = fmaf(a, v.z, x.z); x.w = fmaf(a, v.w, x.w);
    }
}
template <int S>
__device__ __forceinline__ void row_dot(float2& acc, const float4& x, const float4& v) {
    if (S >= 4) {
        dot4(acc, x, v);
    } else {
        acc.x = fmaf(x.x, v.x, acc.x); acc.x = fmaf(x.y, v.y, acc.x);
        acc.x = fmaf(x.z, v.z, acc.x); acc.x = fmaf(x.w, v.w, acc.x);
    }
}

// The work of one float4 column step on RT rows of a row-oriented sweep, the rows' values in x:
// the pending corrections (and the gradient step) applied and stored, then the products' partial sums.
// QS: the vectors of the tile's column chunk are staged in shared memory (uqs / fqs: one vector every
// `cmax` floats, `cs` = this step's first column within the chunk) instead of read through L1.
// FULL: every row and column step of the tile is inside it and all S vectors are worked on (those a
// worker does not have are zeros with zero coefficients), so nothing in the step is conditional.
template <int S, bool UPDATE, bool FORWARD, bool SAME, int RT, bool COH, bool GRAD, bool QS = false, bool FULL = false>
__device__ __forceinline__ void row_columns(const RowShared<S>& sh, const int nu, const int nf, float4 (&x)[RT],
                                            const float (&a)[RT][S], float2 (&acc)[RT][S], const int c,
                                            const int rb, const int r1, const float* const (&xrow)[RT],
                                            const float* __restrict__ X, float* Xw,
                                            const float* __restrict__ Gw, const float eta, const int m,
                                            const int ld, const float* uqs = nullptr, const float* fqs = nullptr,
                                            const int cmax = 0, const int cs = 0) {
    if (UPDATE && SAME) {
        // slot order: first every correction, then every product, as in the general case
        float4 q[S];
#pragma unroll
        for (int v = 0; v < S; ++v) {
            if (FULL || v < nu) {
                q[v] = QS ? *reinterpret_cast<const float4*>(uqs + v * cmax + cs) : ld_vec<COH>(sh.uq[v] + c);
#pragma unroll
                for (int t = 0; t < RT; ++t) {
                    row_axpy<S>(x[t], -a[t][v], q[v]);
                }
            }
        }
        if (GRAD) {
#pragma unroll
            for (int t = 0; t < RT; ++t) {
                float4 gv = ld_stream(Gw + (xrow[t] - X) + c);
                // columns past the matrix are padding: X keeps zeros there whatever G holds
                if (c + 1 >= m) gv.y = 0.0f;
                if (c + 2 >= m) gv.z = 0.0f;
                if (c + 3 >= m) gv.w = 0.0f;
                x[t].x = fmaf(-eta, gv.x, x[t].x); x[t].y = fmaf(-eta, gv.y, x[t].y);
                x[t].z = fmaf(-eta, gv.z, x[t].z); x[t].w = fmaf(-eta, gv.w, x[t].w);
            }
        }
#pragma unroll
        for (int t = 0; t < RT; ++t)
            if (FULL || rb + t < r1) st_stream(const_cast<float*>(xrow[t]) + c, x[t]);
#pragma unroll
        for (int v = 0; v < S; ++v) {
            if (FULL || v < nu) {
#pragma unroll
                for (int t = 0; t < RT; ++t) {
                    row_dot<S>(acc[t][v], x[t], q[v]);
                }
            }
        }
    } else if (UPDATE) {
#pragma unroll
        for (int v = 0; v < S; ++v) {
            if (FULL || v < nu) {
                const float4 q = QS ? *reinterpret_cast<const float4*>(uqs + v * cmax + cs) : ld_vec<COH>(sh.uq[v] + c);
#pragma unroll
                for (int t = 0; t < RT; ++t) {
                    row_axpy<S>(x[t], -a[t][v], q);
                }
            }
        }
        if (GRAD) {
#pragma unroll
            for (int t = 0; t < RT; ++t) {
                float4 gv = ld_stream(Gw + (xrow[t] - X) + c);
                // columns past the matrix are padding: X keeps zeros there whatever G holds
                if (c + 1 >= m) gv.y = 0.0f;
                if (c + 2 >= m) gv.z = 0.0f;
                if (c + 3 >= m) gv.w = 0.0f;
                x[t].x = fmaf(-eta, gv.x, x[t].x); x[t].y = fmaf(-eta, gv.y, x[t].y);
                x[t].z = fmaf(-eta, gv.z, x[t].z); x[t].w = fmaf(-eta, gv.w, x[t].w);
            }
        }
#pragma unroll
        for (int t = 0; t < RT; ++t)
            if (FULL || rb + t < r1) {
                // the update-only sweep may write to the other copy of the stack
                float* dst = FORWARD ? const_cast<float*>(xrow[t]) : Xw + (long long)(rb + t) * ld;
                st_stream(dst + c, x[t]);
            }
    }
    if (FORWARD && !(UPDATE && SAME)) {
#pragma unroll
        for (int v = 0; v < S; ++v) {
            if (FULL || v < nf) {
                const float4 q = QS ? *reinterpret_cast<const float4*>(fqs + v * cmax + cs) : ld_vec<COH>(sh.fq[v] + c);
#pragma unroll
                for (int t = 0; t < RT; ++t) {
                    row_dot<S>(acc[t][v], x[t], q);
                }
            }
        }
    }
}

// GRAD: the update also subtracts eta * G (Algorithm 1, line 6), G laid out like X.
// ST > 0: the rows of X arrive through a ring of ST stages in shared memory, `ring` = ST x RT x 256
// float4, each thread copying ahead (copy_async16) what it will work on itself: a warp has ST - 1
// column steps of RT rows in flight while it works on one, across the row batches of the tile.
// ST = 0: plain loads, one column step in flight (the cooperative kernel, which has no room for a ring).
// Either way a row's sum is taken over the same columns in the same order.
// FULL (ST > 0 only): the tile's rows are whole batches of 8 RT and its columns whole steps of 128.
template <int S, bool UPDATE, bool FORWARD, bool SAME, int RT, bool COH, bool GRAD = false, int ST = 0, bool FULL = false>
__device__ __forceinline__ void row_tile(const DevState& st, const int* __restrict__ tab_u,
                                         const int* __restrict__ tab_f, const Tile tile,
                                         RowShared<S>& sh, float4* ring = nullptr) {
    const LayerGeom g = st.layers[tile.layer];
    const int w = tile.worker;
    const int rank = st.rank;
    float* __restrict__ X = st.X + (long long)w * st.x_stride + g.x_off;
    float* Xw = st.Xw + (long long)w * st.x_stride + g.x_off;
    const float* __restrict__ Gw = GRAD ? st.G + (long long)w * st.x_stride + g.x_off : nullptr;
    const float eta = GRAD ? st.eta : 0.0f;

    const int r0 = tile.rtile * g.f_rows;
    const int r1 = min(g.n, r0 + g.f_rows);
    const int c0 = tile.ctile * g.f_chunk;
    const int c1 = min(g.ld, c0 + g.f_chunk);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ld = g.ld;
    // ring of rows (ST > 0): the first stages are on their way before the tables are read
    const int nc = (c1 - c0 + 127) >> 7;                       // column steps of a row batch
    const int first = r0 + warp * RT;
    const int nb = first < r1 ? (r1 - first + 8 * RT - 1) / (8 * RT) : 0;   // row batches of this warp
    const int cl = c0 + lane * 4;
    float4* const mine = ring + threadIdx.x;                   // slot (stage, t) at mine[(stage * RT + t) * 256]
    int ib = 0, ic = 0, ig = 0;      // the next step to fetch, (batch ib, column step ic), goes to stage ig
    auto issue = [&]() {
        if (ib < nb) {
            const int c = cl + (ic << 7);
            if (c < c1) {
                const int rb = first + ib * 8 * RT;
#pragma unroll
                for (int t = 0; t < RT; ++t)
                    copy_async16(mine + (ig * RT + t) * 256, X + (long long)min(rb + t, r1 - 1) * ld + c);
            }
            if (++ic == nc) { ic = 0; ++ib; }
            if (++ig == ST) ig = 0;
        }
        copy_async_commit();
    };
    if constexpr (ST > 0) {
        if (r1 > r0 && c1 > c0 &&
            PG_OOB(st, kSecX, X + (long long)r0 * ld + c0, (long long)(r1 - 1 - r0) * ld + (c1 - c0)))
            return;                  // (checked build; the same for every thread)
#pragma unroll
        for (int s = 0; s < ST - 1; ++s) issue();
    }

    if (threadIdx.x < S) {
        const int v = threadIdx.x;
        const int slot = v / rank, k = v - slot * rank;
        if (UPDATE) {
            const int deg = tab_u[st.tab.off_degree + w];
            if (slot < deg) {
                const int e = tab_u[st.tab.off_slot_edge + w * st.tab.max_degree + slot];
                const int pair = tab_u[st.tab.off_pair + e];
                sh.uq[v] = st.Q + (long long)pair * st.q_stride + g.q_off + (long long)k * g.ld;
                sh.up[v] = st.Ph + (long long)e * st.ph_stride + g.ph_off + (long long)k * g.npad;
                sh.uc[v] = __int_as_float(tab_u[st.tab.off_slot_coef + w * st.tab.max_degree + slot]);
                if (st.half_odd)   // odd iteration of Algorithm 2: the update is p q-hat^T
                    sh.uc[v] *= ld_f<COH>(&st.Pn[(long long)e * st.n_layers + tile.layer]) *
                                ld_f<COH>(&st.Qinv[((long long)pair * st.n_layers + tile.layer) * rank + k]);
            }
            if (v == 0) sh.nu = deg * rank;
        }
        if (FORWARD) {
            const int deg = tab_f[st.tab.off_degree + w];
            if (slot < deg) {
                const int e = tab_f[st.tab.off_slot_edge + w * st.tab.max_degree + slot];
                const int pair = tab_f[st.tab.off_pair + e];
                sh.fq[v] = st.Q + (long long)pair * st.q_stride + g.q_off + (long long)k * g.ld;
                sh.fs[v] = ld_f<COH>(&st.Qinv[((long long)pair * st.n_layers + tile.layer) * rank + k]);
            }
            if (v == 0) sh.nf = deg * rank;
        }
    }
    __syncthreads();
    const int nu = UPDATE ? sh.nu : 0;
    const int nf = FORWARD ? sh.nf : 0;

    if (r1 > r0 && c1 > c0) {      // (checked build) everything this tile touches; the same for every thread
        const long long span = (long long)(r1 - 1 - r0) * ld + (c1 - c0);
        bool bad = PG_OOB(st, kSecX, X + (long long)r0 * ld + c0, span);
        if (UPDATE && !FORWARD) bad = PG_OOB(st, kSecX, Xw + (long long)r0 * ld + c0, span) || bad;
        for (int v = 0; v < nu; ++v)
            bad = PG_OOB(st, kSecQ, sh.uq[v] + c0, c1 - c0) || PG_OOB(st, kSecPh, sh.up[v] + r0, r1 - r0) || bad;
        for (int v = 0; v < nf; ++v)
            bad = PG_OOB(st, kSecQ, sh.fq[v] + c0, c1 - c0) ||
                  PG_OOB(st, kSecY, st.Y + (long long)w * st.y_stride + g.y_off +
                                        ((long long)v * g.f_csplit + tile.ctile) * g.npad + r0, r1 - r0) || bad;
        if (bad) return;
    }

    if constexpr (ST > 0) {
        // the vectors of this tile's column chunk and the rows' coefficients, staged once for all warps
        const int cmax = st.f_chunk_max;
        float* const uqs = reinterpret_cast<float*>(ring + ST * RT * 256);
        float* const fqs = uqs + ((UPDATE && !SAME) || !FORWARD ? S * cmax : 0);
        float* const as = fqs + (FORWARD ? S * cmax : 0);          // [S][f_rows_max]
        const int amax = st.f_rows_max;
        const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (UPDATE) {
            for (int v = 0; v < nu; ++v)
                for (int i = threadIdx.x * 4; i < c1 - c0; i += 1024) copy_async16(uqs + v * cmax + i, sh.uq[v] + c0 + i);
            for (int i = threadIdx.x; i < nu * amax; i += 256) {
                const int v = i / amax, rr = i - v * amax;
                as[i] = r0 + rr < r1 ? sh.uc[v] * ld_f<COH>(sh.up[v] + r0 + rr) : 0.0f;
            }
            if (FULL) {      // vectors this worker does not have: zeros with zero coefficients, worked on like the rest
                for (int v = nu; v < S; ++v)
                    for (int i = threadIdx.x * 4; i < c1 - c0; i += 1024) *reinterpret_cast<float4*>(uqs + v * cmax + i) = zero4;
                for (int i = nu * amax + threadIdx.x; i < S * amax; i += 256) as[i] = 0.0f;
            }
        }
        if (FORWARD && !(UPDATE && SAME)) {
            for (int v = 0; v < nf; ++v)
                for (int i = threadIdx.x * 4; i < c1 - c0; i += 1024) copy_async16(fqs + v * cmax + i, sh.fq[v] + c0 + i);
            if (FULL)
                for (int v = nf; v < S; ++v)
                    for (int i = threadIdx.x * 4; i < c1 - c0; i += 1024) *reinterpret_cast<float4*>(fqs + v * cmax + i) = zero4;
        }
        copy_async_commit();
        copy_async_wait<0>();
        __syncthreads();
        int stage = 0;
        for (int b = 0; b < nb; ++b) {
            const int rb = first + b * 8 * RT;
            float a[RT][S];
            float2 acc[RT][S];      // even and odd column pairs apart until the row's sum
            const float* xrow[RT];
#pragma unroll
            for (int t = 0; t < RT; ++t) {
                const int r = FULL ? rb + t : min(rb + t, r1 - 1);  // rows past the tile repeat the last one; never stored
                xrow[t] = X + (long long)r * ld;
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    acc[t][v] = make_float2(0.f, 0.f);
                    a[t][v] = 0.0f;
                    if (UPDATE && (FULL || (v < nu && rb + t < r1))) a[t][v] = as[v * amax + r - r0];
                }
            }
            for (int c = cl, k = 0; k < nc; ++k, c += 128) {
                issue();
                copy_async_wait<ST - 1>();
                if (FULL || c < c1) {
                    float4 x[RT];
#pragma unroll
                    for (int t = 0; t < RT; ++t) x[t] = mine[(stage * RT + t) * 256];
                    row_columns<S, UPDATE, FORWARD, SAME, RT, COH, GRAD, true, FULL>(sh, nu, nf, x, a, acc, c, rb, r1, xrow, X,
                                                                               Xw, Gw, eta, g.m, ld, uqs, fqs, cmax,
                                                                               c - c0);
                }
                if (++stage == ST) stage = 0;
            }
            if (FORWARD) {
                float* __restrict__ Y = st.Y + (long long)w * st.y_stride + g.y_off;
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    if (v < nf) {
#pragma unroll
                        for (int t = 0; t < RT; ++t) {
                            const float s = warp_sum(acc[t][v].x + acc[t][v].y);
                            if (lane == 0 && (FULL || rb + t < r1))
                                Y[((long long)v * g.f_csplit + tile.ctile) * g.npad + rb + t] = s * sh.fs[v];
                        }
                    }
                }
            }
        }
        copy_async_wait<0>();
    } else {
        for (int rb = r0 + warp * RT; rb < r1; rb += 8 * RT) {
            float a[RT][S];
            float2 acc[RT][S];      // even and odd column pairs apart until the row's sum
            const float* xrow[RT];
#pragma unroll
            for (int t = 0; t < RT; ++t) {
                const int r = min(rb + t, r1 - 1);  // rows past the tile repeat the last one; never stored
                xrow[t] = X + (long long)r * ld;
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    acc[t][v] = make_float2(0.f, 0.f);
                    a[t][v] = 0.0f;
                    if (UPDATE && v < nu && rb + t < r1) a[t][v] = sh.uc[v] * ld_f<COH>(sh.up[v] + r);
                }
            }
            for (int c = c0 + lane * 4; c < c1; c += 128) {
                float4 x[RT];
#pragma unroll
                for (int t = 0; t < RT; ++t) x[t] = ld_stream(xrow[t] + c);
                row_columns<S, UPDATE, FORWARD, SAME, RT, COH, GRAD>(sh, nu, nf, x, a, acc, c, rb, r1, xrow, X, Xw, Gw, eta,
                                                                     g.m, ld);
            }
            if (FORWARD) {
                float* __restrict__ Y = st.Y + (long long)w * st.y_stride + g.y_off;
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    if (v < nf) {
#pragma unroll
                        for (int t = 0; t < RT; ++t) {
                            const float s = warp_sum(acc[t][v].x + acc[t][v].y);
                            if (lane == 0 && rb + t < r1)
                                Y[((long long)v * g.f_csplit + tile.ctile) * g.npad + rb + t] = s * sh.fs[v];
                        }
                    }
                }
            }
        }
    }
}

template <int S, bool UPDATE, bool FORWARD, bool SAME, int RT, bool GRAD = false>
__global__ void __launch_bounds__(256, row_min_blocks(S))
row_sweep_kernel(DevState st, const int* __restrict__ tab_u, const int* __restrict__ tab_f,
                 const Tile* __restrict__ tiles) {
    grid_dependency_sync();
    __shared__ RowShared<S> sh;
    extern __shared__ float4 row_ring[];
    const Tile tile = tiles[blockIdx.x];
    const LayerGeom& g = st.layers[tile.layer];
    // a tile of whole row batches and whole column steps takes the form without conditions
    const int rows = min(g.n, (tile.rtile + 1) * g.f_rows) - tile.rtile * g.f_rows;
    const int cols = min(g.ld, (tile.ctile + 1) * g.f_chunk) - tile.ctile * g.f_chunk;
    if (rows % (8 * RT) == 0 && cols % 128 == 0)
        row_tile<S, UPDATE, FORWARD, SAME, RT, false, GRAD, row_stages(S, RT), true>(st, tab_u, tab_f, tile, sh, row_ring);
    else
        row_tile<S, UPDATE, FORWARD, SAME, RT, false, GRAD, row_stages(S, RT), false>(st, tab_u, tab_f, tile, sh, row_ring);
}

// --------------------------------------------------------------------------
// Transposed sweep: Z[w][v][c] = sum_r Ph_v[r] X_w[r][c] over one row tile.
// 64 threads across (a float4 of columns each), 4 row groups down.
// --------------------------------------------------------------------------
template <int S>
struct ColShared {
    // P-hat of the tile's rows; up to four vectors each value twice, the operand of a packed FMA (eight
    // vectors would not leave room in the cooperative kernel's static shared memory)
    static constexpr int kDup = S <= 4 ? 2 : 1;
    float p[S][kColTileRowsMax][kDup];
    float a[S][kColTileRowsMax];   // UPDATE: coefficient of the pending correction per row
    float4 red[3][S][64];
};

// UPDATE (half-step mode): the pending correction of the odd iteration,
// X_w -= sum_v a_v[r] Q_v[c], is applied to the tile on its way through and the
// product is taken with the corrected values.
template <int S, bool COH, bool UPDATE>
__device__ __forceinline__ void col_tile(const DevState& st, const int* __restrict__ tab, const Tile tile,
                                         ColShared<S>& sh) {
    const LayerGeom g = st.layers[tile.layer];
    const int w = tile.worker;
    const int rank = st.rank;
    const float* __restrict__ X = st.X + (long long)w * st.x_stride + g.x_off;


    const int r0 = tile.rtile * g.t_rows;
    const int r1 = min(g.n, r0 + g.t_rows);
    const int deg = tab[st.tab.off_degree + w];
    const int nv = deg * rank;
    if (r1 > r0) {      // (checked build) everything this tile touches; the same for every thread
        const int cb = tile.ctile * kColTileCols, ce = min(g.ld, cb + kColTileCols);
        bool bad = ce > cb && PG_OOB(st, kSecX, X + (long long)r0 * g.ld + cb, (long long)(r1 - 1 - r0) * g.ld + (ce - cb));
        for (int v = 0; v < nv && ce > cb; ++v) {
            const int slot = v / rank, k = v - slot * rank;
            const int e = tab[st.tab.off_slot_edge + w * st.tab.max_degree + slot];
            bad = PG_OOB(st, kSecPh, st.Ph + (long long)e * st.ph_stride + g.ph_off + (long long)k * g.npad + r0, r1 - r0) ||
                  PG_OOB(st, kSecZ, st.Z + (long long)w * st.z_stride + g.z_off +
                                        ((long long)v * g.t_rtiles + tile.rtile) * g.ld + cb, ce - cb) || bad;
            if (UPDATE)
                bad = PG_OOB(st, kSecQ, st.Q + (long long)tab[st.tab.off_pair + e] * st.q_stride + g.q_off +
                                            (long long)k * g.ld + cb, ce - cb) || bad;
        }
        if (bad) return;
    }

    for (int idx = threadIdx.x; idx < S * kColTileRowsMax; idx += 256) {
        const int v = idx / kColTileRowsMax, rr = idx - v * kColTileRowsMax;
        float val = 0.0f;
        if (v < nv && r0 + rr < r1) {
            const int slot = v / rank, k = v - slot * rank;
            const int e = tab[st.tab.off_slot_edge + w * st.tab.max_degree + slot];
            val = ld_f<COH>(st.Ph + (long long)e * st.ph_stride + g.ph_off + (long long)k * g.npad + r0 + rr);
            if (UPDATE) {
                const int pair = tab[st.tab.off_pair + e];
                const float coef = __int_as_float(tab[st.tab.off_slot_coef + w * st.tab.max_degree + slot]) *
                                   ld_f<COH>(&st.Pn[(long long)e * st.n_layers + tile.layer]) *
                                   ld_f<COH>(&st.Qinv[((long long)pair * st.n_layers + tile.layer) * rank + k]);
                sh.a[v][rr] = coef * val;
            }
        } else if (UPDATE) {
            sh.a[v][rr] = 0.0f;
        }
#pragma unroll
        for (int d2 = 0; d2 < ColShared<S>::kDup; ++d2) sh.p[v][rr][d2] = val;
    }
    __syncthreads();

    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    const int c = tile.ctile * kColTileCols + tx * 4;
    const int ld = g.ld;
    float4 acc[S];
#pragma unroll
    for (int v = 0; v < S; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);

    float4 qv[S];
    if (UPDATE && c < ld) {
#pragma unroll
        for (int v = 0; v < S; ++v) {
            qv[v] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (v < nv) {
                const int slot = v / rank, k = v - slot * rank;
                const int e = tab[st.tab.off_slot_edge + w * st.tab.max_degree + slot];
                const int pair = tab[st.tab.off_pair + e];
                qv[v] = ld_vec<COH>(st.Q + (long long)pair * st.q_stride + g.q_off + (long long)k * g.ld + c);
            }
        }
    }
    if (!UPDATE && S <= 4 && c < ld && (r1 - r0) % 16 == 0) {
        // whole groups of 16 rows: nothing in the step is conditional.  Vectors the worker does not have were
        // staged as zeros and are worked on like the rest (their sums are never stored); packed FMAs, each
        // lane the same fused multiply-add as in the general form below.
        unsigned long long a2[S][2];
#pragma unroll
        for (int v = 0; v < S; ++v) a2[v][0] = a2[v][1] = 0ull;
        const float* xp = X + (long long)(r0 + ty) * ld + c;
        const long long step4 = 4LL * ld;
        for (int ro = ty; ro < r1 - r0; ro += 16, xp += 4 * step4) {
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = ld_stream(xp + u * step4);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const unsigned long long xlo = pack2(x[u].x, x[u].y), xhi = pack2(x[u].z, x[u].w);
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    const unsigned long long pp = *reinterpret_cast<const unsigned long long*>(&sh.p[v][ro + 4 * u][0]);
                    a2[v][0] = fma2(pp, xlo, a2[v][0]);
                    a2[v][1] = fma2(pp, xhi, a2[v][1]);
                }
            }
        }
#pragma unroll
        for (int v = 0; v < S; ++v) {
            unpack2(a2[v][0], acc[v].x, acc[v].y);
            unpack2(a2[v][1], acc[v].z, acc[v].w);
        }
    } else if (c < ld) {
        const float* xc = X + c;
        for (int r = r0 + ty; r < r1; r += 16) {
            float4 x[4];
            int rr[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                rr[u] = r + 4 * u;                       // rows past r1 read the last row with p = 0
                x[u] = ld_stream(xc + (long long)min(rr[u], r1 - 1) * ld);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ro = min(rr[u] - r0, kColTileRowsMax - 1);
                const bool in = rr[u] < r1;
                if (UPDATE && in) {
#pragma unroll
                    for (int v = 0; v < S; ++v) {
                        if (v < nv) {
                            const float a = sh.a[v][ro];
                            x[u].x = fmaf(-a, qv[v].x, x[u].x); x[u].y = fmaf(-a, qv[v].y, x[u].y);
                            x[u].z = fmaf(-a, qv[v].z, x[u].z); x[u].w = fmaf(-a, qv[v].w, x[u].w);
                        }
                    }
                    st_stream(const_cast<float*>(xc) + (long long)rr[u] * ld, x[u]);
                }
#pragma unroll
                for (int v = 0; v < S; ++v) {
                    if (v < nv) {
                        const float p = in ? sh.p[v][ro][0] : 0.0f;
                        acc[v].x = fmaf(p, x[u].x, acc[v].x);
                        acc[v].y = fmaf(p, x[u].y, acc[v].y);
                        acc[v].z = fmaf(p, x[u].z, acc[v].z);
                        acc[v].w = fmaf(p, x[u].w, acc[v].w);
                    }
                }
            }
        }
    }
    if (ty > 0) {
#pragma unroll
        for (int v = 0; v < S; ++v) sh.red[ty - 1][v][tx] = acc[v];
    }
    __syncthreads();
    if (ty == 0 && c < ld) {
        float* __restrict__ Z = st.Z + (long long)w * st.z_stride + g.z_off;
#pragma unroll
        for (int v = 0; v < S; ++v) {
            if (v < nv) {
                float4 s = acc[v];
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    const float4 o = sh.red[t][v][tx];
                    s.x += o.x; s.y += o.y; s.z += o.z; s.w += o.w;
                }
                *reinterpret_cast<float4*>(Z + ((long long)v * g.t_rtiles + tile.rtile) * ld + c) = s;
            }
        }
    }
}

template <int S, bool UPDATE>
__global__ void __launch_bounds__(256)
col_sweep_kernel(DevState st, const int* __restrict__ tab, const Tile* __restrict__ tiles) {
    grid_dependency_sync();
    __shared__ ColShared<S> sh;
    col_tile<S, false, UPDATE>(st, tab, tiles[blockIdx.x], sh);
}

// Half-step mode, odd iteration: p = Y[i] - Y[j] (fp64 sums of the partials),
// P-hat = p / ||p|| as fp32 and ||p|| kept beside it, so that the update
// p q-hat^T and the next iteration's unit vector both come from P-hat.  A zero or
// non-finite p gives P-hat = 0 (the edge falls silent).  One CTA per (edge, layer).
__global__ void __launch_bounds__(512)
edge_odd_kernel(DevState st, const int* __restrict__ tab) {
    grid_dependency_sync();
    __shared__ double scratch[33];
    const int L = st.n_layers;
    const int e = blockIdx.x / L, l = blockIdx.x - e * L;
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[l];
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int si = tab[st.tab.off_slot_i + e], sj = tab[st.tab.off_slot_j + e];
    const float* yi = st.Y + (long long)wi * st.y_stride + g.y_off + (long long)si * g.f_csplit * g.npad;
    const float* yj = st.Y + (long long)wj * st.y_stride + g.y_off + (long long)sj * g.f_csplit * g.npad;
    float* Ph = st.Ph + (long long)e * st.ph_stride + g.ph_off;
    if (PG_OOB(st, kSecY, yi, (long long)g.f_csplit * g.npad) || PG_OOB(st, kSecY, yj, (long long)g.f_csplit * g.npad) ||
        PG_OOB(st, kSecPh, Ph, g.npad) || PG_OOB(st, kSecPn, st.Pn + (long long)e * L + l, 1))
        return;
    auto raw = [&](int r) {
        double a = 0.0, b = 0.0;
        for (int cs = 0; cs < g.f_csplit; ++cs) {
            a += (double)yi[(long long)cs * g.npad + r];
            b += (double)yj[(long long)cs * g.npad + r];
        }
        return a - b;
    };
    double part = 0.0;
    for (int r = threadIdx.x; r < g.n; r += blockDim.x) {
        const double v = raw(r);
        part += v * v;
    }
    const double nn = block_sum(part, scratch);
    const bool finite = isfinite(nn);
    const bool live = finite && nn > 0.0;
    const double inv = live ? 1.0 / sqrt(nn) : 0.0;
    for (int r = threadIdx.x; r < g.npad; r += blockDim.x)
        Ph[r] = (live && r < g.n) ? (float)(raw(r) * inv) : 0.0f;
    if (threadIdx.x == 0) {
        st.Pn[(long long)e * L + l] = live ? (float)sqrt(nn) : 0.0f;
        st.live[(long long)e * L + l] = 1;     // the even iteration always stores its vector, zero included
        if (!finite) atomicOr(st.status, 1 << kStatusNumeric);
    }
}

// --------------------------------------------------------------------------
// Edge step, left factor: P = Y[i] - Y[j] (partials added in order, fp64),
// modified Gram-Schmidt in column order, P-hat stored as fp32.
// One CTA per (edge, layer).
// --------------------------------------------------------------------------
template <bool COH>
__device__ __forceinline__ void edge_left_step(const DevState& st, const int* __restrict__ tab, int e, int l,
                                               double* scratch) {
    int* live_out = st.live;
    const int L = st.n_layers, rank = st.rank;
    const LayerGeom g = st.layers[l];
    if (g.pair_mode) return;   // handled by the pair sweep's own edge step
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int pair = tab[st.tab.off_pair + e];
    const int si = tab[st.tab.off_slot_i + e], sj = tab[st.tab.off_slot_j + e];
    const float* Yi = st.Y + (long long)wi * st.y_stride + g.y_off;
    const float* Yj = st.Y + (long long)wj * st.y_stride + g.y_off;
    float* Ph = st.Ph + (long long)e * st.ph_stride + g.ph_off;
    double coef[kMaxRank];
    {   // (checked build) the slices of both ends' partial sums, the factor and its flags
        const long long slice = (long long)rank * g.f_csplit * g.npad;
        if (PG_OOB(st, kSecY, Yi + (long long)si * slice, slice) || PG_OOB(st, kSecY, Yj + (long long)sj * slice, slice) ||
            PG_OOB(st, kSecPh, Ph, (long long)rank * g.npad) ||
            PG_OOB(st, kSecLive, live_out + ((long long)e * L + l) * rank, rank))
            return;
    }

    if (rank == 1 && g.npad <= 4 * (int)blockDim.x) {
        // one column and at most four rows per thread: the differences stay in registers
        // between the norm and the scaling (same sums in the same order as the general case)
        const float* yi = Yi + (long long)si * g.f_csplit * g.npad;
        const float* yj = Yj + (long long)sj * g.f_csplit * g.npad;
        double v[4];
        double part = 0.0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int r = threadIdx.x + t * blockDim.x;
            v[t] = 0.0;
            if (r < g.n) {
                double a = 0.0, b = 0.0;
                for (int cs = 0; cs < g.f_csplit; ++cs) {
                    a += (double)ld_f<COH>(yi + (long long)cs * g.npad + r);
                    b += (double)ld_f<COH>(yj + (long long)cs * g.npad + r);
                }
                v[t] = a - b;
                part += v[t] * v[t];
            }
        }
        const double nn = block_sum(part, scratch);
        const bool finite = isfinite(nn);
        const bool live = finite && nn > 0.0;
        const double inv = live ? 1.0 / sqrt(nn) : 0.0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int r = threadIdx.x + t * blockDim.x;
            if (r < g.npad) Ph[r] = live ? (float)(v[t] * inv) : 0.0f;
        }
        if (threadIdx.x == 0) {
            live_out[(long long)e * L + l] = live ? 1 : 0;
            if (!finite) atomicOr(st.status, 1 << kStatusNumeric);
        }
        return;
    }

    for (int k = 0; k < rank; ++k) {
        const float* yi = Yi + (long long)(si * rank + k) * g.f_csplit * g.npad;
        const float* yj = Yj + (long long)(sj * rank + k) * g.f_csplit * g.npad;
        // the difference of the two endpoints' products, one row at a time
        auto raw = [&](int r) {
            double a = 0.0, b = 0.0;
            for (int cs = 0; cs < g.f_csplit; ++cs) {
                a += (double)ld_f<COH>(yi + (long long)cs * g.npad + r);
                b += (double)ld_f<COH>(yj + (long long)cs * g.npad + r);
            }
            return a - b;
        };
        double part = 0.0;
        for (int r = threadIdx.x; r < g.n; r += blockDim.x) {
            const double v = raw(r);
            part += v * v;
        }
        const double pre = block_sum(part, scratch);
        // project out the earlier columns one after the other (modified Gram-Schmidt)
        for (int h = 0; h < k; ++h) {
            part = 0.0;
            for (int r = threadIdx.x; r < g.n; r += blockDim.x) {
                double v = raw(r);
                for (int h2 = 0; h2 < h; ++h2) v -= coef[h2] * (double)ld_own<COH>(Ph + (long long)h2 * g.npad + r);
                part += v * (double)ld_own<COH>(Ph + (long long)h * g.npad + r);
            }
            coef[h] = block_sum(part, scratch);
        }
        double nn = pre;
        if (k > 0) {
            part = 0.0;
            for (int r = threadIdx.x; r < g.n; r += blockDim.x) {
                double v = raw(r);
                for (int h = 0; h < k; ++h) v -= coef[h] * (double)ld_own<COH>(Ph + (long long)h * g.npad + r);
                part += v * v;
            }
            nn = block_sum(part, scratch);
        }
        const bool finite = isfinite(nn);
        // a residual below 1e-5 of the column's length is rounding noise of the fp32 inputs
        const bool live = finite && nn > 0.0 && (k == 0 || nn > 1e-10 * pre);
        const double inv = live ? 1.0 / sqrt(nn) : 0.0;
        for (int r = threadIdx.x; r < g.npad; r += blockDim.x) {
            double v = 0.0;
            if (live && r < g.n) {
                v = raw(r);
                for (int h = 0; h < k; ++h) v -= coef[h] * (double)ld_own<COH>(Ph + (long long)h * g.npad + r);
                v *= inv;
            }
            Ph[(long long)k * g.npad + r] = (float)v;
        }
        if (threadIdx.x == 0) {
            live_out[((long long)e * L + l) * rank + k] = live ? 1 : 0;
            if (!finite) atomicOr(st.status, 1 << kStatusNumeric);
        }
        __syncthreads();  // the stored column is read by the next column's projections
    }
    (void)pair;
}

__global__ void __launch_bounds__(512)
edge_left_kernel(DevState st, const int* __restrict__ tab) {
    grid_dependency_sync();
    __shared__ double scratch[33];
    const int e = blockIdx.x / st.n_layers, l = blockIdx.x - e * st.n_layers;
    if (e >= tab[st.tab.off_n_edges]) return;
    edge_left_step<false>(st, tab, e, l, scratch);
}

// --------------------------------------------------------------------------
// Edge step, right factor: Q' = Z[i] - Z[j] (row-tile partials added in order,
// fp64), stored as the pair's new Q with 1/||Q'||.  Degenerate columns keep
// their old vector.  One CTA per (edge, layer).
// --------------------------------------------------------------------------
template <bool COH>
__device__ __forceinline__ void edge_right_step(const DevState& st, const int* __restrict__ tab, int e, int l,
                                                double* scratch) {
    const int* live_in = st.live;
    const int L = st.n_layers, rank = st.rank;
    const LayerGeom g = st.layers[l];
    if (g.pair_mode) return;
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int pair = tab[st.tab.off_pair + e];
    const int si = tab[st.tab.off_slot_i + e], sj = tab[st.tab.off_slot_j + e];
    const float* Zi = st.Z + (long long)wi * st.z_stride + g.z_off;
    const float* Zj = st.Z + (long long)wj * st.z_stride + g.z_off;
    float* Q = st.Q + (long long)pair * st.q_stride + g.q_off;
    {   // (checked build) the slices of both ends' partial sums and the stored vectors
        const long long slice = (long long)rank * g.t_rtiles * g.ld;
        if (PG_OOB(st, kSecZ, Zi + (long long)si * slice, slice) || PG_OOB(st, kSecZ, Zj + (long long)sj * slice, slice) ||
            PG_OOB(st, kSecQ, Q, (long long)rank * g.ld) ||
            PG_OOB(st, kSecQinv, st.Qinv + ((long long)pair * L + l) * rank, rank) ||
            PG_OOB(st, kSecLive, live_in + ((long long)e * L + l) * rank, rank))
            return;
    }

    for (int k = 0; k < rank; ++k) {
        if (!ld_i<COH>(&live_in[((long long)e * L + l) * rank + k])) continue;  // uniform over the block
        const float* zi = Zi + (long long)(si * rank + k) * g.t_rtiles * g.ld;
        const float* zj = Zj + (long long)(sj * rank + k) * g.t_rtiles * g.ld;
        double part = 0.0;
        // two columns per thread and pass, four tiles of both ends at a time: sixteen
        // independent loads in flight, added in tile order
        for (int c0 = threadIdx.x; c0 < g.m; c0 += 2 * blockDim.x) {
            const int c1 = c0 + blockDim.x;
            const bool two = c1 < g.m;
            double a0 = 0.0, b0 = 0.0, a1 = 0.0, b1 = 0.0;
            for (int rt = 0; rt < g.t_rtiles; rt += 4) {
                float vi0[4], vj0[4], vi1[4], vj1[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool in = rt + j < g.t_rtiles;
                    const long long row = (long long)(rt + j) * g.ld;
                    vi0[j] = in ? ld_own<COH>(zi + row + c0) : 0.0f;
                    vj0[j] = in ? ld_own<COH>(zj + row + c0) : 0.0f;
                    vi1[j] = in && two ? ld_own<COH>(zi + row + c1) : 0.0f;
                    vj1[j] = in && two ? ld_own<COH>(zj + row + c1) : 0.0f;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a0 += (double)vi0[j]; b0 += (double)vj0[j];
                    a1 += (double)vi1[j]; b1 += (double)vj1[j];
                }
            }
            const float q0 = (float)(a0 - b0);
            Q[(long long)k * g.ld + c0] = q0;
            part += (double)q0 * (double)q0;
            if (two) {
                const float q1 = (float)(a1 - b1);
                Q[(long long)k * g.ld + c1] = q1;
                part += (double)q1 * (double)q1;
            }
        }
        const double nn = block_sum(part, scratch);
        if (threadIdx.x == 0) {
            st.Qinv[((long long)pair * L + l) * rank + k] = nn > 0.0 ? (float)(1.0 / sqrt(nn)) : 0.0f;
            if (!isfinite(nn)) atomicOr(st.status, 1 << kStatusNumeric);
        }
    }
}

__global__ void __launch_bounds__(512)
edge_right_kernel(DevState st, const int* __restrict__ tab) {
    grid_dependency_sync();
    __shared__ double scratch[33];
    const int e = blockIdx.x / st.n_layers, l = blockIdx.x - e * st.n_layers;
    if (e >= tab[st.tab.off_n_edges]) return;
    edge_right_step<false>(st, tab, e, l, scratch);
}

// --------------------------------------------------------------------------
// Random-projection compressors (Section 5.1 of the paper): fresh directions.
// Philox4x32-10 (Salmon et al., SC'11) and Box-Muller in fp64, the same stream
// as the seeded initial vectors but under the step's key; entry e of column k of
// pair (i<j), layer l uses counter (e/4, l, i, j*256+k).  The rank columns are
// then orthonormalised (modified Gram-Schmidt in fp64 against the stored fp32
// columns, same dependent-column rule as the power step).
// side 0: directions in R^cols, written to the pair's Q with 1/norm = 1;
// side 1: directions in R^rows, written to the edge's P-hat.
// One CTA per (edge, layer).
// --------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(unsigned c0, unsigned c1, unsigned c2, unsigned c3,
                                              unsigned k0, unsigned k1, unsigned out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const unsigned hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const unsigned n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

__global__ void __launch_bounds__(256)
random_directions_kernel(DevState st, const int* __restrict__ tab, unsigned key_lo, unsigned key_hi, int side) {
    grid_dependency_sync();
    __shared__ double scratch[33];
    const int L = st.n_layers, rank = st.rank;
    const int e = blockIdx.x / L, l = blockIdx.x - e * L;
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[l];
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int pair = tab[st.tab.off_pair + e];
    const int len = side == 0 ? g.m : g.n;
    const int stride = side == 0 ? g.ld : g.npad;
    float* dst = side == 0 ? st.Q + (long long)pair * st.q_stride + g.q_off
                           : st.Ph + (long long)e * st.ph_stride + g.ph_off;
    double coef[kMaxRank];
    if (PG_OOB(st, side == 0 ? kSecQ : kSecPh, dst, (long long)rank * stride)) return;
    for (int k = 0; k < rank; ++k) {
        float* col = dst + (long long)k * stride;
        for (int b = threadIdx.x; 4 * b < stride; b += blockDim.x) {
            unsigned x[4];
            philox4x32_10((unsigned)b, (unsigned)l, (unsigned)wi, (unsigned)wj * 256u + (unsigned)k, key_lo, key_hi, x);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const double u1 = ((double)x[2 * h] + 0.5) * (1.0 / 4294967296.0);
                const double u2 = ((double)x[2 * h + 1] + 0.5) * (1.0 / 4294967296.0);
                const double radius = sqrt(-2.0 * log(u1));
                const double angle = 6.283185307179586476925286766559 * u2;
                const int e0 = 4 * b + 2 * h;
                if (e0 < stride) col[e0] = e0 < len ? (float)(radius * cos(angle)) : 0.0f;
                if (e0 + 1 < stride) col[e0 + 1] = e0 + 1 < len ? (float)(radius * sin(angle)) : 0.0f;
            }
        }
        __syncthreads();
        auto resid = [&](int r, int upto) {
            double v = (double)col[r];
            for (int h = 0; h < upto; ++h) v -= coef[h] * (double)dst[(long long)h * stride + r];
            return v;
        };
        double part = 0.0;
        for (int r = threadIdx.x; r < len; r += blockDim.x) part += (double)col[r] * (double)col[r];
        const double pre = block_sum(part, scratch);
        for (int h = 0; h < k; ++h) {
            part = 0.0;
            for (int r = threadIdx.x; r < len; r += blockDim.x) part += resid(r, h) * (double)dst[(long long)h * stride + r];
            coef[h] = block_sum(part, scratch);
        }
        part = 0.0;
        for (int r = threadIdx.x; r < len; r += blockDim.x) {
            const double v = resid(r, k);
            part += v * v;
        }
        const double nn = block_sum(part, scratch);
        const bool live = isfinite(nn) && nn > 0.0 && (k == 0 || nn > 1e-10 * pre);
        const double inv = live ? 1.0 / sqrt(nn) : 0.0;
        for (int r = threadIdx.x; r < len; r += blockDim.x) col[r] = live ? (float)(resid(r, k) * inv) : 0.0f;
        if (threadIdx.x == 0) {
            if (side == 0) st.Qinv[((long long)pair * L + l) * rank + k] = live ? 1.0f : 0.0f;
            st.live[((long long)e * L + l) * rank + k] = 1;
        }
        __syncthreads();
    }
}

// P = Y[i] - Y[j], unnormalised (the directions are orthonormal already): the
// left factor of the random right projection's update (X_i U - X_j U) U^T.
__global__ void __launch_bounds__(256)
edge_raw_kernel(DevState st, const int* __restrict__ tab) {
    grid_dependency_sync();
    const int L = st.n_layers, rank = st.rank;
    const int e = blockIdx.x / L, l = blockIdx.x - e * L;
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[l];
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int si = tab[st.tab.off_slot_i + e], sj = tab[st.tab.off_slot_j + e];
    const float* Yi = st.Y + (long long)wi * st.y_stride + g.y_off;
    const float* Yj = st.Y + (long long)wj * st.y_stride + g.y_off;
    float* Ph = st.Ph + (long long)e * st.ph_stride + g.ph_off;
    {
        const long long slice = (long long)rank * g.f_csplit * g.npad;
        if (PG_OOB(st, kSecY, Yi + (long long)si * slice, slice) || PG_OOB(st, kSecY, Yj + (long long)sj * slice, slice) ||
            PG_OOB(st, kSecPh, Ph, (long long)rank * g.npad))
            return;
    }
    for (int k = 0; k < rank; ++k) {
        const float* yi = Yi + (long long)(si * rank + k) * g.f_csplit * g.npad;
        const float* yj = Yj + (long long)(sj * rank + k) * g.f_csplit * g.npad;
        for (int r = threadIdx.x; r < g.npad; r += blockDim.x) {
            double a = 0.0, b = 0.0;
            if (r < g.n)
                for (int cs = 0; cs < g.f_csplit; ++cs) {
                    a += (double)yi[(long long)cs * g.npad + r];
                    b += (double)yj[(long long)cs * g.npad + r];
                }
            Ph[(long long)k * g.npad + r] = (float)(a - b);
        }
    }
}

// 1 / ||Q_k|| of a pair-sweep layer from the shares the pair edge step left.
__device__ __forceinline__ float pair_qinv(const DevState& st, int pair, int layer, int k = 0) {
    const double* n2 = st.Qn2 + (((long long)pair * st.n_layers + layer) * st.rank + k) * kEdgeChunks;
    double t = 0.0;
#pragma unroll
    for (int k = 0; k < kEdgeChunks; ++k) t += n2[k];
    return t > 0.0 ? (float)(1.0 / sqrt(t)) : 0.0f;
}

// Factors of the corrections that are still pending at one end of an edge: the
// previous step left at most D of them at a worker (one per incident edge), each
// coef * p-hat_r * q' with p-hat of that edge and the edge's new stored vector.
template <int D>
struct PendingEnd {
    const float* vec[D];
    const float* ph[D];
    float coef[D];
};
template <int D>
__device__ __forceinline__ void pending_of(const DevState& st, const int* __restrict__ tab_prev, int w,
                                           const LayerGeom& g, const float* dflt, PendingEnd<D>& pe) {
    const int deg = min(tab_prev[st.tab.off_degree + w], D);
#pragma unroll
    for (int s = 0; s < D; ++s) {
        pe.vec[s] = dflt;
        pe.ph[s] = nullptr;
        pe.coef[s] = 0.0f;
        if (s < deg) {
            const int ep = tab_prev[st.tab.off_slot_edge + w * st.tab.max_degree + s];
            pe.vec[s] = st.Qr + (long long)tab_prev[st.tab.off_pair + ep] * st.q_stride + g.q_off;
            pe.ph[s] = st.Ph + (long long)ep * st.ph_stride + g.ph_off;
            pe.coef[s] = __int_as_float(tab_prev[st.tab.off_slot_coef + w * st.tab.max_degree + s]);
        }
    }
}

// The raw form of the pair sweep (graphs where a row has several readers).  With
// the corrections of the previous step still pending, the difference of an edge
// (i<j) is   D' = D - sum_k c_k p-hat_k q'_k^T   where D = X_i - X_j as stored and k
// runs over the edges of the previous step at either end (c_k = coef at i, minus
// coef at j; the edge itself, present at both ends, gets both).  Then
//     p   = D' q-hat = D q-hat - sum_k c_k (q'_k . q-hat) p-hat_k
//     D'^T p        = D^T p   - sum_k c_k (p-hat_k . p) q'_k
// so the sweep needs the rows only as they are in memory: the pending terms enter p
// as one scalar per row and D^T p as a few vectors, added by the pair edge step.
// Only the one CTA that owns a worker's rows corrects and writes them.  Terms in the
// order: the slots of worker i, then the slots of worker j without the edge itself.
struct RawTerm {
    int edge;
    float coef;
};
__device__ __forceinline__ int raw_terms(const DevState& st, const int* __restrict__ tab, int e, int wi, int wj,
                                         RawTerm* out) {
    const int md = st.tab.max_degree;
    const int di = min(tab[st.tab.off_degree + wi], md), dj = min(tab[st.tab.off_degree + wj], md);
    int n = 0;
    for (int s = 0; s < di && n < kMaxTerms; ++s) {
        out[n].edge = tab[st.tab.off_slot_edge + wi * md + s];
        out[n].coef = __int_as_float(tab[st.tab.off_slot_coef + wi * md + s]);
        ++n;
    }
    for (int s = 0; s < dj; ++s) {
        const int ep = tab[st.tab.off_slot_edge + wj * md + s];
        const float c = __int_as_float(tab[st.tab.off_slot_coef + wj * md + s]);
        if (ep == e) {
            for (int k = 0; k < n; ++k)
                if (out[k].edge == e) out[k].coef -= c;
        } else if (n < kMaxTerms) {
            out[n].edge = ep;
            out[n].coef = -c;
            ++n;
        }
    }
    return n;
}

// (checked build) what a pair-sweep tile touches: rows [r0, r1) of both ends where it reads and where it
// writes, the edge's stored vectors (`rank` columns), the rows of its raw left factor, its shares of
// D^T P and its scalars.  True if any of it lies outside its section; the same for every thread.
__device__ __forceinline__ bool pair_tile_out_of_bounds(const DevState& st, const LayerGeom& g, const float* Xi,
                                                        const float* Xj, const float* Xi_w, const float* Xj_w,
                                                        int r0, int r1, const float* q, const float* Pw,
                                                        const float* up, int up_count, const double* sp) {
    if (r1 <= r0) return false;
    const long long first = (long long)r0 * g.ld, span = (long long)(r1 - r0) * g.ld;
    bool bad = PG_OOB(st, kSecX, Xi + first, span) || PG_OOB(st, kSecX, Xj + first, span);
    bad = PG_OOB(st, kSecX, Xi_w + first, span) || PG_OOB(st, kSecX, Xj_w + first, span) || bad;
    bad = PG_OOB(st, kSecQ, q, (long long)st.rank * g.ld) || bad;
    for (int k = 0; k < st.rank; ++k) bad = PG_OOB(st, kSecPh, Pw + (long long)k * g.npad + r0, r1 - r0) || bad;
    bad = PG_OOB(st, kSecUp, up, up_count) || PG_OOB(st, kSecSp, sp, kSpPerTile) || bad;
    return bad;
}
// (checked build) the vectors and left factors of the corrections pending at one end
template <int D>
__device__ __forceinline__ bool pending_out_of_bounds(const DevState& st, const LayerGeom& g, const PendingEnd<D>& pe,
                                                      int r0, int r1) {
    bool bad = false;
#pragma unroll
    for (int s = 0; s < D; ++s)
        if (pe.ph[s]) bad = PG_OOB(st, kSecQ, pe.vec[s], g.ld) || PG_OOB(st, kSecPh, pe.ph[s] + r0, r1 - r0) || bad;
    return bad;
}

// Prologue of a raw sweep (whole CTA of 256 threads): the terms of edge e and, for the
// rows [r0, r1) of the tile, the scalar each row's product loses to them,
//     corr[r] = sum_k c_k (q'_k . q-hat) p-hat_k[r],
// the products q'_k . q-hat taken in fp64 from the fp32 vectors (q-hat = `q` * qinv).
// Returns the number of terms; s_ph[k] points at p-hat_k.
__device__ int raw_prologue(const DevState& st, const int* __restrict__ tab, int e, int wi, int wj,
                            const LayerGeom& g, const float* __restrict__ q, float qinv, int r0, int r1,
                            float* s_corr, const float** s_ph, double* s_red /* 8 x kMaxTerms + kMaxTerms */) {
    RawTerm terms[kMaxTerms];
    int nt = raw_terms(st, tab, e, wi, wj, terms);
    const float* vec[kMaxTerms];
    double part[kMaxTerms];
#pragma unroll
    for (int k = 0; k < kMaxTerms; ++k) {
        part[k] = 0.0;
        vec[k] = q;
        if (k < nt) vec[k] = st.Qr + (long long)tab[st.tab.off_pair + terms[k].edge] * st.q_stride + g.q_off;
    }
    for (int k = 0; k < nt; ++k)      // (checked build) a term that points outside drops all of them
        if (PG_OOB(st, kSecQ, vec[k], g.ld) ||
            (r1 > r0 && PG_OOB(st, kSecPh, st.Ph + (long long)terms[k].edge * st.ph_stride + g.ph_off + r0, r1 - r0)))
            nt = 0;
    for (int idx = threadIdx.x; idx < g.m; idx += blockDim.x) {
        const double qh = (double)(q[idx] * qinv);
#pragma unroll
        for (int k = 0; k < kMaxTerms; ++k)
            if (k < nt) part[k] += (double)vec[k][idx] * qh;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < kMaxTerms; ++k) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part[k] += __shfl_xor_sync(0xffffffffu, part[k], o);
        if (lane == 0) s_red[warp * kMaxTerms + k] = part[k];
    }
    __syncthreads();
    if (threadIdx.x < kMaxTerms) {
        double beta = 0.0;
        for (int w8 = 0; w8 < 8; ++w8) beta += s_red[w8 * kMaxTerms + threadIdx.x];
        const int k = threadIdx.x;
        s_red[8 * kMaxTerms + k] = k < nt ? (double)terms[k].coef * beta : 0.0;
        s_ph[k] = st.Ph + (long long)(k < nt ? terms[k].edge : e) * st.ph_stride + g.ph_off;
    }
    __syncthreads();
    for (int r = r0 + threadIdx.x; r < r1; r += blockDim.x) {
        float c = 0.0f;
#pragma unroll
        for (int k = 0; k < kMaxTerms; ++k)
            if (k < nt) c = fmaf((float)s_red[8 * kMaxTerms + k], __ldg(s_ph[k] + r), c);
        s_corr[r - r0] = c;
    }
    return nt;      // the caller's next barrier publishes s_corr
}

// --------------------------------------------------------------------------
// Pair sweep (rank 1; a matching, or a static graph of degree <= 2, where a row
// can have two readers).  One CTA owns a block of rows of BOTH ends of an edge
// (i<j) and reads each row of X_i and X_j once:
//   - applies the correction that is still pending from the previous step to
//     each row (each end has its own previous edges) and writes the rows back,
//   - forms the row of D = X_i - X_j, its product with q-hat:  p_r = D_r . q-hat,
//   - accumulates u += p_r D_r, i.e. its share of D^T p, and of ||p||^2.
// The normalisation is a scalar, so it is applied afterwards by the pair edge
// step:  p-hat = p / ||p||,  Q' = D^T p-hat = u / ||p||.  This is the same power
// step as the three-sweep path with X read once instead of twice.
// Four kernels by row length: a warp per row, a CTA per row (fed by bulk copies
// where its registers hold the row, by plain loads beyond), a cluster per row.
// --------------------------------------------------------------------------

// --------------------------------------------------------------------------
// Pair sweep, a warp per row (rows of up to kPairMaxLd floats), fed by bulk
// asynchronous copies (TMA).  The rows of a tile are contiguous in memory (full rows, padded leading
// dimension), so one thread moves kBulkRows rows of X_i and of X_j into shared
// memory with two cp.async.bulk copies per stage; an mbarrier per stage counts
// the bytes.  kBulkStages stages are in flight, so the loads of the next stages
// never wait for registers or for the arithmetic of the current one.  Every
// warp then takes one row of the stage out of shared memory into registers (up
// to 8 float4 per lane) and writes the corrected rows straight to global memory.  All mbarrier waits are bounded: a wait that runs out raises the
// time-out bit of the status word and the CTA leaves after waiting (bounded
// again) for the copies it still has in flight.
// --------------------------------------------------------------------------
constexpr int kBulkRows = 8;      // rows per stage = warps per CTA
constexpr int kBulkStages = 3;
constexpr int kBulkSpinLimit = 1 << 24;

__device__ __forceinline__ unsigned smem_addr(const void* p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// bytes and both addresses must be multiples of 16
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, unsigned bytes,
                                          unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// waits for phase `parity` of `bar`; false if it gave up (or another thread did)
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity, volatile int* abort_flag,
                                                  int* status) {
    for (int spin = 0; spin < kBulkSpinLimit; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    atomicOr(status, 1 << kStatusTimeout);
    return false;
}

template <int NV, bool UPDATE, int D>
__global__ void __launch_bounds__(256, 1)
pair_sweep_bulk_kernel(DevState st, const int* __restrict__ tab_prev, const int* __restrict__ tab_cur,
                       const Tile* __restrict__ tiles) {
    grid_dependency_sync();
    constexpr int STAGES = kBulkStages;
    extern __shared__ __align__(128) unsigned char s_dyn[];
    __shared__ __align__(16) float s_q[NV * 128];
    __shared__ __align__(16) float s_ui[D][NV * 128];
    __shared__ __align__(16) float s_uj[D][NV * 128];
    __shared__ __align__(8) unsigned long long s_full[STAGES];
    __shared__ double s_s[8];
    __shared__ int s_abort;

    const Tile tile = tiles[blockIdx.x];
    const int e = tile.worker;
    if (e >= tab_cur[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab_cur[st.tab.off_edge_i + e], wj = tab_cur[st.tab.off_edge_j + e];
    const int pair = tab_cur[st.tab.off_pair + e];
    float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;
    const unsigned row_bytes = (unsigned)ld * 4u;                 // multiple of 16: ld is a multiple of 4
    float* s_stage = reinterpret_cast<float*>(s_dyn);             // [stage][matrix][row][ld]

    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv = pair_qinv(st, pair, tile.layer);
    // only the edge that owns a worker's rows writes them back (to Xw, which is X itself
    // unless rows have a second reader; on a matching every edge owns both of its ends)
    // (with one slot per worker every edge owns both ends and the rows are corrected in place: known at compile time)
    const int own = D == 1 ? 3 : tab_cur[st.tab.off_own + e];
    const bool own_i = D == 1 || (own & 1) != 0, own_j = D == 1 || (own & 2) != 0;
    float* Xi_w = D == 1 ? const_cast<float*>(Xi) : st.Xw + (long long)wi * st.x_stride + g.x_off;
    float* Xj_w = D == 1 ? const_cast<float*>(Xj) : st.Xw + (long long)wj * st.x_stride + g.x_off;
    PendingEnd<D> pi, pj;
    if (UPDATE) {
        pending_of<D>(st, tab_prev, wi, g, q, pi);
        pending_of<D>(st, tab_prev, wj, g, q, pj);
    }
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    const int n_stages = (r1 - r0 + kBulkRows - 1) / kBulkRows;
    if (pair_tile_out_of_bounds(st, g, Xi, Xj, Xi_w, Xj_w, r0, r1, q, st.PhNext + (long long)e * st.ph_stride + g.ph_off,
                                st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld, ld,
                                st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile) ||
        (UPDATE && (pending_out_of_bounds<D>(st, g, pi, r0, r1) || pending_out_of_bounds<D>(st, g, pj, r0, r1))))
        return;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s2 = 0; s2 < STAGES; ++s2) mbar_init(&s_full[s2], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int idx = threadIdx.x; idx < NV * 128; idx += 256) {
        const bool in = idx < ld;
        s_q[idx] = in ? q[idx] * qinv : 0.0f;
        if (UPDATE) {
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                s_ui[s2][idx] = in ? pi.vec[s2][idx] : 0.0f;
                s_uj[s2][idx] = in ? pj.vec[s2][idx] : 0.0f;
            }
        }
    }
    __syncthreads();

    // stage `sidx` covers rows r0 + sidx*kBulkRows ...; both slabs are contiguous in global memory
    auto issue = [&](int sidx) {
        const int slot = sidx % STAGES;
        const int row = r0 + sidx * kBulkRows;
        const unsigned bytes = (unsigned)min(kBulkRows, r1 - row) * row_bytes;
        float* dst = s_stage + (size_t)slot * 2 * kBulkRows * ld;
        mbar_expect_tx(&s_full[slot], 2 * bytes);
        bulk_load(dst, Xi + (long long)row * ld, bytes, &s_full[slot]);
        bulk_load(dst + (size_t)kBulkRows * ld, Xj + (long long)row * ld, bytes, &s_full[slot]);
    };
    int issued = 0;
    if (threadIdx.x == 0)
        for (; issued < STAGES - 1 && issued < n_stages; ++issued) issue(issued);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    float4 u[NV];
#pragma unroll
    for (int k = 0; k < NV; ++k) u[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    float ssum = 0.0f;
    bool ok = true;

    for (int it = 0; it < n_stages; ++it) {
        const int slot = it % STAGES;
        if (threadIdx.x == 0 && it + STAGES - 1 < n_stages) {
            issue(it + STAGES - 1);      // its slot was read for the last time before the barrier below
            issued = it + STAGES;
        }
        const bool mine = mbar_wait_bounded(&s_full[slot], (unsigned)((it / STAGES) & 1), &s_abort, st.status);
        ok = __syncthreads_and(mine) != 0;        // either every thread goes on or all leave together
        if (!ok) break;
        const int r = r0 + it * kBulkRows + warp;
        if (r < r1) {
            const float* si = s_stage + (size_t)slot * 2 * kBulkRows * ld + (size_t)warp * ld;
            const float* sj = si + (size_t)kBulkRows * ld;
            float4 xi[NV], xj[NV];
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int col = (k * 32 + lane) * 4;
                if (col < ld) {
                    xi[k] = *reinterpret_cast<const float4*>(si + col);
                    xj[k] = *reinterpret_cast<const float4*>(sj + col);
                } else {
                    xi[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                    xj[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
            if (UPDATE) {
                float ai[D], aj[D];
#pragma unroll
                for (int s2 = 0; s2 < D; ++s2) {
                    ai[s2] = pi.ph[s2] ? pi.coef[s2] * __ldg(pi.ph[s2] + r) : 0.0f;
                    aj[s2] = pj.ph[s2] ? pj.coef[s2] * __ldg(pj.ph[s2] + r) : 0.0f;
                }
                float* rowi = Xi_w + (long long)r * ld;
                float* rowj = Xj_w + (long long)r * ld;
#pragma unroll
                for (int k = 0; k < NV; ++k) {
                    const int col = (k * 32 + lane) * 4;
#pragma unroll
                    for (int s2 = 0; s2 < D; ++s2) {      // slot order, as the row sweep applies them
                        const float4 vi = *reinterpret_cast<const float4*>(&s_ui[s2][col]);
                        const float4 vj = *reinterpret_cast<const float4*>(&s_uj[s2][col]);
                        xi[k].x = fmaf(-ai[s2], vi.x, xi[k].x); xi[k].y = fmaf(-ai[s2], vi.y, xi[k].y);
                        xi[k].z = fmaf(-ai[s2], vi.z, xi[k].z); xi[k].w = fmaf(-ai[s2], vi.w, xi[k].w);
                        xj[k].x = fmaf(-aj[s2], vj.x, xj[k].x); xj[k].y = fmaf(-aj[s2], vj.y, xj[k].y);
                        xj[k].z = fmaf(-aj[s2], vj.z, xj[k].z); xj[k].w = fmaf(-aj[s2], vj.w, xj[k].w);
                    }
                    if (col < ld) {
                        if (own_i) st_stream(rowi + col, xi[k]);
                        if (own_j) st_stream(rowj + col, xj[k]);
                    }
                }
            }
            float dot = 0.0f;
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                const int col = (k * 32 + lane) * 4;
                const float4 vq = *reinterpret_cast<const float4*>(&s_q[col]);
                xi[k].x -= xj[k].x; xi[k].y -= xj[k].y; xi[k].z -= xj[k].z; xi[k].w -= xj[k].w;
                dot = fmaf(xi[k].x, vq.x, dot); dot = fmaf(xi[k].y, vq.y, dot);
                dot = fmaf(xi[k].z, vq.z, dot); dot = fmaf(xi[k].w, vq.w, dot);
            }
            const float p = warp_sum(dot);
#pragma unroll
            for (int k = 0; k < NV; ++k) {
                u[k].x = fmaf(p, xi[k].x, u[k].x); u[k].y = fmaf(p, xi[k].y, u[k].y);
                u[k].z = fmaf(p, xi[k].z, u[k].z); u[k].w = fmaf(p, xi[k].w, u[k].w);
            }
            ssum = fmaf(p, p, ssum);
            if (lane == 0) Pw[r] = p;
        }
        __syncthreads();          // every warp is done with this slot before it is filled again
    }
    if (!ok) {
        // leave only after the copies still in flight have landed (bounded)
        if (threadIdx.x == 0)
            for (int sidx = 0; sidx < issued; ++sidx) {
                const int slot = sidx % STAGES;
                for (int spin = 0; spin < kBulkSpinLimit; ++spin)
                    if (mbar_try_wait(&s_full[slot], (unsigned)((sidx / STAGES) & 1))) break;
            }
        return;
    }
    // the stage buffers are free now: reduce u across the warps through them
    float* s_red = s_stage;                                  // [8][NV*128]
#pragma unroll
    for (int k = 0; k < NV; ++k) *reinterpret_cast<float4*>(&s_red[warp * NV * 128 + (k * 32 + lane) * 4]) = u[k];
    if (lane == 0) s_s[warp] = (double)ssum;
    __syncthreads();
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld;
    for (int idx = threadIdx.x; idx < ld; idx += 256) {
        float t = s_red[idx];
#pragma unroll
        for (int w8 = 1; w8 < 8; ++w8) t += s_red[w8 * NV * 128 + idx];
        Up[idx] = t;
    }
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w8 = 0; w8 < 8; ++w8) t += s_s[w8];
        st.Sp[(long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile] = t;
    }
}

// --------------------------------------------------------------------------
// Pair sweep for rows too long for one warp: a cluster of kPairCluster CTAs
// shares every row.  CTA `rank` owns the columns [rank*slice, (rank+1)*slice):
// it keeps that slice of the three vectors in shared memory for the whole tile
// and its slice of the rows in flight in registers.  The row products
// p_r = D_r . q-hat need all columns, so every CTA writes its share into the
// shared memory of all CTAs of the cluster (distributed shared memory) and a
// cluster barrier makes them visible; the shares are added in rank order, so
// every CTA gets the same bits.  Each thread then adds p_r D_r to the columns it
// owns: no reduction is needed for u.  The barrier is split (arrive ... wait)
// and the loads of the next rows are issued in between.
// --------------------------------------------------------------------------
template <int NVW, bool UPDATE, int D>
__global__ void __cluster_dims__(kPairCluster, 1, 1) __launch_bounds__(256, kPairWideMinBlocks)
pair_sweep_wide_kernel(DevState st, const int* __restrict__ tab_prev, const int* __restrict__ tab_cur,
                       const Tile* __restrict__ tiles, int slice_pad) {
    grid_dependency_sync();
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) float s_vec[];               // slices of q-hat, D x u_i, D x u_j
    __shared__ __align__(16) float s_share[2][kPairCluster][kPairWideStep];    // [parity][rank][row]
    __shared__ float s_warp[8][kPairWideStep];
    __shared__ __align__(8) unsigned long long s_arrived[2];     // one mbarrier per parity: counts the shares' bytes
    __shared__ int s_gave_up;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();

    const Tile tile = tiles[blockIdx.x / kPairCluster];
    const int e = tile.worker;
    if (e >= tab_cur[st.tab.off_n_edges]) return;                // the same for the whole cluster
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab_cur[st.tab.off_edge_i + e], wj = tab_cur[st.tab.off_edge_j + e];
    const int pair = tab_cur[st.tab.off_pair + e];
    float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;
    const int c_begin = rank * g.p_slice;
    const int c_end = min(ld, c_begin + g.p_slice);

    float* s_q = s_vec;
    float* s_ui = s_vec + slice_pad;                  // [D][slice_pad]
    float* s_uj = s_vec + (1 + D) * slice_pad;        // [D][slice_pad]
    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv = pair_qinv(st, pair, tile.layer);
    // only the edge that owns a worker's rows writes them back (to Xw, which is X itself
    // unless rows have a second reader; on a matching every edge owns both of its ends)
    // (with one slot per worker every edge owns both ends and the rows are corrected in place: known at compile time)
    const int own = D == 1 ? 3 : tab_cur[st.tab.off_own + e];
    const bool own_i = D == 1 || (own & 1) != 0, own_j = D == 1 || (own & 2) != 0;
    float* Xi_w = D == 1 ? const_cast<float*>(Xi) : st.Xw + (long long)wi * st.x_stride + g.x_off;
    float* Xj_w = D == 1 ? const_cast<float*>(Xj) : st.Xw + (long long)wj * st.x_stride + g.x_off;
    PendingEnd<D> pi, pj;
    if (UPDATE) {
        pending_of<D>(st, tab_prev, wi, g, q, pi);
        pending_of<D>(st, tab_prev, wj, g, q, pj);
    }
    if (threadIdx.x == 0) {
        s_gave_up = 0;
        mbar_init(&s_arrived[0], 1);
        mbar_init(&s_arrived[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int idx = threadIdx.x; idx < slice_pad; idx += 256) {
        const int col = c_begin + idx;
        const bool in = col < c_end;
        s_q[idx] = in ? q[col] * qinv : 0.0f;
        if (UPDATE) {
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                s_ui[s2 * slice_pad + idx] = in ? pi.vec[s2][col] : 0.0f;
                s_uj[s2 * slice_pad + idx] = in ? pj.vec[s2][col] : 0.0f;
            }
        }
    }
    cluster.sync();      // every CTA's mbarriers exist before a peer signals them

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    // (checked build; after the cluster's barrier, so that a CTA that backs out leaves no peer waiting for
    //  its mbarriers to exist - the whole cluster sees the same tile and backs out together)
    if (pair_tile_out_of_bounds(st, g, Xi, Xj, Xi_w, Xj_w, r0, r1, q, Pw,
                                st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld, ld,
                                st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile) ||
        (UPDATE && (pending_out_of_bounds<D>(st, g, pi, r0, r1) || pending_out_of_bounds<D>(st, g, pj, r0, r1))))
        return;
    constexpr int RS = kPairWideStep;
    float4 u[NVW];
#pragma unroll
    for (int k = 0; k < NVW; ++k) u[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    float ssum = 0.0f;

    // rows r .. r+RS-1 of both ends, this CTA's slice; rows past the tile read as zero
    float4 xi[RS][NVW], xj[RS][NVW];
    auto load_rows = [&](int r) {
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            const bool in_row = r + t < r1;
            const long long base = (long long)(in_row ? r + t : r1 - 1) * ld + c_begin;
#pragma unroll
            for (int k = 0; k < NVW; ++k) {
                const int off = (k * 256 + threadIdx.x) * 4;
                if (in_row && c_begin + off < c_end) {
                    xi[t][k] = ld_stream(Xi + base + off);
                    xj[t][k] = ld_stream(Xj + base + off);
                } else {
                    xi[t][k] = make_float4(0.f, 0.f, 0.f, 0.f);
                    xj[t][k] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
    };
    load_rows(r0);
    int it = 0;
    for (int r = r0; r < r1; r += RS, ++it) {
        float4 d[RS][NVW];        // this CTA's slice of RS rows of D
        float dot[RS];
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            dot[t] = 0.0f;
            const bool in_row = r + t < r1;
            const long long base = (long long)(in_row ? r + t : r1 - 1) * ld + c_begin;
            float ai[D], aj[D];
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                ai[s2] = (UPDATE && in_row && pi.ph[s2]) ? pi.coef[s2] * __ldg(pi.ph[s2] + r + t) : 0.0f;
                aj[s2] = (UPDATE && in_row && pj.ph[s2]) ? pj.coef[s2] * __ldg(pj.ph[s2] + r + t) : 0.0f;
            }
#pragma unroll
            for (int k = 0; k < NVW; ++k) {
                const int off = (k * 256 + threadIdx.x) * 4;
                const bool in = in_row && c_begin + off < c_end;
                if (UPDATE && in) {
#pragma unroll
                    for (int s2 = 0; s2 < D; ++s2) {      // slot order, as the row sweep applies them
                        const float4 vi = *reinterpret_cast<const float4*>(&s_ui[s2 * slice_pad + off]);
                        const float4 vj = *reinterpret_cast<const float4*>(&s_uj[s2 * slice_pad + off]);
                        xi[t][k].x = fmaf(-ai[s2], vi.x, xi[t][k].x); xi[t][k].y = fmaf(-ai[s2], vi.y, xi[t][k].y);
                        xi[t][k].z = fmaf(-ai[s2], vi.z, xi[t][k].z); xi[t][k].w = fmaf(-ai[s2], vi.w, xi[t][k].w);
                        xj[t][k].x = fmaf(-aj[s2], vj.x, xj[t][k].x); xj[t][k].y = fmaf(-aj[s2], vj.y, xj[t][k].y);
                        xj[t][k].z = fmaf(-aj[s2], vj.z, xj[t][k].z); xj[t][k].w = fmaf(-aj[s2], vj.w, xj[t][k].w);
                    }
                    if (own_i) st_stream(Xi_w + base + off, xi[t][k]);
                    if (own_j) st_stream(Xj_w + base + off, xj[t][k]);
                }
                d[t][k].x = xi[t][k].x - xj[t][k].x; d[t][k].y = xi[t][k].y - xj[t][k].y;
                d[t][k].z = xi[t][k].z - xj[t][k].z; d[t][k].w = xi[t][k].w - xj[t][k].w;
                if (in) {
                    const float4 vq = *reinterpret_cast<const float4*>(&s_q[off]);
                    dot[t] = fmaf(d[t][k].x, vq.x, dot[t]); dot[t] = fmaf(d[t][k].y, vq.y, dot[t]);
                    dot[t] = fmaf(d[t][k].z, vq.z, dot[t]); dot[t] = fmaf(d[t][k].w, vq.w, dot[t]);
                }
            }
        }
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            dot[t] = warp_sum(dot[t]);
            if (lane == 0) s_warp[warp][t] = dot[t];
        }
        __syncthreads();
        // Data-flow exchange instead of a cluster-wide barrier: this CTA expects the
        // RS floats of every rank on its own mbarrier of this parity, and sends its share
        // to every rank (itself included) with a store that completes the receiver's count.
        if (threadIdx.x == 0) mbar_expect_tx(&s_arrived[it & 1], (unsigned)(kPairCluster * RS * sizeof(float)));
        if (threadIdx.x < RS * kPairCluster) {
            const int dst = threadIdx.x / RS, t = threadIdx.x % RS;
            float share = 0.0f;
#pragma unroll
            for (int w8 = 0; w8 < 8; ++w8) share += s_warp[w8][t];
            unsigned remote_data, remote_bar;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote_data)
                         : "r"(smem_addr(&s_share[it & 1][rank][t])), "r"(dst));
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote_bar)
                         : "r"(smem_addr(&s_arrived[it & 1])), "r"(dst));
            asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                         ::"r"(remote_data), "r"(__float_as_uint(share)), "r"(remote_bar) : "memory");
        }
        if (r + RS < r1) load_rows(r + RS);      // the next rows' loads are in flight during the wait
        // bounded wait; a CTA that gives up keeps going (its peers still need its shares)
        if (!s_gave_up)
            mbar_wait_bounded(&s_arrived[it & 1], (unsigned)((it >> 1) & 1), &s_gave_up, st.status);
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            float p = 0.0f;
#pragma unroll
            for (int rk = 0; rk < kPairCluster; ++rk) p += s_share[it & 1][rk][t];
#pragma unroll
            for (int k = 0; k < NVW; ++k) {
                u[k].x = fmaf(p, d[t][k].x, u[k].x); u[k].y = fmaf(p, d[t][k].y, u[k].y);
                u[k].z = fmaf(p, d[t][k].z, u[k].z); u[k].w = fmaf(p, d[t][k].w, u[k].w);
            }
            ssum = fmaf(p, p, ssum);
            if (rank == 0 && threadIdx.x == 0 && r + t < r1) Pw[r + t] = p;
        }
    }
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld + c_begin;
#pragma unroll
    for (int k = 0; k < NVW; ++k) {
        const int off = (k * 256 + threadIdx.x) * 4;
        if (c_begin + off < c_end) *reinterpret_cast<float4*>(Up + off) = u[k];
    }
    if (rank == 0 && threadIdx.x == 0)
        st.Sp[(long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile] = (double)ssum;
    cluster.sync();              // nobody leaves while a peer could still address its shared memory
}

// --------------------------------------------------------------------------
// Pair sweep for rows of up to kPairMidMaxLd floats: a CTA shares every row.
// Thread t owns the columns 4*(k*256 + t) .. +3 for k < NVM of every row, keeps
// them in registers and adds p_r D_r to its own columns of u, so u needs no
// reduction.  The row product p_r is the sum of the eight warps' shares, added
// in warp order by every thread; one barrier per row, with the next row's loads
// issued before it.
// --------------------------------------------------------------------------
template <int NVM, bool UPDATE, int D>
__global__ void __launch_bounds__(256, (NVM <= 2 ? 3 : (NVM <= 5 ? 2 : 1)))
pair_sweep_mid_kernel(DevState st, const int* __restrict__ tab_prev, const int* __restrict__ tab_cur,
                      const Tile* __restrict__ tiles, int ld_pad) {
    grid_dependency_sync();
    extern __shared__ __align__(16) float s_vec[];               // q-hat, D x u_i, D x u_j; ld_pad floats each
    __shared__ float s_warp[2][8];

    const Tile tile = tiles[blockIdx.x];
    const int e = tile.worker;
    if (e >= tab_cur[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab_cur[st.tab.off_edge_i + e], wj = tab_cur[st.tab.off_edge_j + e];
    const int pair = tab_cur[st.tab.off_pair + e];
    const float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    const float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;

    float* s_q = s_vec;
    float* s_ui = s_vec + ld_pad;                     // [D][ld_pad]
    float* s_uj = s_vec + (1 + D) * ld_pad;           // [D][ld_pad]
    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv = pair_qinv(st, pair, tile.layer);
    // only the edge that owns a worker's rows writes them back (to Xw, which is X itself
    // unless rows have a second reader; on a matching every edge owns both of its ends)
    // (with one slot per worker every edge owns both ends and the rows are corrected in place: known at compile time)
    const int own = D == 1 ? 3 : tab_cur[st.tab.off_own + e];
    const bool own_i = D == 1 || (own & 1) != 0, own_j = D == 1 || (own & 2) != 0;
    float* Xi_w = D == 1 ? const_cast<float*>(Xi) : st.Xw + (long long)wi * st.x_stride + g.x_off;
    float* Xj_w = D == 1 ? const_cast<float*>(Xj) : st.Xw + (long long)wj * st.x_stride + g.x_off;
    PendingEnd<D> pi, pj;
    if (UPDATE) {
        pending_of<D>(st, tab_prev, wi, g, q, pi);
        pending_of<D>(st, tab_prev, wj, g, q, pj);
    }
    for (int idx = threadIdx.x; idx < ld_pad; idx += 256) {
        const bool in = idx < ld;
        s_q[idx] = in ? q[idx] * qinv : 0.0f;
        if (UPDATE) {
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                s_ui[s2 * ld_pad + idx] = in ? pi.vec[s2][idx] : 0.0f;
                s_uj[s2 * ld_pad + idx] = in ? pj.vec[s2][idx] : 0.0f;
            }
        }
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    if (pair_tile_out_of_bounds(st, g, Xi, Xj, Xi_w, Xj_w, r0, r1, q, Pw,
                                st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld, ld,
                                st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile) ||
        (UPDATE && (pending_out_of_bounds<D>(st, g, pi, r0, r1) || pending_out_of_bounds<D>(st, g, pj, r0, r1))))
        return;
    float4 u[NVM];
#pragma unroll
    for (int k = 0; k < NVM; ++k) u[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    float ssum = 0.0f;

    float4 xi[NVM], xj[NVM];
    auto load_row = [&](int r) {
        const long long base = (long long)r * ld;
#pragma unroll
        for (int k = 0; k < NVM; ++k) {
            const int off = (k * 256 + threadIdx.x) * 4;
            if (off < ld) {
                xi[k] = ld_stream(Xi + base + off);
                xj[k] = ld_stream(Xj + base + off);
            } else {
                xi[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                xj[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    };
    load_row(r0);
    int it = 0;
    for (int r = r0; r < r1; ++r, ++it) {
        float4 d[NVM];            // this thread's columns of row r of D
        float dot = 0.0f;
        const long long base = (long long)r * ld;
        float ai[D], aj[D];
#pragma unroll
        for (int s2 = 0; s2 < D; ++s2) {
            ai[s2] = (UPDATE && pi.ph[s2]) ? pi.coef[s2] * __ldg(pi.ph[s2] + r) : 0.0f;
            aj[s2] = (UPDATE && pj.ph[s2]) ? pj.coef[s2] * __ldg(pj.ph[s2] + r) : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < NVM; ++k) {
            const int off = (k * 256 + threadIdx.x) * 4;
            const bool in = off < ld;
            if (UPDATE && in) {
#pragma unroll
                for (int s2 = 0; s2 < D; ++s2) {      // slot order, as the row sweep applies them
                    const float4 vi = *reinterpret_cast<const float4*>(&s_ui[s2 * ld_pad + off]);
                    const float4 vj = *reinterpret_cast<const float4*>(&s_uj[s2 * ld_pad + off]);
                    xi[k].x = fmaf(-ai[s2], vi.x, xi[k].x); xi[k].y = fmaf(-ai[s2], vi.y, xi[k].y);
                    xi[k].z = fmaf(-ai[s2], vi.z, xi[k].z); xi[k].w = fmaf(-ai[s2], vi.w, xi[k].w);
                    xj[k].x = fmaf(-aj[s2], vj.x, xj[k].x); xj[k].y = fmaf(-aj[s2], vj.y, xj[k].y);
                    xj[k].z = fmaf(-aj[s2], vj.z, xj[k].z); xj[k].w = fmaf(-aj[s2], vj.w, xj[k].w);
                }
                if (own_i) st_stream(Xi_w + base + off, xi[k]);
                if (own_j) st_stream(Xj_w + base + off, xj[k]);
            }
            d[k].x = xi[k].x - xj[k].x; d[k].y = xi[k].y - xj[k].y;
            d[k].z = xi[k].z - xj[k].z; d[k].w = xi[k].w - xj[k].w;
            if (in) {
                const float4 vq = *reinterpret_cast<const float4*>(&s_q[off]);
                dot = fmaf(d[k].x, vq.x, dot); dot = fmaf(d[k].y, vq.y, dot);
                dot = fmaf(d[k].z, vq.z, dot); dot = fmaf(d[k].w, vq.w, dot);
            }
        }
        dot = warp_sum(dot);
        if (lane == 0) s_warp[it & 1][warp] = dot;
        if (r + 1 < r1) load_row(r + 1);          // in flight across the barrier
        __syncthreads();
        // the buffer of this parity is written again two rows on, after the next barrier
        float p = 0.0f;
#pragma unroll
        for (int w8 = 0; w8 < 8; ++w8) p += s_warp[it & 1][w8];
#pragma unroll
        for (int k = 0; k < NVM; ++k) {
            u[k].x = fmaf(p, d[k].x, u[k].x); u[k].y = fmaf(p, d[k].y, u[k].y);
            u[k].z = fmaf(p, d[k].z, u[k].z); u[k].w = fmaf(p, d[k].w, u[k].w);
        }
        ssum = fmaf(p, p, ssum);
        if (threadIdx.x == 0) Pw[r] = p;
    }
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld;
#pragma unroll
    for (int k = 0; k < NVM; ++k) {
        const int off = (k * 256 + threadIdx.x) * 4;
        if (off < ld) *reinterpret_cast<float4*>(Up + off) = u[k];
    }
    if (threadIdx.x == 0) st.Sp[(long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile] = (double)ssum;
}

// --------------------------------------------------------------------------
// The same CTA-per-row sweep fed by bulk asynchronous copies (TMA), for rows of
// up to kMidBulkNv * 1024 floats.  One thread moves kMidRows consecutive rows of
// X_i and of X_j (contiguous in memory) into a shared-memory stage with two
// cp.async.bulk copies, n_stage stages ahead of the arithmetic; an mbarrier per
// stage counts the bytes.  A thread always works on the same columns, so it keeps
// its part of q-hat and of the pending corrections' vectors in registers and
// shared memory holds nothing but rows in flight.  The barrier that publishes
// the warps' shares of the row products also tells that every thread has taken
// its columns out of the stage, so the stage is refilled right after it.  Waits
// are bounded as in the row-per-warp variant; a wait that runs out ends the CTA
// at the next barrier.
// --------------------------------------------------------------------------
constexpr int kMidStagesMax = 4;
constexpr int kMidBulkNv = 5;     // most float4 per thread and row (registers)
// rows per stage and per barrier: more of them where a row is short
__host__ __device__ constexpr int mid_rows(int nvm) { return nvm <= 2 ? 4 : 2; }
// two CTAs per SM where the registers allow it, so one CTA's prologue hides behind the other's rows
__host__ __device__ constexpr int mid_min_blocks(int nvm, int d) { return (1 + 2 * d) * nvm <= 10 ? 2 : 1; }

// RAW (graphs where a row has two readers; see raw_terms): the rows enter the products
// as stored and the pending terms as one scalar per row; only the CTA that owns a worker
// corrects and writes its rows, and the thread keeps in registers the pending vectors of
// just the ENDS (1 or 2) ends this CTA may own.  The per-row scalars (that correction of
// p_r, the coefficients of the owned rows' corrections, and p_r itself for the terms'
// products at the end) sit in shared memory behind the stages, `rows_pad` floats each.
template <int NVM, bool UPDATE, int D, bool RAW, int ENDS>
__global__ void __launch_bounds__(256, mid_min_blocks(NVM, RAW ? (ENDS * D + 1) / 2 : D))
pair_sweep_mid_bulk_kernel(DevState st, const int* __restrict__ tab_prev, const int* __restrict__ tab_cur,
                           const Tile* __restrict__ tiles, int ld_pad, int n_stage, int rows_pad) {
    grid_dependency_sync();
    extern __shared__ __align__(128) float s_stage[];            // [slot][matrix][RS * ld_pad], then the scalars
    __shared__ __align__(8) unsigned long long s_full[kMidStagesMax];
    constexpr int RS = mid_rows(NVM);
    __shared__ float s_warp[2][RS][8];
    __shared__ double s_red[8 * kMaxTerms + kMaxTerms];
    __shared__ const float* s_tph[kMaxTerms];
    __shared__ int s_abort;

    const Tile tile = tiles[blockIdx.x];
    const int e = tile.worker;
    if (e >= tab_cur[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab_cur[st.tab.off_edge_i + e], wj = tab_cur[st.tab.off_edge_j + e];
    const int pair = tab_cur[st.tab.off_pair + e];
    const float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    const float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;
    const unsigned row_bytes = (unsigned)ld * 4u;     // multiple of 16: ld is a multiple of 4

    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv = pair_qinv(st, pair, tile.layer);
    // which ends' rows this CTA writes back (to Xw, which is X itself unless rows have several readers),
    // and which it corrects: all that it forms the difference from, or only the ones it writes
    // (with one slot per worker every edge owns both ends and the rows are corrected in place: known at compile time)
    const int own = !UPDATE ? 0 : (D == 1 ? 3 : tab_cur[st.tab.off_own + e]);
    const bool st_i = UPDATE && (D == 1 || (own & 1) != 0), st_j = UPDATE && (D == 1 || (own & 2) != 0);
    const bool act_i = UPDATE && (!RAW || st_i), act_j = UPDATE && (!RAW || st_j);
    float* Xi_w = D == 1 ? const_cast<float*>(Xi) : st.Xw + (long long)wi * st.x_stride + g.x_off;
    float* Xj_w = D == 1 ? const_cast<float*>(Xj) : st.Xw + (long long)wj * st.x_stride + g.x_off;
    // ENDS == 1: the vectors of the one end this CTA corrects (worker j if `one_is_j`)
    const bool one_is_j = ENDS == 1 && !act_i;
    const bool act_a = ENDS == 1 ? (act_i || act_j) : act_i;     // the end whose vectors are in va
    PendingEnd<D> pa, pb;
    if (UPDATE) {
        pending_of<D>(st, tab_prev, one_is_j ? wj : wi, g, q, pa);
        if (ENDS == 2) pending_of<D>(st, tab_prev, wj, g, q, pb);
    }
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    const int n_iter = (r1 - r0 + RS - 1) / RS;
    // per-row scalars behind the stages (RAW only)
    float* s_corr = s_stage + (size_t)n_stage * 2 * RS * ld_pad;
    float* s_p = s_corr + rows_pad;
    float* s_ca = s_p + rows_pad;                     // [D][rows_pad]: coefficients of end a's corrections
    float* s_cb = s_ca + (size_t)D * rows_pad;        // [D][rows_pad]: end b's (ENDS == 2)
    if (pair_tile_out_of_bounds(st, g, Xi, Xj, Xi_w, Xj_w, r0, r1, q, st.PhNext + (long long)e * st.ph_stride + g.ph_off,
                                st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld, ld,
                                st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile) ||
        (UPDATE && (pending_out_of_bounds<D>(st, g, pa, r0, r1) ||
                    (ENDS == 2 && pending_out_of_bounds<D>(st, g, pb, r0, r1)))) ||
        (RAW && r1 - r0 > rows_pad))
        return;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s2 = 0; s2 < n_stage; ++s2) mbar_init(&s_full[s2], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int idx) {       // rows r0 + idx*RS ... into slot idx % n_stage
        const int slot = idx % n_stage;
        const int row = r0 + idx * RS;
        const unsigned bytes = (unsigned)min(RS, r1 - row) * row_bytes;
        float* dst = s_stage + (size_t)slot * 2 * RS * ld_pad;
        mbar_expect_tx(&s_full[slot], 2 * bytes);
        bulk_load(dst, Xi + (long long)row * ld, bytes, &s_full[slot]);
        bulk_load(dst + (size_t)RS * ld_pad, Xj + (long long)row * ld, bytes, &s_full[slot]);
    };
    int issued = 0;
    if (threadIdx.x == 0)
        for (; issued < n_stage && issued < n_iter; ++issued) issue(issued);

    // while the first rows are on their way: the pending terms of this edge and the scalars of the tile's rows
    int nt = 0;
    if (RAW && UPDATE) {
        nt = raw_prologue(st, tab_prev, e, wi, wj, g, q, qinv, r0, r1, s_corr, s_tph, s_red);
        for (int r = r0 + threadIdx.x; r < r1; r += 256) {
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                s_ca[s2 * rows_pad + r - r0] = (act_a && pa.ph[s2]) ? pa.coef[s2] * __ldg(pa.ph[s2] + r) : 0.0f;
                if (ENDS == 2) s_cb[s2 * rows_pad + r - r0] = (act_j && pb.ph[s2]) ? pb.coef[s2] * __ldg(pb.ph[s2] + r) : 0.0f;
            }
        }
        __syncthreads();
    }

    // this thread's columns of the vectors, for the whole tile
    float4 vq[NVM], va[D][NVM], vb[ENDS == 2 ? D : 1][ENDS == 2 ? NVM : 1];
#pragma unroll
    for (int k = 0; k < NVM; ++k) {
        const int off = (k * 256 + threadIdx.x) * 4;
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
        vq[k] = zero;
        if (off < ld) {
            vq[k] = *reinterpret_cast<const float4*>(q + off);
            vq[k].x *= qinv; vq[k].y *= qinv; vq[k].z *= qinv; vq[k].w *= qinv;
        }
#pragma unroll
        for (int s2 = 0; s2 < D; ++s2) {
            va[s2][k] = (act_a && off < ld) ? *reinterpret_cast<const float4*>(pa.vec[s2] + off) : zero;
            if (ENDS == 2) vb[s2][k] = (act_j && off < ld) ? *reinterpret_cast<const float4*>(pb.vec[s2] + off) : zero;
        }
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    float4 u[NVM];
#pragma unroll
    for (int k = 0; k < NVM; ++k) u[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    float ssum = 0.0f;
    bool ok = true;

    for (int it = 0; it < n_iter; ++it) {
        const int r = r0 + it * RS;
        const int slot = it % n_stage;
        const bool mine = mbar_wait_bounded(&s_full[slot], (unsigned)((it / n_stage) & 1), &s_abort, st.status);
        const float* si = s_stage + (size_t)slot * 2 * RS * ld_pad;      // rows follow each other ld floats apart
        const float* sj = si + (size_t)RS * ld_pad;
        float4 d[RS][NVM];
        float dot[RS];
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            const bool in_row = mine && r + t < r1;
            const long long base = (long long)(r + t) * ld;
            dot[t] = 0.0f;
            float aa[D], ab[D];
#pragma unroll
            for (int s2 = 0; s2 < D; ++s2) {
                if (RAW) {
                    aa[s2] = (UPDATE && in_row) ? s_ca[s2 * rows_pad + r + t - r0] : 0.0f;
                    ab[s2] = (UPDATE && ENDS == 2 && in_row) ? s_cb[s2 * rows_pad + r + t - r0] : 0.0f;
                } else {
                    aa[s2] = (act_a && in_row && pa.ph[s2]) ? pa.coef[s2] * __ldg(pa.ph[s2] + r + t) : 0.0f;
                    ab[s2] = (act_j && in_row && pb.ph[s2]) ? pb.coef[s2] * __ldg(pb.ph[s2] + r + t) : 0.0f;
                }
            }
#pragma unroll
            for (int k = 0; k < NVM; ++k) {
                const int off = (k * 256 + threadIdx.x) * 4;
                const bool in = in_row && off < ld;
                float4 xi = make_float4(0.f, 0.f, 0.f, 0.f), xj = xi;
                if (in) {
                    xi = *reinterpret_cast<const float4*>(si + (size_t)t * ld + off);
                    xj = *reinterpret_cast<const float4*>(sj + (size_t)t * ld + off);
                }
                if (RAW) {   // the difference of the rows as stored; corrected rows only go back to memory
                    d[t][k].x = xi.x - xj.x; d[t][k].y = xi.y - xj.y; d[t][k].z = xi.z - xj.z; d[t][k].w = xi.w - xj.w;
                }
                if (UPDATE && in) {
                    if (ENDS == 1) {
                        if (act_a) {
                            float4 x = one_is_j ? xj : xi;
#pragma unroll
                            for (int s2 = 0; s2 < D; ++s2) {      // slot order, as the row sweep applies them
                                const float4 v = va[s2][k];
                                x.x = fmaf(-aa[s2], v.x, x.x); x.y = fmaf(-aa[s2], v.y, x.y);
                                x.z = fmaf(-aa[s2], v.z, x.z); x.w = fmaf(-aa[s2], v.w, x.w);
                            }
                            st_stream((one_is_j ? Xj_w : Xi_w) + base + off, x);
                        }
                    } else {
                        if (act_i) {
#pragma unroll
                            for (int s2 = 0; s2 < D; ++s2) {
                                const float4 v = va[s2][k];
                                xi.x = fmaf(-aa[s2], v.x, xi.x); xi.y = fmaf(-aa[s2], v.y, xi.y);
                                xi.z = fmaf(-aa[s2], v.z, xi.z); xi.w = fmaf(-aa[s2], v.w, xi.w);
                            }
                            if (st_i) st_stream(Xi_w + base + off, xi);
                        }
                        if (act_j) {
#pragma unroll
                            for (int s2 = 0; s2 < D; ++s2) {
                                xj.x = fmaf(-ab[s2], vb[s2][k].x, xj.x); xj.y = fmaf(-ab[s2], vb[s2][k].y, xj.y);
                                xj.z = fmaf(-ab[s2], vb[s2][k].z, xj.z); xj.w = fmaf(-ab[s2], vb[s2][k].w, xj.w);
                            }
                            if (st_j) st_stream(Xj_w + base + off, xj);
                        }
                    }
                }
                if (!RAW) {
                    d[t][k].x = xi.x - xj.x; d[t][k].y = xi.y - xj.y; d[t][k].z = xi.z - xj.z; d[t][k].w = xi.w - xj.w;
                }
                dot[t] = fmaf(d[t][k].x, vq[k].x, dot[t]); dot[t] = fmaf(d[t][k].y, vq[k].y, dot[t]);
                dot[t] = fmaf(d[t][k].z, vq[k].z, dot[t]); dot[t] = fmaf(d[t][k].w, vq[k].w, dot[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            dot[t] = warp_sum(dot[t]);
            if (lane == 0) s_warp[it & 1][t][warp] = dot[t];
        }
        ok = __syncthreads_and(mine) != 0;        // shares visible, stage drained; all go on or all leave
        if (!ok) break;
        if (threadIdx.x == 0 && it + n_stage < n_iter) {
            issue(it + n_stage);
            issued = it + n_stage + 1;
        }
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            float p = 0.0f;
#pragma unroll
            for (int w8 = 0; w8 < 8; ++w8) p += s_warp[it & 1][t][w8];
            if (RAW && UPDATE && r + t < r1) p -= s_corr[r + t - r0];
#pragma unroll
            for (int k = 0; k < NVM; ++k) {
                u[k].x = fmaf(p, d[t][k].x, u[k].x); u[k].y = fmaf(p, d[t][k].y, u[k].y);
                u[k].z = fmaf(p, d[t][k].z, u[k].z); u[k].w = fmaf(p, d[t][k].w, u[k].w);
            }
            if (r + t < r1) {
                ssum = fmaf(p, p, ssum);
                if (threadIdx.x == 0) {
                    Pw[r + t] = p;
                    if (RAW && UPDATE) s_p[r + t - r0] = p;
                }
            }
        }
    }
    if (!ok) {
        // leave only after the copies still in flight have landed (bounded)
        if (threadIdx.x == 0)
            for (int idx = 0; idx < issued; ++idx) {
                const int slot = idx % n_stage;
                for (int spin = 0; spin < kBulkSpinLimit; ++spin)
                    if (mbar_try_wait(&s_full[slot], (unsigned)((idx / n_stage) & 1))) break;
            }
        return;
    }
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * ld;
#pragma unroll
    for (int k = 0; k < NVM; ++k) {
        const int off = (k * 256 + threadIdx.x) * 4;
        if (off < ld) *reinterpret_cast<float4*>(Up + off) = u[k];
    }
    double* sp = st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile;
    if (threadIdx.x == 0) sp[0] = (double)ssum;
    if (RAW) {
        // this tile's share of p-hat_k . p for every pending term: warp k adds it up in row order
        __syncthreads();          // s_p complete
        if (warp < kMaxTerms) {
            double a = 0.0;
            if (warp < nt)
                for (int r = r0 + lane; r < r1; r += 32) a += (double)s_p[r - r0] * (double)__ldg(s_tph[warp] + r);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) sp[4 + warp] = a;
        }
    }
}

// --------------------------------------------------------------------------
// Rank 2 on a static graph of degree <= 2 (a ring, a path): the CTA-per-row sweep
// with two columns.  For an edge (i<j) one pass over the rows of X_i and X_j gives
//   P = D [q-hat_0 q-hat_1]   (rows x 2)      and      U = D^T P   (cols x 2),
// and the pair edge step orthonormalises afterwards:  P-hat = P T,  Q' = D^T P-hat
// = U T  with the 2 x 2 triangular T of the Gram-Schmidt step, taken from P^T P.
// The graph is static, so the corrections still pending at a worker belong to its
// current edges, and the vector of a pending correction of this edge is the edge's
// stored Q itself (what q-hat is scaled from): a thread keeps its columns (float4
// number k * 384 + thread of a row) of three vector pairs in registers - this edge's
// and the other edge's of either end.
// Corrections are applied in slot order, columns within a slot in order, as the
// row sweep applies them; the edge in a worker's slot 0 writes the corrected row to
// the second copy of the stack.  Rows arrive as in the rank-1 kernel above.
// --------------------------------------------------------------------------
// 384 threads (12 warps) a CTA: with 256 the two-column arithmetic of a row is latency-bound
// (VGG-shaped ring, rank 2: 1.24 -> 1.13 ms per round); rows of up to 4 x 384 float4.
constexpr int kMid2Threads = 384;
__host__ __device__ constexpr int mid2_rows(int nvm) { return nvm <= 3 ? 2 : 1; }

// a - b (as fma(b, -1, a): the same rounding as the subtraction)
__device__ __forceinline__ float4 sub4(const float4& a, const float4& b) {
    const unsigned long long m = pack2(-1.0f, -1.0f);
    float4 d;
    unpack2(fma2(pack2(b.x, b.y), m, pack2(a.x, a.y)), d.x, d.y);
    unpack2(fma2(pack2(b.z, b.w), m, pack2(a.z, a.w)), d.z, d.w);
    return d;
}
template <int NVM, bool UPDATE>
__global__ void __launch_bounds__(kMid2Threads, 1)
pair_sweep_mid2_kernel(DevState st, const int* __restrict__ tab, const Tile* __restrict__ tiles, int ld_pad,
                       int n_stage) {
    grid_dependency_sync();
    constexpr int R = 2;
    constexpr int NT = kMid2Threads;
    constexpr int RS = mid2_rows(NVM);
    extern __shared__ __align__(128) float s_stage[];            // [slot][matrix][RS * ld_pad]
    __shared__ __align__(8) unsigned long long s_full[kMidStagesMax];
    __shared__ float s_warp[2][RS][R][NT / 32];
    __shared__ int s_abort;

    const Tile tile = tiles[blockIdx.x];
    const int e = tile.worker;
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int pair = tab[st.tab.off_pair + e];
    const float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    const float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    float* Xi_w = st.Xw + (long long)wi * st.x_stride + g.x_off;
    float* Xj_w = st.Xw + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;
    const unsigned row_bytes = (unsigned)ld * 4u;     // multiple of 16: ld is a multiple of 4
    const int md = st.tab.max_degree;

    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv0 = pair_qinv(st, pair, tile.layer, 0), qinv1 = pair_qinv(st, pair, tile.layer, 1);
    // slot of this edge at either end, and the other edge there (if the worker has two)
    const int si = tab[st.tab.off_slot_i + e], sj = tab[st.tab.off_slot_j + e];
    const bool two_i = tab[st.tab.off_degree + wi] > 1, two_j = tab[st.tab.off_degree + wj] > 1;
    const bool first_i = si == 0, first_j = sj == 0;  // slot order: is this edge's correction the first at that end
    const int own = tab[st.tab.off_own + e];          // the ends whose corrected rows this CTA writes
    const bool own_i = (own & 1) != 0, own_j = (own & 2) != 0;
    const float* ph_e = st.Ph + (long long)e * st.ph_stride + g.ph_off;
    const float* ph_oi = ph_e;
    const float* ph_oj = ph_e;
    const float* q_oi = q;
    const float* q_oj = q;
    float ce_i = 0.f, ce_j = 0.f, co_i = 0.f, co_j = 0.f;
    if (UPDATE) {
        ce_i = __int_as_float(tab[st.tab.off_slot_coef + wi * md + si]);
        ce_j = __int_as_float(tab[st.tab.off_slot_coef + wj * md + sj]);
        if (two_i) {
            const int eo = tab[st.tab.off_slot_edge + wi * md + (1 - si)];
            q_oi = st.Qr + (long long)tab[st.tab.off_pair + eo] * st.q_stride + g.q_off;
            ph_oi = st.Ph + (long long)eo * st.ph_stride + g.ph_off;
            co_i = __int_as_float(tab[st.tab.off_slot_coef + wi * md + (1 - si)]);
        }
        if (two_j) {
            const int eo = tab[st.tab.off_slot_edge + wj * md + (1 - sj)];
            q_oj = st.Qr + (long long)tab[st.tab.off_pair + eo] * st.q_stride + g.q_off;
            ph_oj = st.Ph + (long long)eo * st.ph_stride + g.ph_off;
            co_j = __int_as_float(tab[st.tab.off_slot_coef + wj * md + (1 - sj)]);
        }
    }
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    const int n_iter = (r1 - r0 + RS - 1) / RS;
    if (pair_tile_out_of_bounds(st, g, Xi, Xj, Xi_w, Xj_w, r0, r1, q, st.PhNext + (long long)e * st.ph_stride + g.ph_off,
                                st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * 2 * ld, 2 * ld,
                                st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile) ||
        (UPDATE && (PG_OOB(st, kSecQ, q_oi, 2LL * ld) || PG_OOB(st, kSecQ, q_oj, 2LL * ld))) ||
        (UPDATE && r1 > r0 && (PG_OOB(st, kSecPh, ph_e + g.npad + r0, r1 - r0) || PG_OOB(st, kSecPh, ph_oi + g.npad + r0, r1 - r0) ||
                               PG_OOB(st, kSecPh, ph_oj + g.npad + r0, r1 - r0) || PG_OOB(st, kSecPh, ph_e + r0, r1 - r0))))
        return;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s2 = 0; s2 < n_stage; ++s2) mbar_init(&s_full[s2], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int idx) {       // rows r0 + idx*RS ... into slot idx % n_stage
        const int slot = idx % n_stage;
        const int row = r0 + idx * RS;
        const unsigned bytes = (unsigned)min(RS, r1 - row) * row_bytes;
        float* dst = s_stage + (size_t)slot * 2 * RS * ld_pad;
        mbar_expect_tx(&s_full[slot], 2 * bytes);
        bulk_load(dst, Xi + (long long)row * ld, bytes, &s_full[slot]);
        bulk_load(dst + (size_t)RS * ld_pad, Xj + (long long)row * ld, bytes, &s_full[slot]);
    };
    int issued = 0;
    if (threadIdx.x == 0)
        for (; issued < n_stage && issued < n_iter; ++issued) issue(issued);

    // this thread's columns of the three vector pairs, for the whole tile
    float4 vq[R][NVM], vi[R][NVM], vj[R][NVM];
#pragma unroll
    for (int k = 0; k < NVM; ++k) {
        const int off = (k * NT + threadIdx.x) * 4;
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int c = 0; c < R; ++c) {
            vq[c][k] = off < ld ? *reinterpret_cast<const float4*>(q + (long long)c * ld + off) : zero;
            vi[c][k] = (UPDATE && two_i && off < ld) ? *reinterpret_cast<const float4*>(q_oi + (long long)c * ld + off) : zero;
            vj[c][k] = (UPDATE && two_j && off < ld) ? *reinterpret_cast<const float4*>(q_oj + (long long)c * ld + off) : zero;
        }
    }

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    float4 u[R][NVM];
#pragma unroll
    for (int c = 0; c < R; ++c)
#pragma unroll
        for (int k = 0; k < NVM; ++k) u[c][k] = make_float4(0.f, 0.f, 0.f, 0.f);
    double g00 = 0.0, g01 = 0.0, g11 = 0.0;       // this tile's share of P^T P (thread 0)
    bool ok = true;

    for (int it = 0; it < n_iter; ++it) {
        const int r = r0 + it * RS;
        const int slot = it % n_stage;
        const bool mine = mbar_wait_bounded(&s_full[slot], (unsigned)((it / n_stage) & 1), &s_abort, st.status);
        const float* si_rows = s_stage + (size_t)slot * 2 * RS * ld_pad;      // rows follow each other ld floats apart
        const float* sj_rows = si_rows + (size_t)RS * ld_pad;
        float4 d[RS][NVM];
        float2 dot[RS][R];      // even and odd columns apart until the warp's sum
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            const bool in_row = mine && r + t < r1;
            const long long base = (long long)(r + t) * ld;
            dot[t][0] = dot[t][1] = make_float2(0.f, 0.f);
            // coefficients of the pending corrections of this row: this edge's and the other edge's, per column
            float ae_i[R], ae_j[R], ao_i[R], ao_j[R];
#pragma unroll
            for (int c = 0; c < R; ++c) {
                const bool on = UPDATE && in_row;
                ae_i[c] = on ? -ce_i * __ldg(ph_e + (long long)c * g.npad + r + t) : 0.0f;
                ae_j[c] = on ? -ce_j * __ldg(ph_e + (long long)c * g.npad + r + t) : 0.0f;
                ao_i[c] = (on && two_i) ? -co_i * __ldg(ph_oi + (long long)c * g.npad + r + t) : 0.0f;
                ao_j[c] = (on && two_j) ? -co_j * __ldg(ph_oj + (long long)c * g.npad + r + t) : 0.0f;
            }
#pragma unroll
            for (int k = 0; k < NVM; ++k) {
                const int off = (k * NT + threadIdx.x) * 4;
                const bool in = in_row && off < ld;
                float4 xi = make_float4(0.f, 0.f, 0.f, 0.f), xj = xi;
                if (in) {
                    xi = *reinterpret_cast<const float4*>(si_rows + (size_t)t * ld + off);
                    xj = *reinterpret_cast<const float4*>(sj_rows + (size_t)t * ld + off);
                }
                if (UPDATE && in) {
                    if (first_i) {     // this edge is in slot 0 of worker i: its correction first
                        fma4(xi, ae_i[0], vq[0][k]); fma4(xi, ae_i[1], vq[1][k]);
                        fma4(xi, ao_i[0], vi[0][k]); fma4(xi, ao_i[1], vi[1][k]);
                    } else {
                        fma4(xi, ao_i[0], vi[0][k]); fma4(xi, ao_i[1], vi[1][k]);
                        fma4(xi, ae_i[0], vq[0][k]); fma4(xi, ae_i[1], vq[1][k]);
                    }
                    if (own_i) st_stream(Xi_w + base + off, xi);
                    if (first_j) {
                        fma4(xj, ae_j[0], vq[0][k]); fma4(xj, ae_j[1], vq[1][k]);
                        fma4(xj, ao_j[0], vj[0][k]); fma4(xj, ao_j[1], vj[1][k]);
                    } else {
                        fma4(xj, ao_j[0], vj[0][k]); fma4(xj, ao_j[1], vj[1][k]);
                        fma4(xj, ae_j[0], vq[0][k]); fma4(xj, ae_j[1], vq[1][k]);
                    }
                    if (own_j) st_stream(Xj_w + base + off, xj);
                }
                d[t][k] = sub4(xi, xj);
#pragma unroll
                for (int c = 0; c < R; ++c) dot4(dot[t][c], d[t][k], vq[c][k]);
            }
        }
#pragma unroll
        for (int t = 0; t < RS; ++t)
#pragma unroll
            for (int c = 0; c < R; ++c) {
                const float sum = warp_sum(dot[t][c].x + dot[t][c].y);
                if (lane == 0) s_warp[it & 1][t][c][warp] = sum;
            }
        ok = __syncthreads_and(mine) != 0;        // shares visible, stage drained; all go on or all leave
        if (!ok) break;
        if (threadIdx.x == 0 && it + n_stage < n_iter) {
            issue(it + n_stage);
            issued = it + n_stage + 1;
        }
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            float p[R];
#pragma unroll
            for (int c = 0; c < R; ++c) {
                p[c] = 0.0f;
#pragma unroll
                for (int w8 = 0; w8 < NT / 32; ++w8) p[c] += s_warp[it & 1][t][c][w8];
            }
            p[0] *= qinv0;        // the products with the unit columns
            p[1] *= qinv1;
#pragma unroll
            for (int c = 0; c < R; ++c)
#pragma unroll
                for (int k = 0; k < NVM; ++k) fma4(u[c][k], p[c], d[t][k]);
            if (threadIdx.x == 0 && r + t < r1) {
                g00 += (double)p[0] * (double)p[0];
                g01 += (double)p[0] * (double)p[1];
                g11 += (double)p[1] * (double)p[1];
                Pw[r + t] = p[0];
                Pw[g.npad + r + t] = p[1];
            }
        }
    }
    if (!ok) {
        // leave only after the copies still in flight have landed (bounded)
        if (threadIdx.x == 0)
            for (int idx = 0; idx < issued; ++idx) {
                const int slot = idx % n_stage;
                for (int spin = 0; spin < kBulkSpinLimit; ++spin)
                    if (mbar_try_wait(&s_full[slot], (unsigned)((idx / n_stage) & 1))) break;
            }
        return;
    }
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * R * ld;
#pragma unroll
    for (int c = 0; c < R; ++c)
#pragma unroll
        for (int k = 0; k < NVM; ++k) {
            const int off = (k * NT + threadIdx.x) * 4;
            if (off < ld) *reinterpret_cast<float4*>(Up + (long long)c * ld + off) = u[c][k];
        }
    if (threadIdx.x == 0) {
        double* sp = st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile;
        sp[0] = g00;
        sp[1] = g01;
        sp[2] = g11;
    }
}

// The raw form of the rank-2 sweep (see raw_terms), for graphs in which no edge owns both of
// its ends, with corrections pending.  The rows enter P = D [q-hat_0 q-hat_1] and U = D^T P as
// stored; with D' = D - sum_k c_k (p-hat_{k,0} q'_{k,0}^T + p-hat_{k,1} q'_{k,1}^T) over the pending
// edges k,
//     P[r][c]   -= sum_{k,c'} c_k (q'_{k,c'} . q-hat_c) p-hat_{k,c'}[r]        (one scalar per row and column)
//     U[:, c]   -= sum_{k,c'} c_k (p-hat_{k,c'} . P[:, c]) q'_{k,c'}            (by the pair edge step)
// and only the CTA that owns a worker's rows applies its four pending rank-1 terms (slot order,
// columns in order) and writes the rows.  A thread keeps the columns of the edge's two vectors and
// of the owned end's four in registers; the per-row scalars sit behind the stages.
template <int NVM>
__global__ void __launch_bounds__(kMid2Threads, 1)
pair_sweep_mid2_raw_kernel(DevState st, const int* __restrict__ tab, const Tile* __restrict__ tiles, int ld_pad,
                           int n_stage, int rows_pad) {
    grid_dependency_sync();
    constexpr int R = 2;
    constexpr int NT = kMid2Threads;
    constexpr int RS = mid2_rows(NVM);
    constexpr int NB = kMaxTerms * R * R;      // products q'_{k,c'} . q-hat_c
    extern __shared__ __align__(128) float s_stage[];            // [slot][matrix][RS * ld_pad], then the scalars
    __shared__ __align__(8) unsigned long long s_full[kMidStagesMax];
    __shared__ float s_warp[2][RS][R][NT / 32];
    __shared__ double s_red[NT / 32][NB];
    __shared__ float s_beta[NB];                // c_k (q'_{k,c'} . q-hat_c), index (k * 2 + c') * 2 + c
    __shared__ const float* s_tph[kMaxTerms];
    __shared__ int s_abort;

    const Tile tile = tiles[blockIdx.x];
    const int e = tile.worker;
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[tile.layer];
    const int wi = tab[st.tab.off_edge_i + e], wj = tab[st.tab.off_edge_j + e];
    const int pair = tab[st.tab.off_pair + e];
    const float* __restrict__ Xi = st.X + (long long)wi * st.x_stride + g.x_off;
    const float* __restrict__ Xj = st.X + (long long)wj * st.x_stride + g.x_off;
    const int ld = g.ld;
    const unsigned row_bytes = (unsigned)ld * 4u;     // multiple of 16: ld is a multiple of 4
    const int md = st.tab.max_degree;

    const float* q = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const float qinv0 = pair_qinv(st, pair, tile.layer, 0), qinv1 = pair_qinv(st, pair, tile.layer, 1);
    // the end whose rows this CTA corrects and writes (if any), and its pending edges in slot order
    const int own = tab[st.tab.off_own + e];
    const bool act = own != 0;
    const bool own_j = (own & 1) == 0;
    const int wo = own_j ? wj : wi;
    float* Xo_w = st.Xw + (long long)wo * st.x_stride + g.x_off;
    const float* o_vec[2] = {q, q};
    const float* o_ph[2] = {nullptr, nullptr};
    float o_coef[2] = {0.f, 0.f};
    if (act) {
        const int deg = min(tab[st.tab.off_degree + wo], 2);
        for (int s2 = 0; s2 < deg; ++s2) {
            const int ep = tab[st.tab.off_slot_edge + wo * md + s2];
            o_vec[s2] = st.Qr + (long long)tab[st.tab.off_pair + ep] * st.q_stride + g.q_off;
            o_ph[s2] = st.Ph + (long long)ep * st.ph_stride + g.ph_off;
            o_coef[s2] = __int_as_float(tab[st.tab.off_slot_coef + wo * md + s2]);
        }
    }
    const int r0 = tile.rtile * g.p_rows;
    const int r1 = min(g.n, r0 + g.p_rows);
    const int n_iter = (r1 - r0 + RS - 1) / RS;
    // per-row scalars behind the stages
    float* s_corr = s_stage + (size_t)n_stage * 2 * RS * ld_pad;     // [R][rows_pad]
    float* s_p = s_corr + (size_t)R * rows_pad;                       // [R][rows_pad]
    float* s_oa = s_p + (size_t)R * rows_pad;                         // [2 slots][R][rows_pad]
    {
        bool bad = pair_tile_out_of_bounds(st, g, Xi, Xj, Xo_w, Xo_w, r0, r1, q,
                                           st.PhNext + (long long)e * st.ph_stride + g.ph_off,
                                           st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * 2 * ld,
                                           2 * ld, st.Sp + (long long)e * st.sp_stride + g.sp_off +
                                                       (long long)tile.rtile * kSpPerTile) ||
                   r1 - r0 > rows_pad;
        for (int s2 = 0; s2 < 2; ++s2)
            if (o_ph[s2] && r1 > r0)
                bad = PG_OOB(st, kSecQ, o_vec[s2], 2LL * ld) || PG_OOB(st, kSecPh, o_ph[s2] + r0, r1 - r0) ||
                      PG_OOB(st, kSecPh, o_ph[s2] + g.npad + r0, r1 - r0) || bad;
        if (bad) return;
    }

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s2 = 0; s2 < n_stage; ++s2) mbar_init(&s_full[s2], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int idx) {       // rows r0 + idx*RS ... into slot idx % n_stage
        const int slot = idx % n_stage;
        const int row = r0 + idx * RS;
        const unsigned bytes = (unsigned)min(RS, r1 - row) * row_bytes;
        float* dst = s_stage + (size_t)slot * 2 * RS * ld_pad;
        mbar_expect_tx(&s_full[slot], 2 * bytes);
        bulk_load(dst, Xi + (long long)row * ld, bytes, &s_full[slot]);
        bulk_load(dst + (size_t)RS * ld_pad, Xj + (long long)row * ld, bytes, &s_full[slot]);
    };
    int issued = 0;
    if (threadIdx.x == 0)
        for (; issued < n_stage && issued < n_iter; ++issued) issue(issued);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // while the first rows are on their way: the pending terms, their products with the unit columns ...
    RawTerm terms[kMaxTerms];
    const int nt = raw_terms(st, tab, e, wi, wj, terms);
    {
        double part[NB];
        const float* tv[kMaxTerms];
#pragma unroll
        for (int k = 0; k < kMaxTerms; ++k)
            tv[k] = k < nt ? st.Qr + (long long)tab[st.tab.off_pair + terms[k].edge] * st.q_stride + g.q_off : q;
#pragma unroll
        for (int b = 0; b < NB; ++b) part[b] = 0.0;
        for (int idx = threadIdx.x; idx < g.m; idx += NT) {
            const double qh0 = (double)(q[idx] * qinv0), qh1 = (double)(q[(long long)ld + idx] * qinv1);
#pragma unroll
            for (int k = 0; k < kMaxTerms; ++k)
                if (k < nt) {
#pragma unroll
                    for (int c2 = 0; c2 < R; ++c2) {
                        const double v = (double)tv[k][(long long)c2 * ld + idx];
                        part[(k * R + c2) * R + 0] += v * qh0;
                        part[(k * R + c2) * R + 1] += v * qh1;
                    }
                }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part[b] += __shfl_xor_sync(0xffffffffu, part[b], o);
            if (lane == 0) s_red[warp][b] = part[b];
        }
        __syncthreads();
        if (threadIdx.x < NB) {
            double t = 0.0;
            for (int w8 = 0; w8 < NT / 32; ++w8) t += s_red[w8][threadIdx.x];
            const int k = threadIdx.x / (R * R);
            s_beta[threadIdx.x] = k < nt ? (float)((double)terms[k].coef * t) : 0.0f;
        }
        if (threadIdx.x < kMaxTerms)
            s_tph[threadIdx.x] = st.Ph + (long long)(threadIdx.x < nt ? terms[threadIdx.x].edge : e) * st.ph_stride + g.ph_off;
        __syncthreads();
    }
    // ... and the scalars of the tile's rows: what the pending terms take from P[r][c], and the
    // coefficients of the owned rows' four corrections
    for (int r = r0 + threadIdx.x; r < r1; r += NT) {
        float c0 = 0.0f, c1 = 0.0f;
        for (int k = 0; k < nt; ++k)
#pragma unroll
            for (int c2 = 0; c2 < R; ++c2) {
                const float phv = __ldg(s_tph[k] + (long long)c2 * g.npad + r);
                c0 = fmaf(s_beta[(k * R + c2) * R + 0], phv, c0);
                c1 = fmaf(s_beta[(k * R + c2) * R + 1], phv, c1);
            }
        s_corr[r - r0] = c0;
        s_corr[rows_pad + r - r0] = c1;
#pragma unroll
        for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
            for (int c2 = 0; c2 < R; ++c2)
                s_oa[(size_t)(s2 * R + c2) * rows_pad + r - r0] =
                    o_ph[s2] ? -o_coef[s2] * __ldg(o_ph[s2] + (long long)c2 * g.npad + r) : 0.0f;
    }
    __syncthreads();

    // this thread's columns of the edge's two vectors and of the owned end's four, for the whole tile
    float4 vq[R][NVM], vo[2][R][NVM];
#pragma unroll
    for (int k = 0; k < NVM; ++k) {
        const int off = (k * NT + threadIdx.x) * 4;
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int c = 0; c < R; ++c) {
            vq[c][k] = off < ld ? *reinterpret_cast<const float4*>(q + (long long)c * ld + off) : zero;
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2)
                vo[s2][c][k] = (act && off < ld) ? *reinterpret_cast<const float4*>(o_vec[s2] + (long long)c * ld + off) : zero;
        }
    }

    float* __restrict__ Pw = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    float4 u[R][NVM];
#pragma unroll
    for (int c = 0; c < R; ++c)
#pragma unroll
        for (int k = 0; k < NVM; ++k) u[c][k] = make_float4(0.f, 0.f, 0.f, 0.f);
    double g00 = 0.0, g01 = 0.0, g11 = 0.0;       // this tile's share of P^T P (thread 0)
    bool ok = true;

    for (int it = 0; it < n_iter; ++it) {
        const int r = r0 + it * RS;
        const int slot = it % n_stage;
        const bool mine = mbar_wait_bounded(&s_full[slot], (unsigned)((it / n_stage) & 1), &s_abort, st.status);
        const float* si_rows = s_stage + (size_t)slot * 2 * RS * ld_pad;      // rows follow each other ld floats apart
        const float* sj_rows = si_rows + (size_t)RS * ld_pad;
        float4 d[RS][NVM];
        float2 dot[RS][R];      // even and odd columns apart until the warp's sum
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            const bool in_row = mine && r + t < r1;
            const long long base = (long long)(r + t) * ld;
            dot[t][0] = dot[t][1] = make_float2(0.f, 0.f);
            float oa[2][R];
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
                for (int c = 0; c < R; ++c)
                    oa[s2][c] = (act && in_row) ? s_oa[(size_t)(s2 * R + c) * rows_pad + r + t - r0] : 0.0f;
#pragma unroll
            for (int k = 0; k < NVM; ++k) {
                const int off = (k * NT + threadIdx.x) * 4;
                const bool in = in_row && off < ld;
                float4 xi = make_float4(0.f, 0.f, 0.f, 0.f), xj = xi;
                if (in) {
                    xi = *reinterpret_cast<const float4*>(si_rows + (size_t)t * ld + off);
                    xj = *reinterpret_cast<const float4*>(sj_rows + (size_t)t * ld + off);
                }
                d[t][k] = sub4(xi, xj);
                if (act && in) {
                    float4 x = own_j ? xj : xi;
                    fma4(x, oa[0][0], vo[0][0][k]); fma4(x, oa[0][1], vo[0][1][k]);
                    fma4(x, oa[1][0], vo[1][0][k]); fma4(x, oa[1][1], vo[1][1][k]);
                    st_stream(Xo_w + base + off, x);
                }
#pragma unroll
                for (int c = 0; c < R; ++c) dot4(dot[t][c], d[t][k], vq[c][k]);
            }
        }
#pragma unroll
        for (int t = 0; t < RS; ++t)
#pragma unroll
            for (int c = 0; c < R; ++c) {
                const float sum = warp_sum(dot[t][c].x + dot[t][c].y);
                if (lane == 0) s_warp[it & 1][t][c][warp] = sum;
            }
        ok = __syncthreads_and(mine) != 0;        // shares visible, stage drained; all go on or all leave
        if (!ok) break;
        if (threadIdx.x == 0 && it + n_stage < n_iter) {
            issue(it + n_stage);
            issued = it + n_stage + 1;
        }
        // the warps' shares of the RS x R row products: lane (t, c) of every warp adds one up in warp order,
        // the others take it from there
        float lane_sum = 0.0f;
        if (lane < RS * R) {
            const float* sh_w = &s_warp[it & 1][0][0][0] + lane * (NT / 32);
#pragma unroll
            for (int w8 = 0; w8 < NT / 32; ++w8) lane_sum += sh_w[w8];
        }
#pragma unroll
        for (int t = 0; t < RS; ++t) {
            float p[R];
#pragma unroll
            for (int c = 0; c < R; ++c) p[c] = __shfl_sync(0xffffffffu, lane_sum, t * R + c);
            const int rr = min(r + t, r1 - 1) - r0;
            p[0] = p[0] * qinv0 - s_corr[rr];        // the products with the unit columns, less the pending terms' part
            p[1] = p[1] * qinv1 - s_corr[rows_pad + rr];
#pragma unroll
            for (int c = 0; c < R; ++c)
#pragma unroll
                for (int k = 0; k < NVM; ++k) fma4(u[c][k], p[c], d[t][k]);
            if (threadIdx.x == 0 && r + t < r1) {
                g00 += (double)p[0] * (double)p[0];
                g01 += (double)p[0] * (double)p[1];
                g11 += (double)p[1] * (double)p[1];
                Pw[r + t] = p[0];
                Pw[g.npad + r + t] = p[1];
                s_p[rr] = p[0];
                s_p[rows_pad + rr] = p[1];
            }
        }
    }
    if (!ok) {
        // leave only after the copies still in flight have landed (bounded)
        if (threadIdx.x == 0)
            for (int idx = 0; idx < issued; ++idx) {
                const int slot = idx % n_stage;
                for (int spin = 0; spin < kBulkSpinLimit; ++spin)
                    if (mbar_try_wait(&s_full[slot], (unsigned)((idx / n_stage) & 1))) break;
            }
        return;
    }
    float* __restrict__ Up = st.Up + (long long)e * st.up_stride + g.up_off + (long long)tile.rtile * R * ld;
#pragma unroll
    for (int c = 0; c < R; ++c)
#pragma unroll
        for (int k = 0; k < NVM; ++k) {
            const int off = (k * NT + threadIdx.x) * 4;
            if (off < ld) *reinterpret_cast<float4*>(Up + (long long)c * ld + off) = u[c][k];
        }
    double* sp = st.Sp + (long long)e * st.sp_stride + g.sp_off + (long long)tile.rtile * kSpPerTile;
    if (threadIdx.x == 0) {
        sp[0] = g00;
        sp[1] = g01;
        sp[2] = g11;
    }
    // this tile's share of p-hat_{k,c'} . P[:, c] for every pending term: warp (k, c', c) adds it up in row order
    __syncthreads();          // s_p complete
    if (warp < NB) {
        const int k = warp / (R * R), c2 = (warp / R) % R, c = warp % R;
        double a = 0.0;
        if (k < nt)
            for (int r = r0 + lane; r < r1; r += 32)
                a += (double)s_p[(size_t)c * rows_pad + r - r0] * (double)__ldg(s_tph[k] + (long long)c2 * g.npad + r);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) sp[4 + warp] = a;
    }
}

// Pair edge step at rank 2: the Gram matrix P^T P from the tiles' shares, then the
// Gram-Schmidt step in column order as a 2 x 2 triangular map applied to P (in place,
// giving P-hat) and to U = D^T P (giving Q').  Column 0 is dead iff its squared norm
// is 0; column 1 iff its residual's squared norm is at most 1e-10 of its own before
// the projection.  A dead column leaves a zero P-hat column and its stored vector as
// it was.  Same CTA layout as the rank-1 step below.
__device__ void pair_edge_rank2(const DevState& st, const int* __restrict__ tab, int e, int l, int chunk,
                                double* scratch) {
    const int L = st.n_layers;
    const LayerGeom g = st.layers[l];
    const int pair = tab[st.tab.off_pair + e];
    const double* sp = st.Sp + (long long)e * st.sp_stride + g.sp_off;
    if (PG_OOB(st, kSecSp, sp, (long long)g.p_rtiles * kSpPerTile) ||
        PG_OOB(st, kSecPh, st.PhNext + (long long)e * st.ph_stride + g.ph_off, 2LL * g.npad) ||
        PG_OOB(st, kSecUp, st.Up + (long long)e * st.up_stride + g.up_off, (long long)g.p_rtiles * 2 * g.ld) ||
        PG_OOB(st, kSecQ, st.Qw + (long long)pair * st.q_stride + g.q_off, 2LL * g.ld) ||
        PG_OOB(st, kSecQ, st.Qr + (long long)pair * st.q_stride + g.q_off, 2LL * g.ld) ||
        PG_OOB(st, kSecQn2, st.Qn2 + ((long long)pair * L + l) * 2 * kEdgeChunks, 2 * kEdgeChunks))
        return;
    double a00 = 0.0, a01 = 0.0, a11 = 0.0;
    for (int t = threadIdx.x; t < g.p_rtiles; t += blockDim.x) {
        a00 += sp[kSpPerTile * t];
        a01 += sp[kSpPerTile * t + 1];
        a11 += sp[kSpPerTile * t + 2];
    }
    const double g00 = block_sum(a00, scratch);      // same order, hence same bits, in every chunk
    const double g01 = block_sum(a01, scratch);
    const double g11 = block_sum(a11, scratch);
    // Raw sweep with corrections pending: U[:, c] -= sum_{k,c'} c_k (p-hat_{k,c'} . P[:, c]) q'_{k,c'}.
    // Warp w < 12 adds product w = (k * 2 + c') * 2 + c of every tile in tile order.
    __shared__ double s_gam[kMaxTerms * 4];
    RawTerm terms[kMaxTerms];
    int nt = 0;
    if (g.raw && st.raw_pending)
        nt = raw_terms(st, tab, e, tab[st.tab.off_edge_i + e], tab[st.tab.off_edge_j + e], terms);
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int w = warp; w < nt * 4; w += (int)blockDim.x / 32) {
            double a = 0.0;
            for (int t = lane; t < g.p_rtiles; t += 32) a += sp[(long long)t * kSpPerTile + 4 + w];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) s_gam[w] = a * (double)terms[w / 4].coef;
        }
        __syncthreads();
    }
    const bool finite = isfinite(g00) && isfinite(g01) && isfinite(g11);
    const bool live0 = finite && g00 > 0.0;
    const double inv0 = live0 ? 1.0 / sqrt(g00) : 0.0;
    const double proj = live0 ? g01 * inv0 : 0.0;     // p-hat_0 . p_1
    const double res = g11 - proj * proj;
    const bool live1 = finite && res > 0.0 && res > 1e-10 * g11;
    const double inv1 = live1 ? 1.0 / sqrt(res) : 0.0;
    float* P = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    const int nch = g.e_chunks;
    const int rw = (g.npad + nch - 1) / nch;
    for (int r = chunk * rw + threadIdx.x; r < min(g.npad, (chunk + 1) * rw); r += blockDim.x) {
        const bool in = r < g.n;
        const float h0 = (live0 && in) ? (float)((double)P[r] * inv0) : 0.0f;
        const float h1 = (live1 && in) ? (float)(((double)P[g.npad + r] - proj * (double)h0) * inv1) : 0.0f;
        P[r] = h0;
        P[g.npad + r] = h1;
    }
    if (chunk == 0 && threadIdx.x == 0) {
        st.live[((long long)e * L + l) * 2] = live0 ? 1 : 0;
        st.live[((long long)e * L + l) * 2 + 1] = live1 ? 1 : 0;
        if (!finite) atomicOr(st.status, 1 << kStatusNumeric);
    }
    const float* up = st.Up + (long long)e * st.up_stride + g.up_off;
    float* Q = st.Qw + (long long)pair * st.q_stride + g.q_off;
    const float* Qold = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const int cw = (g.m + nch - 1) / nch;
    const int c_lo = chunk * cw, c_hi = min(g.m, (chunk + 1) * cw);
    if (Q != Qold)   // the vectors live in two copies that swap roles: a dead column's vector moves over unchanged
        for (int c = c_lo + threadIdx.x; c < c_hi; c += blockDim.x) {
            if (!live0) Q[c] = Qold[c];
            if (!live1) Q[g.ld + c] = Qold[g.ld + c];
        }
    if (!live0 && !live1) return;   // uniform over the block
    double part0 = 0.0, part1 = 0.0;
    for (int c = c_lo + threadIdx.x; c < c_hi; c += blockDim.x) {
        double u0 = 0.0, u1 = 0.0;
        for (int t = 0; t < g.p_rtiles; t += 4) {        // eight independent loads, added in tile order
            float v0[4], v1[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = t + j < g.p_rtiles;
                v0[j] = in ? up[((long long)(t + j) * 2) * g.ld + c] : 0.0f;
                v1[j] = in ? up[((long long)(t + j) * 2 + 1) * g.ld + c] : 0.0f;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                u0 += (double)v0[j];
                u1 += (double)v1[j];
            }
        }
        for (int k = 0; k < nt; ++k) {
            const float* tv = st.Qr + (long long)tab[st.tab.off_pair + terms[k].edge] * st.q_stride + g.q_off;
            const double t0 = (double)tv[c], t1 = (double)tv[g.ld + c];
            u0 -= s_gam[(k * 2 + 0) * 2 + 0] * t0 + s_gam[(k * 2 + 1) * 2 + 0] * t1;
            u1 -= s_gam[(k * 2 + 0) * 2 + 1] * t0 + s_gam[(k * 2 + 1) * 2 + 1] * t1;
        }
        const double q0 = u0 * inv0;
        if (live0) {
            const float q = (float)q0;
            Q[c] = q;
            part0 += (double)q * (double)q;
        }
        if (live1) {
            const float q = (float)((u1 - proj * q0) * inv1);
            Q[g.ld + c] = q;
            part1 += (double)q * (double)q;
        }
    }
    const double qq0 = block_sum(part0, scratch);
    const double qq1 = block_sum(part1, scratch);
    if (threadIdx.x == 0) {
        double* n2 = st.Qn2 + (((long long)pair * L + l) * 2) * kEdgeChunks;
        if (live0) n2[chunk] = qq0;
        if (live1) n2[kEdgeChunks + chunk] = qq1;
        if (!isfinite(qq0) || !isfinite(qq1)) atomicOr(st.status, 1 << kStatusNumeric);
    }
}

// Pair edge step: ||p||^2 from the tiles' shares, p-hat = p / ||p|| in place,
// Q' = (sum of the tiles' shares of D^T p) / ||p||, and the shares of ||Q'||^2
// (the sweep that uses Q' next adds them up).  A zero or non-finite norm leaves
// the stored vector alone and zeroes p-hat.  LayerGeom::e_chunks CTAs per (edge,
// layer), each taking a slice of the rows and of the columns; st.edge_tab lists
// the (layer, chunk) pairs of one edge.
// RAW: the layer's sweep takes the raw form; `pending`: it ran on rows with corrections pending, so
// the pending terms apply.
template <bool RAW>
__device__ void pair_edge_rank1(const DevState& st, const int* __restrict__ tab, int e, int l, int chunk, int nch,
                                bool pending) {
    __shared__ double scratch[33];
    __shared__ double s_tot[kMaxTerms + 1];
    __shared__ double s_grp[8][32];
    const int L = st.n_layers;
    const LayerGeom g = st.layers[l];
    const int pair = tab[st.tab.off_pair + e];
    const double* sp = st.Sp + (long long)e * st.sp_stride + g.sp_off;
    if (PG_OOB(st, kSecSp, sp, (long long)g.p_rtiles * kSpPerTile) ||
        PG_OOB(st, kSecPh, st.PhNext + (long long)e * st.ph_stride + g.ph_off, g.npad) ||
        PG_OOB(st, kSecUp, st.Up + (long long)e * st.up_stride + g.up_off, (long long)g.p_rtiles * g.ld) ||
        PG_OOB(st, kSecQ, st.Qw + (long long)pair * st.q_stride + g.q_off, g.ld) ||
        PG_OOB(st, kSecQ, st.Qr + (long long)pair * st.q_stride + g.q_off, g.ld) ||
        PG_OOB(st, kSecQn2, st.Qn2 + ((long long)pair * L + l) * kEdgeChunks, kEdgeChunks))
        return;
    // Raw sweep with corrections pending: the terms of this edge (same order as in the sweep).
    // Warp w adds scalar w of every tile in tile order: ||p||^2 (w = 0) and sum_r p_r p-hat_k[r]
    // (w = 1 + k); every chunk's CTA gets the same bits.
    RawTerm terms[RAW ? kMaxTerms : 1];
    int nt = 0;
    if (RAW && pending)
        nt = raw_terms(st, tab, e, tab[st.tab.off_edge_i + e], tab[st.tab.off_edge_j + e], terms);
    {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        if (warp <= nt) {
            const int which = warp == 0 ? 0 : 3 + warp;
            double a = 0.0;
            for (int t = lane; t < g.p_rtiles; t += 32) a += sp[(long long)t * kSpPerTile + which];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
            if (lane == 0) s_tot[warp] = a;
        }
        __syncthreads();
    }
    const double nn = s_tot[0];
    const bool finite = isfinite(nn);
    const bool live = finite && nn > 0.0;
    const double inv = live ? 1.0 / sqrt(nn) : 0.0;
    float* P = st.PhNext + (long long)e * st.ph_stride + g.ph_off;
    const int rw = (g.npad + nch - 1) / nch;
    for (int r = chunk * rw + threadIdx.x; r < min(g.npad, (chunk + 1) * rw); r += blockDim.x)
        P[r] = (live && r < g.n) ? (float)((double)P[r] * inv) : 0.0f;
    if (chunk == 0 && threadIdx.x == 0) {
        st.live[(long long)e * L + l] = live ? 1 : 0;
        if (!finite) atomicOr(st.status, 1 << kStatusNumeric);
    }
    float* Q = st.Qw + (long long)pair * st.q_stride + g.q_off;
    const float* Qold = st.Qr + (long long)pair * st.q_stride + g.q_off;
    const int cw = (g.m + nch - 1) / nch;
    const int c_lo = chunk * cw, c_hi = min(g.m, (chunk + 1) * cw);
    if (!live) {   // uniform over the block; with two copies of the vectors the old one moves over unchanged
        if (Q != Qold)
            for (int c = c_lo + threadIdx.x; c < c_hi; c += blockDim.x) Q[c] = Qold[c];
        return;
    }
    const float* up = st.Up + (long long)e * st.up_stride + g.up_off;
    // D'^T p = D^T p - sum_k c_k (p-hat_k . p) q'_k with the previous vectors of the pending edges
    constexpr int NTERM = RAW ? kMaxTerms : 0;
    const float* tvec[RAW ? kMaxTerms : 1];
    double tcoef[RAW ? kMaxTerms : 1];
#pragma unroll
    for (int k = 0; k < NTERM; ++k) {
        tvec[k] = Qold;
        tcoef[k] = 0.0;
        if (k < nt) {
            tvec[k] = st.Qr + (long long)tab[st.tab.off_pair + terms[k].edge] * st.q_stride + g.q_off;
            tcoef[k] = (double)terms[k].coef * s_tot[1 + k];
        }
    }
    double part = 0.0;
    if (cw <= 32) {
        // few columns, many tiles: 8 thread groups each add every 8th tile's share, then the
        // groups are added in order (a fixed order, so the result is reproducible)
        const int col = threadIdx.x & 31, grp = threadIdx.x >> 5;
        const int c = c_lo + col;
        double a = 0.0;
        if (c < c_hi)
            for (int t = grp; t < g.p_rtiles; t += 8) a += (double)up[(long long)t * g.ld + c];
        s_grp[grp][col] = a;
        __syncthreads();
        if (grp == 0 && c < c_hi) {
            double tot = 0.0;
#pragma unroll
            for (int k = 0; k < 8; ++k) tot += s_grp[k][col];
#pragma unroll
            for (int k = 0; k < NTERM; ++k)
                if (k < nt) tot -= tcoef[k] * (double)tvec[k][c];
            const float q = (float)(tot * inv);
            Q[c] = q;
            part = (double)q * (double)q;
        }
    } else {
        for (int c = c_lo + threadIdx.x; c < c_hi; c += blockDim.x) {
            double a = 0.0;
            for (int t = 0; t < g.p_rtiles; t += 8) {        // eight independent loads, added in tile order
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = t + j < g.p_rtiles ? up[(long long)(t + j) * g.ld + c] : 0.0f;
#pragma unroll
                for (int j = 0; j < 8; ++j) a += (double)v[j];
            }
#pragma unroll
            for (int k = 0; k < NTERM; ++k)
                if (k < nt) a -= tcoef[k] * (double)tvec[k][c];
            const float q = (float)(a * inv);
            Q[c] = q;
            part += (double)q * (double)q;
        }
    }
    const double qq = block_sum(part, scratch);
    if (threadIdx.x == 0) {
        st.Qn2[((long long)pair * L + l) * kEdgeChunks + chunk] = qq;
        if (!isfinite(qq)) atomicOr(st.status, 1 << kStatusNumeric);
    }
}

__global__ void __launch_bounds__(256)
pair_edge_kernel(DevState st, const int* __restrict__ tab) {
    grid_dependency_sync();
    __shared__ double scratch[33];
    const int e = blockIdx.x / st.e_total;
    const int slot = blockIdx.x - e * st.e_total;
    const int l = st.edge_tab[2 * slot], chunk = st.edge_tab[2 * slot + 1];
    if (e >= tab[st.tab.off_n_edges]) return;
    const LayerGeom g = st.layers[l];
    if (!g.pair_mode) return;
    if (st.rank == 2) {
        pair_edge_rank2(st, tab, e, l, chunk, scratch);
        return;
    }
    if (g.raw)
        pair_edge_rank1<true>(st, tab, e, l, chunk, g.e_chunks, st.raw_pending != 0);
    else
        pair_edge_rank1<false>(st, tab, e, l, chunk, g.e_chunks, false);
}

// 1 / ||column|| of every stored right factor (after initialisation or an
// external write).  One CTA per (pair, layer).
__global__ void __launch_bounds__(256)
column_norms_kernel(DevState st) {
    __shared__ double scratch[33];
    const int L = st.n_layers, rank = st.rank;
    const long long pair = blockIdx.x / L;
    const int l = blockIdx.x - (int)pair * L;
    const LayerGeom g = st.layers[l];
    const float* Q = (g.pair_mode ? st.Qr : st.Q) + pair * st.q_stride + g.q_off;
    if (PG_OOB(st, kSecQ, Q, (long long)rank * g.ld) || PG_OOB(st, kSecQinv, st.Qinv + (pair * L + l) * rank, rank) ||
        PG_OOB(st, kSecQn2, st.Qn2 + (pair * L + l) * rank * kEdgeChunks, rank * kEdgeChunks))
        return;
    for (int k = 0; k < rank; ++k) {
        double part = 0.0;
        for (int c = threadIdx.x; c < g.m; c += blockDim.x) {
            const double q = (double)Q[(long long)k * g.ld + c];
            part += q * q;
        }
        const double nn = block_sum(part, scratch);
        if (threadIdx.x == 0) {
            st.Qinv[(pair * L + l) * rank + k] = nn > 0.0 ? (float)(1.0 / sqrt(nn)) : 0.0f;
            {   // the pair sweep reads the squared norm as kEdgeChunks shares
                double* n2 = st.Qn2 + ((pair * L + l) * rank + k) * kEdgeChunks;
                n2[0] = nn;
                for (int t = 1; t < kEdgeChunks; ++t) n2[t] = 0.0;
            }
        }
    }
}

// --------------------------------------------------------------------------
// Persistent rounds for small stacks (everything stays in L2): one cooperative
// launch runs any number of power steps.  The four phases of a step are
// separated by a grid barrier instead of a kernel boundary.  The barrier is a
// counter plus a generation word in global memory; a CTA that waits gives up
// after `spin_limit` polls, raises the time-out bit of the status word and
// leaves, so a launch can never hang the device.
// --------------------------------------------------------------------------

__device__ bool grid_barrier(int* bar, int expected_blocks, int* status, long long spin_limit, int* s_ok) {
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        __threadfence();                                  // this CTA's results are out before it is counted
        volatile int* gen_word = bar + 1;
        const int gen = *gen_word;
        if (atomicAdd(&bar[0], 1) == expected_blocks - 1) {
            atomicExch(&bar[0], 0);
            __threadfence();
            atomicAdd(&bar[1], 1);                        // release the others
        } else {
            long long spins = 0;
            while (*gen_word == gen) {                    // bounded: a few seconds at most
                if (++spins > spin_limit) {
                    atomicOr(status, 1 << kStatusTimeout);
                    ok = 0;
                    break;
                }
            }
        }
        __threadfence();
        *s_ok = ok;
    }
    __syncthreads();
    return *s_ok != 0;
}

template <int S, int RT>
__global__ void __launch_bounds__(256, 2)
persistent_rounds_kernel(DevState st, const int* __restrict__ tab, const Tile* __restrict__ row_tiles,
                         int n_rows, const Tile* __restrict__ col_tiles, int n_cols, int n_steps,
                         int forward_first, int* bar, int expected_blocks, long long spin_limit) {
    constexpr size_t kBytes = sizeof(ColShared<S>) > sizeof(RowShared<S>) ? sizeof(ColShared<S>) : sizeof(RowShared<S>);
    __shared__ __align__(16) unsigned char s_raw[kBytes];
    __shared__ double scratch[33];
    __shared__ int s_ok;
    RowShared<S>& rsh = *reinterpret_cast<RowShared<S>*>(s_raw);
    ColShared<S>& csh = *reinterpret_cast<ColShared<S>*>(s_raw);
    const int nb = gridDim.x;
    const int L = st.n_layers;
    const int n_items = tab[st.tab.off_n_edges] * L;

    if (forward_first) {
        for (int t = blockIdx.x; t < n_rows; t += nb) {
            row_tile<S, false, true, false, RT, true>(st, tab, tab, row_tiles[t], rsh);
            __syncthreads();
        }
        if (!grid_barrier(bar, expected_blocks, st.status, spin_limit, &s_ok)) return;
    }
    for (int step = 0; step < n_steps; ++step) {
        for (int it = blockIdx.x; it < n_items; it += nb) edge_left_step<true>(st, tab, it / L, it % L, scratch);
        if (!grid_barrier(bar, expected_blocks, st.status, spin_limit, &s_ok)) return;
        for (int t = blockIdx.x; t < n_cols; t += nb) {
            col_tile<S, true, false>(st, tab, col_tiles[t], csh);
            __syncthreads();
        }
        if (!grid_barrier(bar, expected_blocks, st.status, spin_limit, &s_ok)) return;
        for (int it = blockIdx.x; it < n_items; it += nb) edge_right_step<true>(st, tab, it / L, it % L, scratch);
        if (!grid_barrier(bar, expected_blocks, st.status, spin_limit, &s_ok)) return;
        for (int t = blockIdx.x; t < n_rows; t += nb) {
            row_tile<S, true, true, true, RT, true>(st, tab, tab, row_tiles[t], rsh);
            __syncthreads();
        }
        if (step + 1 < n_steps && !grid_barrier(bar, expected_blocks, st.status, spin_limit, &s_ok)) return;
    }
}

// A barrier that one arrival too few will reach: every CTA must give up after
// `spin_limit` polls and report the time-out instead of hanging.
__global__ void __launch_bounds__(64)
barrier_timeout_probe_kernel(int* bar, int* status, long long spin_limit) {
    __shared__ int s_ok;
    grid_barrier(bar, (int)gridDim.x + 1, status, spin_limit, &s_ok);
}

// Launch, with programmatic stream serialisation if `allowed`: the kernel may then be
// scheduled before the previous kernel of the stream has finished, and waits for it on
// the device (grid_dependency_sync).
template <typename... Params, typename... Args>
cudaError_t launch_dep(int allowed, void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = allowed ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

template <int S, bool UPDATE, bool FORWARD, bool SAME, int RT, bool GRAD>
cudaError_t launch_row_t(const DevState& st, const int* tab_u, const int* tab_f, const Tile* tiles, int n_tiles,
                         cudaStream_t stream) {
    const size_t smem = row_ring_bytes(S, RT) +
                        sizeof(float) * S * ((size_t)st.f_chunk_max * (UPDATE && FORWARD && !SAME ? 2 : 1) + st.f_rows_max);
    cudaError_t rc = cudaFuncSetAttribute(row_sweep_kernel<S, UPDATE, FORWARD, SAME, RT, GRAD>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (rc != cudaSuccess) return rc;
    launch_dep(st.dep_launch & kDepSweep, row_sweep_kernel<S, UPDATE, FORWARD, SAME, RT, GRAD>, dim3(n_tiles),
               dim3(256), smem, stream, st, tab_u, tab_f, tiles);
    return cudaGetLastError();
}

template <bool UPDATE, bool FORWARD, bool SAME, bool GRAD>
cudaError_t launch_row_s(const DevState& st, const int* tab_u, const int* tab_f, const Tile* tiles, int n_tiles,
                         cudaStream_t stream) {
    const int slots = st.max_degree * st.rank;
    if (slots <= 1) return launch_row_t<1, UPDATE, FORWARD, SAME, kRowsPerWarp1, GRAD>(st, tab_u, tab_f, tiles, n_tiles, stream);
    if (slots <= 2) return launch_row_t<2, UPDATE, FORWARD, SAME, kRowsPerWarp2, GRAD>(st, tab_u, tab_f, tiles, n_tiles, stream);
    if (slots <= 4) return launch_row_t<4, UPDATE, FORWARD, SAME, kRowsPerWarp4, GRAD>(st, tab_u, tab_f, tiles, n_tiles, stream);
    return launch_row_t<8, UPDATE, FORWARD, SAME, kRowsPerWarp8, GRAD>(st, tab_u, tab_f, tiles, n_tiles, stream);
}

template <bool UPDATE, bool FORWARD, bool SAME>
cudaError_t launch_row(const DevState& st, const int* tab_u, const int* tab_f, const Tile* tiles,
                       int n_tiles, cudaStream_t stream) {
    if (n_tiles <= 0) return cudaSuccess;
    if (UPDATE && st.G)      // the update also takes the caller's gradient step
        return launch_row_s<UPDATE, FORWARD, SAME, UPDATE>(st, tab_u, tab_f, tiles, n_tiles, stream);
    return launch_row_s<UPDATE, FORWARD, SAME, false>(st, tab_u, tab_f, tiles, n_tiles, stream);
}

}  // namespace

cudaError_t launch_forward(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                           cudaStream_t stream) {
    return launch_row<false, true, false>(st, tab, tab, tiles, n_tiles, stream);
}

cudaError_t launch_update_forward(const DevState& st, const int* tab_update, const int* tab_forward,
                                  const Tile* tiles, int n_tiles, cudaStream_t stream) {
    // the same table means the same edges, pairs and vectors for both halves
    if (tab_update == tab_forward)
        return launch_row<true, true, true>(st, tab_update, tab_forward, tiles, n_tiles, stream);
    return launch_row<true, true, false>(st, tab_update, tab_forward, tiles, n_tiles, stream);
}

cudaError_t launch_update(const DevState& st, const int* tab_update, const Tile* tiles, int n_tiles,
                          cudaStream_t stream) {
    return launch_row<true, false, false>(st, tab_update, tab_update, tiles, n_tiles, stream);
}

template <int NV, bool UPDATE, int D>
static cudaError_t launch_pair_bulk_t(const DevState& st, const int* tab_prev, const int* tab_cur,
                                      const Tile* tiles, int n_tiles, int max_ld, cudaStream_t stream) {
    // stage buffers; they also hold the 8 x NV*128 floats of the final reduction
    size_t smem = sizeof(float) * (size_t)kBulkStages * 2 * kBulkRows * max_ld;
    const size_t red = sizeof(float) * 8 * NV * 128;
    if (smem < red) smem = red;
    cudaError_t rc = cudaFuncSetAttribute(pair_sweep_bulk_kernel<NV, UPDATE, D>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (rc != cudaSuccess) return rc;
    launch_dep(st.dep_launch & kDepPairRow, pair_sweep_bulk_kernel<NV, UPDATE, D>, dim3(n_tiles), dim3(256), smem, stream, st, tab_prev, tab_cur, tiles);
    return cudaGetLastError();
}

template <bool UPDATE, int D>
static cudaError_t launch_pair_bulk(const DevState& st, const int* tab_prev, const int* tab_cur, const Tile* tiles,
                                    int n_tiles, int nv, cudaStream_t stream) {
    const int max_ld = nv * 128;
    switch (nv) {
        case 1: return launch_pair_bulk_t<1, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 2: return launch_pair_bulk_t<2, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 3: return launch_pair_bulk_t<3, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 4: return launch_pair_bulk_t<4, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 5: return launch_pair_bulk_t<5, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 6: return launch_pair_bulk_t<6, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        case 7: return launch_pair_bulk_t<7, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
        default: return launch_pair_bulk_t<8, UPDATE, D>(st, tab_prev, tab_cur, tiles, n_tiles, max_ld, stream);
    }
}

// `tiles` must list tiles of layers with the same number of float4 per lane
// (ceil(ld / 128)); the host launches one group per value.
// pend_slots: how many corrections can be pending at a worker (its largest degree).
cudaError_t launch_pair_sweep(const DevState& st, const int* tab_prev, const int* tab_cur, bool apply_pending,
                              const Tile* tiles, int n_tiles, int nv, int pend_slots, cudaStream_t stream) {
    if (n_tiles <= 0) return cudaSuccess;
    if (!apply_pending) return launch_pair_bulk<false, 1>(st, tab_prev, tab_cur, tiles, n_tiles, nv, stream);
    if (pend_slots > 2) return cudaErrorInvalidValue;
    return pend_slots > 1 ? launch_pair_bulk<true, 2>(st, tab_prev, tab_cur, tiles, n_tiles, nv, stream)
                          : launch_pair_bulk<true, 1>(st, tab_prev, tab_cur, tiles, n_tiles, nv, stream);
}

template <int NVW, bool UPDATE, int D>
static cudaError_t launch_wide_t(const DevState& st, const int* tab_prev, const int* tab_cur, const Tile* tiles,
                                 int n_tiles, int slice_pad, cudaStream_t stream) {
    const dim3 grid(static_cast<unsigned>(n_tiles) * kPairCluster);
    const size_t smem = sizeof(float) * (1 + 2 * D) * static_cast<size_t>(slice_pad);
    if (smem > 48 * 1024) {
        cudaError_t rc = cudaFuncSetAttribute(pair_sweep_wide_kernel<NVW, UPDATE, D>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (rc != cudaSuccess) return rc;
    }
    launch_dep(st.dep_launch & kDepPairWide, pair_sweep_wide_kernel<NVW, UPDATE, D>, dim3(grid), dim3(256), smem, stream, st, tab_prev, tab_cur, tiles, slice_pad);
    return cudaGetLastError();
}

template <int NVW>
static cudaError_t launch_wide(const DevState& st, const int* tab_prev, const int* tab_cur, bool upd, int pend_slots,
                               const Tile* tiles, int n_tiles, int slice_pad, cudaStream_t stream) {
    if (!upd) return launch_wide_t<NVW, false, 1>(st, tab_prev, tab_cur, tiles, n_tiles, slice_pad, stream);
    return pend_slots > 1 ? launch_wide_t<NVW, true, 2>(st, tab_prev, tab_cur, tiles, n_tiles, slice_pad, stream)
                          : launch_wide_t<NVW, true, 1>(st, tab_prev, tab_cur, tiles, n_tiles, slice_pad, stream);
}

// `tiles`: cluster tiles of layers with the same float4 count per thread `nv` and
// the same slice width `slice` (columns per CTA).
cudaError_t launch_pair_sweep_wide(const DevState& st, const int* tab_prev, const int* tab_cur,
                                   bool apply_pending, const Tile* tiles, int n_tiles, int nv, int slice,
                                   int pend_slots, cudaStream_t stream) {
    if (n_tiles <= 0) return cudaSuccess;
    const int slice_pad = (slice + 3) / 4 * 4;
    switch (nv) {
        case 1: return launch_wide<1>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 2: return launch_wide<2>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 3: return launch_wide<3>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 4: return launch_wide<4>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 5: return launch_wide<5>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 6: return launch_wide<6>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        case 7: return launch_wide<7>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
        default: return launch_wide<8>(st, tab_prev, tab_cur, apply_pending, pend_slots, tiles, n_tiles, slice_pad, stream);
    }
}

template <int NVW, int D>
static int resident_clusters(int slice_pad) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kPairCluster * 1024);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = sizeof(float) * (1 + 2 * D) * static_cast<size_t>(slice_pad);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kPairCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    cudaError_t rc = cudaSuccess;
    if (cfg.dynamicSmemBytes > 48 * 1024)
        rc = cudaFuncSetAttribute(pair_sweep_wide_kernel<NVW, true, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)cfg.dynamicSmemBytes);
    if (rc == cudaSuccess) rc = cudaOccupancyMaxActiveClusters(&n, pair_sweep_wide_kernel<NVW, true, D>, &cfg);
    if (rc != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

int pair_wide_resident_clusters(int nv, int slice, int pend_slots) {
    const int slice_pad = (slice + 3) / 4 * 4;
    if (pend_slots > 1) switch (nv) {
        case 1: return resident_clusters<1, 2>(slice_pad);
        case 2: return resident_clusters<2, 2>(slice_pad);
        case 3: return resident_clusters<3, 2>(slice_pad);
        case 4: return resident_clusters<4, 2>(slice_pad);
        case 5: return resident_clusters<5, 2>(slice_pad);
        case 6: return resident_clusters<6, 2>(slice_pad);
        case 7: return resident_clusters<7, 2>(slice_pad);
        default: return resident_clusters<8, 2>(slice_pad);
    }
    switch (nv) {
        case 1: return resident_clusters<1, 1>(slice_pad);
        case 2: return resident_clusters<2, 1>(slice_pad);
        case 3: return resident_clusters<3, 1>(slice_pad);
        case 4: return resident_clusters<4, 1>(slice_pad);
        case 5: return resident_clusters<5, 1>(slice_pad);
        case 6: return resident_clusters<6, 1>(slice_pad);
        case 7: return resident_clusters<7, 1>(slice_pad);
        default: return resident_clusters<8, 1>(slice_pad);
    }
}

// dst[r][c] = src[r * cols + c]: a dense matrix into its padded place in the stack.
__global__ void __launch_bounds__(256)
unpack_rows_kernel(float* __restrict__ dst, long long ld, const float* __restrict__ src, int rows, int cols) {
    const long long total = (long long)rows * cols;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const long long r = idx / cols;
        dst[r * ld + (idx - r * cols)] = src[idx];
    }
}

cudaError_t launch_unpack_rows(float* dst, long long ld, const float* src, int rows, int cols, cudaStream_t stream) {
    const long long total = (long long)rows * cols;
    const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 16);
    unpack_rows_kernel<<<blocks, 256, 0, stream>>>(dst, ld, src, rows, cols);
    return cudaGetLastError();
}

cudaError_t launch_pair_edge(const DevState& st, const int* tab, int max_edges, cudaStream_t stream) {
    if (st.e_total <= 0) return cudaSuccess;
    launch_dep(st.dep_launch & kDepPairEdge, pair_edge_kernel, dim3(max_edges * st.e_total), dim3(256), 0, stream, st, tab);
    return cudaGetLastError();
}

// Shared memory one CTA may ask for, less the kernels' static part.
constexpr size_t kMidSmemBudget = 227 * 1024 - 1024;

template <int NVM, bool UPDATE, int D, bool RAW, int ENDS>
static cudaError_t launch_mid_t(const DevState& st, const int* tab_prev, const int* tab_cur, const Tile* tiles,
                                int n_tiles, int ld_pad, int max_rows, cudaStream_t stream) {
    // TMA-fed variant when the row fits its registers and at least two stages fit in shared memory
    if constexpr (NVM <= kMidBulkNv) {
        // the raw form keeps 2 + ENDS * D scalars per row of the tile behind the stages
        const int rows_pad = (max_rows + 3) / 4 * 4;
        const size_t scalars = RAW ? sizeof(float) * (2 + ENDS * D) * static_cast<size_t>(rows_pad) : 0;
        const size_t stage = sizeof(float) * 2 * mid_rows(NVM) * static_cast<size_t>(ld_pad);
        // leave room for the second CTA where the kernel is built for two per SM
        const size_t budget = kMidSmemBudget / mid_min_blocks(NVM, RAW ? (ENDS * D + 1) / 2 : D);
        const int n_stage = budget > scalars ? (int)std::min<size_t>((budget - scalars) / stage, kMidStagesMax) : 0;
        if (n_stage >= 2) {
            const size_t total = n_stage * stage + scalars;
            cudaError_t rc = cudaFuncSetAttribute(pair_sweep_mid_bulk_kernel<NVM, UPDATE, D, RAW, ENDS>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
            if (rc != cudaSuccess) return rc;
            launch_dep(st.dep_launch & kDepPairMid, pair_sweep_mid_bulk_kernel<NVM, UPDATE, D, RAW, ENDS>, dim3(n_tiles), dim3(256), total, stream, st, tab_prev, tab_cur, tiles, ld_pad, n_stage, rows_pad);
            return cudaGetLastError();
        }
    }
    if constexpr (RAW) {
        return cudaErrorInvalidValue;      // the host gives the raw form only rows the TMA-fed kernel takes
    } else {
        const size_t smem = sizeof(float) * (1 + 2 * D) * static_cast<size_t>(ld_pad);
        if (smem > 48 * 1024) {
            cudaError_t rc = cudaFuncSetAttribute(pair_sweep_mid_kernel<NVM, UPDATE, D>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (rc != cudaSuccess) return rc;
        }
        launch_dep(st.dep_launch & kDepPairMid, pair_sweep_mid_kernel<NVM, UPDATE, D>, dim3(n_tiles), dim3(256), smem, stream, st, tab_prev, tab_cur, tiles, ld_pad);
        return cudaGetLastError();
    }
}

template <int NVM>
static cudaError_t launch_mid(const DevState& st, const int* tab_prev, const int* tab_cur, bool upd, int pend_slots,
                              bool raw, bool single_owner, const Tile* tiles, int n_tiles, int ld_pad, int max_rows,
                              cudaStream_t stream) {
    if (!upd) return launch_mid_t<NVM, false, 1, false, 2>(st, tab_prev, tab_cur, tiles, n_tiles, ld_pad, max_rows, stream);
    if (pend_slots > 2) return cudaErrorInvalidValue;
    if (pend_slots <= 1) return launch_mid_t<NVM, true, 1, false, 2>(st, tab_prev, tab_cur, tiles, n_tiles, ld_pad, max_rows, stream);
    if constexpr (NVM <= kMidBulkNv) {
        if (raw)
            return single_owner ? launch_mid_t<NVM, true, 2, true, 1>(st, tab_prev, tab_cur, tiles, n_tiles, ld_pad, max_rows, stream)
                                : launch_mid_t<NVM, true, 2, true, 2>(st, tab_prev, tab_cur, tiles, n_tiles, ld_pad, max_rows, stream);
    }
    return launch_mid_t<NVM, true, 2, false, 2>(st, tab_prev, tab_cur, tiles, n_tiles, ld_pad, max_rows, stream);
}

template <int NVM, bool UPDATE>
static cudaError_t launch_mid2_t(const DevState& st, const int* tab, const Tile* tiles, int n_tiles, int ld_pad,
                                 cudaStream_t stream) {
    const size_t stage = sizeof(float) * 2 * mid2_rows(NVM) * static_cast<size_t>(ld_pad);
    const int n_stage = (int)std::min<size_t>(kMidSmemBudget / stage, kMidStagesMax);
    if (n_stage < 2) return cudaErrorInvalidValue;
    const size_t total = n_stage * stage;
    cudaError_t rc = cudaFuncSetAttribute(pair_sweep_mid2_kernel<NVM, UPDATE>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
    if (rc != cudaSuccess) return rc;
    launch_dep(st.dep_launch & kDepPairMid, pair_sweep_mid2_kernel<NVM, UPDATE>, dim3(n_tiles), dim3(kMid2Threads),
               total, stream, st, tab, tiles, ld_pad, n_stage);
    return cudaGetLastError();
}

template <int NVM>
static cudaError_t launch_mid2_raw_t(const DevState& st, const int* tab, const Tile* tiles, int n_tiles, int ld_pad,
                                     int max_rows, cudaStream_t stream) {
    const size_t stage = sizeof(float) * 2 * mid2_rows(NVM) * static_cast<size_t>(ld_pad);
    const int rows_pad = (max_rows + 3) / 4 * 4;
    const size_t scalars = sizeof(float) * 8 * static_cast<size_t>(rows_pad);       // 2 + 2 + 4 per row
    const size_t budget = kMidSmemBudget - 2048;                                    // the kernel's static part
    const int n_stage = budget > scalars ? (int)std::min<size_t>((budget - scalars) / stage, kMidStagesMax) : 0;
    if (n_stage < 2) return cudaErrorInvalidValue;
    const size_t total = n_stage * stage + scalars;
    cudaError_t rc = cudaFuncSetAttribute(pair_sweep_mid2_raw_kernel<NVM>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize, (int)total);
    if (rc != cudaSuccess) return rc;
    launch_dep(st.dep_launch & kDepPairMid, pair_sweep_mid2_raw_kernel<NVM>, dim3(n_tiles), dim3(kMid2Threads),
               total, stream, st, tab, tiles, ld_pad, n_stage, rows_pad);
    return cudaGetLastError();
}

// Rank 2: static graphs only, so one table serves the pending corrections and the step.
static cudaError_t launch_mid2(const DevState& st, const int* tab, bool upd, bool raw, const Tile* tiles, int n_tiles,
                               int ld_pad, int max_rows, cudaStream_t stream) {
    const int nvm = (ld_pad / 4 + kMid2Threads - 1) / kMid2Threads;     // float4 per thread and row
    if (upd && raw) switch (nvm) {
        case 1: return launch_mid2_raw_t<1>(st, tab, tiles, n_tiles, ld_pad, max_rows, stream);
        case 2: return launch_mid2_raw_t<2>(st, tab, tiles, n_tiles, ld_pad, max_rows, stream);
        case 3: return launch_mid2_raw_t<3>(st, tab, tiles, n_tiles, ld_pad, max_rows, stream);
        case 4: return launch_mid2_raw_t<4>(st, tab, tiles, n_tiles, ld_pad, max_rows, stream);
        default: return cudaErrorInvalidValue;
    }
    switch (nvm) {
        case 1: return upd ? launch_mid2_t<1, true>(st, tab, tiles, n_tiles, ld_pad, stream)
                           : launch_mid2_t<1, false>(st, tab, tiles, n_tiles, ld_pad, stream);
        case 2: return upd ? launch_mid2_t<2, true>(st, tab, tiles, n_tiles, ld_pad, stream)
                           : launch_mid2_t<2, false>(st, tab, tiles, n_tiles, ld_pad, stream);
        case 3: return upd ? launch_mid2_t<3, true>(st, tab, tiles, n_tiles, ld_pad, stream)
                           : launch_mid2_t<3, false>(st, tab, tiles, n_tiles, ld_pad, stream);
        case 4: return upd ? launch_mid2_t<4, true>(st, tab, tiles, n_tiles, ld_pad, stream)
                           : launch_mid2_t<4, false>(st, tab, tiles, n_tiles, ld_pad, stream);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_pair_sweep_mid(const DevState& st, const int* tab_prev, const int* tab_cur,
                                  bool apply_pending, const Tile* tiles, int n_tiles, int nv, int ld_pad,
                                  int pend_slots, bool raw, bool single_owner, int max_rows, cudaStream_t stream) {
    if (n_tiles <= 0) return cudaSuccess;
    if (st.rank == 2) {
        if (tab_prev != tab_cur || pend_slots != 2) return cudaErrorInvalidValue;
        return launch_mid2(st, tab_cur, apply_pending, raw, tiles, n_tiles, ld_pad, max_rows, stream);
    }
    switch (nv) {
        case 1: return launch_mid<1>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 2: return launch_mid<2>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 3: return launch_mid<3>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 4: return launch_mid<4>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 5: return launch_mid<5>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 6: return launch_mid<6>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        case 7: return launch_mid<7>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
        default: return launch_mid<8>(st, tab_prev, tab_cur, apply_pending, pend_slots, raw, single_owner, tiles, n_tiles, ld_pad, max_rows, stream);
    }
}

template <bool UPDATE>
static cudaError_t launch_col(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                              cudaStream_t stream) {
    if (n_tiles <= 0) return cudaSuccess;
    const int slots = st.max_degree * st.rank;
    if (slots <= 1)
        launch_dep(st.dep_launch & kDepSweep, col_sweep_kernel<1, UPDATE>, dim3(n_tiles), dim3(256), 0, stream, st, tab, tiles);
    else if (slots <= 2)
        launch_dep(st.dep_launch & kDepSweep, col_sweep_kernel<2, UPDATE>, dim3(n_tiles), dim3(256), 0, stream, st, tab, tiles);
    else if (slots <= 4)
        launch_dep(st.dep_launch & kDepSweep, col_sweep_kernel<4, UPDATE>, dim3(n_tiles), dim3(256), 0, stream, st, tab, tiles);
    else
        launch_dep(st.dep_launch & kDepSweep, col_sweep_kernel<8, UPDATE>, dim3(n_tiles), dim3(256), 0, stream, st, tab, tiles);
    return cudaGetLastError();
}

cudaError_t launch_transposed(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                              cudaStream_t stream) {
    return launch_col<false>(st, tab, tiles, n_tiles, stream);
}

cudaError_t launch_transposed_update(const DevState& st, const int* tab, const Tile* tiles, int n_tiles,
                                     cudaStream_t stream) {
    return launch_col<true>(st, tab, tiles, n_tiles, stream);
}

cudaError_t launch_random_directions(const DevState& st, const int* tab, int max_edges, unsigned key_lo,
                                     unsigned key_hi, int side, cudaStream_t stream) {
    launch_dep(st.dep_launch & kDepSweep, random_directions_kernel, dim3(max_edges * st.n_layers), dim3(256), 0, stream, st, tab, key_lo, key_hi, side);
    return cudaGetLastError();
}

cudaError_t launch_edge_raw(const DevState& st, const int* tab, int max_edges, cudaStream_t stream) {
    launch_dep(st.dep_launch & kDepSweep, edge_raw_kernel, dim3(max_edges * st.n_layers), dim3(256), 0, stream, st, tab);
    return cudaGetLastError();
}

cudaError_t launch_edge_odd(const DevState& st, const int* tab, int max_edges, cudaStream_t stream) {
    launch_dep(st.dep_launch & kDepSweep, edge_odd_kernel, dim3(max_edges * st.n_layers), dim3(512), 0, stream, st, tab);
    return cudaGetLastError();
}

cudaError_t launch_edge_left(const DevState& st, const int* tab, int max_edges, cudaStream_t stream) {
    launch_dep(st.dep_launch & kDepSweep, edge_left_kernel, dim3(max_edges * st.n_layers), dim3(512), 0, stream, st, tab);
    return cudaGetLastError();
}

cudaError_t launch_edge_right(const DevState& st, const int* tab, int max_edges, cudaStream_t stream) {
    launch_dep(st.dep_launch & kDepSweep, edge_right_kernel, dim3(max_edges * st.n_layers), dim3(512), 0, stream, st, tab);
    return cudaGetLastError();
}

template <int S, int RT>
static cudaError_t launch_persistent_t(const DevState& st, const int* tab, const Tile* row_tiles, int n_rows,
                                       const Tile* col_tiles, int n_cols, int n_steps, bool forward_first,
                                       int* bar, int max_blocks, cudaStream_t stream) {
    int per_sm = 0, dev = 0, sms = 0;
    cudaError_t rc = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, persistent_rounds_kernel<S, RT>, 256, 0);
    if (rc == cudaSuccess) rc = cudaGetDevice(&dev);
    if (rc == cudaSuccess) rc = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (rc != cudaSuccess) return rc;
    int grid = per_sm * sms;                       // all CTAs resident at once: the barrier needs that
    if (grid > max_blocks) grid = max_blocks;
    if (grid < 1) return cudaErrorInvalidConfiguration;
    rc = cudaMemsetAsync(bar, 0, 2 * sizeof(int), stream);
    if (rc != cudaSuccess) return rc;
    DevState st_copy = st;
    int fwd = forward_first ? 1 : 0, expected = grid;
    long long limit = kBarrierSpinLimit;
    void* args[] = {&st_copy, &tab, &row_tiles, &n_rows, &col_tiles, &n_cols, &n_steps, &fwd, &bar, &expected, &limit};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(persistent_rounds_kernel<S, RT>), dim3(grid),
                                       dim3(256), args, 0, stream);
}

cudaError_t launch_persistent(const DevState& st, const int* tab, const Tile* row_tiles, int n_rows,
                              const Tile* col_tiles, int n_cols, int n_steps, bool forward_first, int* bar,
                              cudaStream_t stream) {
    const int slots = st.max_degree * st.rank;
    const int max_blocks = n_rows > n_cols ? n_rows : n_cols;
    if (slots <= 1)
        return launch_persistent_t<1, kRowsPerWarp1>(st, tab, row_tiles, n_rows, col_tiles, n_cols, n_steps, forward_first, bar, max_blocks, stream);
    if (slots <= 2)
        return launch_persistent_t<2, kRowsPerWarp2>(st, tab, row_tiles, n_rows, col_tiles, n_cols, n_steps, forward_first, bar, max_blocks, stream);
    if (slots <= 4)
        return launch_persistent_t<4, kRowsPerWarp4>(st, tab, row_tiles, n_rows, col_tiles, n_cols, n_steps, forward_first, bar, max_blocks, stream);
    return launch_persistent_t<8, kRowsPerWarp8>(st, tab, row_tiles, n_rows, col_tiles, n_cols, n_steps, forward_first, bar, max_blocks, stream);
}

// Asks the bounds check about one range inside the parameter section and one that ends a float past
// it; nothing is read or written.  The checked build raises the bounds bit for the second range.
__global__ void bounds_probe_kernel(DevState st) {
#ifdef PG_BOUNDS_CHECK
    const float* last = reinterpret_cast<const float*>(st.sec_hi[kSecX]) - 4;
    if (PG_OOB(st, kSecX, last, 4)) atomicOr(st.status, 1 << kStatusTimeout);     // must not happen
    (void)PG_OOB(st, kSecX, last, 5);
#else
    (void)st;
#endif
}

cudaError_t launch_bounds_probe(const DevState& st, cudaStream_t stream) {
    bounds_probe_kernel<<<1, 32, 0, stream>>>(st);
    return cudaGetLastError();
}

cudaError_t launch_barrier_timeout_probe(int* bar, int* status, cudaStream_t stream) {
    cudaError_t rc = cudaMemsetAsync(bar, 0, 2 * sizeof(int), stream);
    if (rc != cudaSuccess) return rc;
    barrier_timeout_probe_kernel<<<4, 64, 0, stream>>>(bar, status, 20000);   // a few milliseconds of polling
    return cudaGetLastError();
}

cudaError_t launch_column_norms(const DevState& st, long long n_pairs, cudaStream_t stream) {
    column_norms_kernel<<<(unsigned)(n_pairs * st.n_layers), 256, 0, stream>>>(st);
    return cudaGetLastError();
}

}  // namespace pg
