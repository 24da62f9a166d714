// Device code of the DEF / DEF-A / EF step for sm_100a.
//
// The step (Algorithm 1 from its error-feedback step to its update, with the momentum form of Eq. 10) is separate
// per model coordinate: a coordinate j needs g, m, e of its W workers and, if j is
// one of the k block coordinates, x[j].  Two facts shape the kernels:
//   * Outside the block nothing crosses workers (C(p) = 0, e' = p), so that part --
//     all but k of the d coordinates -- is plain streaming of the [W, d] tensors and
//     can be cut any way the memory system likes best.
//   * On the block, the sum over workers that stands in for the ring-allreduce of
//     Algorithm 1 is a register accumulation by one thread in the fixed order
//     w = 0..W-1: deterministic, with no shuffle, shared memory or atomics.
// Either way g, m, e are read once and m', e' written once (20 bytes per gradient
// element, the least the method can move) with 128-bit coalesced accesses, p never
// goes to memory, and x is touched on the block only (Algorithm 1's update).  The block is a
// predicate on j, never a slice: nothing is gathered or scattered.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace defk {

// ---------------------------------------------------------------------------
// Shared block start (Section 1: one uniformly random start per iteration, the
// same on every worker).  Philox4x32-10 of Salmon et al. (SC'11), keyed by the seed,
// counter = (step, tag).  Written for the GPU's 32-bit multiplier pair.
// ---------------------------------------------------------------------------
__host__ __device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1) {
#ifdef __CUDA_ARCH__
    const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]);
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]);
#else
    const uint32_t hi0 = (uint32_t)(((uint64_t)0xD2511F53u * c[0]) >> 32);
    const uint32_t hi1 = (uint32_t)(((uint64_t)0xCD9E8D57u * c[2]) >> 32);
#endif
    const uint32_t lo0 = 0xD2511F53u * c[0];
    const uint32_t lo1 = 0xCD9E8D57u * c[2];
    const uint32_t a = hi1 ^ c[1] ^ k0;
    const uint32_t b = hi0 ^ c[3] ^ k1;
    c[0] = a; c[1] = lo1; c[2] = b; c[3] = lo0;
}

__host__ __device__ __forceinline__ int64_t block_start(uint64_t seed, uint64_t step, int64_t d) {
    uint32_t c[4] = {(uint32_t)step, (uint32_t)(step >> 32), 0x52424753u /* "RBGS" */, 0u};
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        philox_round(c, k0, k1);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    const uint64_t r64 = (uint64_t)c[0] | ((uint64_t)c[1] << 32);
#ifdef __CUDA_ARCH__
    return (int64_t)__umul64hi(r64, (uint64_t)d);
#else
    return (int64_t)(uint64_t)(((unsigned __int128)r64 * (unsigned __int128)(uint64_t)d) >> 64);
#endif
}

__global__ void block_start_batch_kernel(const uint64_t *__restrict__ seeds,
                                         const uint64_t *__restrict__ steps,
                                         const int64_t *__restrict__ ds, int64_t n,
                                         int64_t *__restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = block_start(seeds[i], steps[i], ds[i]);
}

// ---------------------------------------------------------------------------
// Vector types: V consecutive floats moved by one load / store.
// ---------------------------------------------------------------------------
template <int V> struct Vec;
template <> struct Vec<1> { float v[1]; };
template <> struct alignas(8) Vec<2> { float v[2]; };
template <> struct alignas(16) Vec<4> { float v[4]; };

// Cache policy of the [W, d] traffic.  g, m and e are read once per step and m', e' are
// not read again before the next step.  kCacheDefault leaves write-back to the L2's own
// replacement; kCacheStreaming marks loads and stores evict-first (ld.cs / st.cs).
constexpr int kCacheDefault = 0;
constexpr int kCacheStreaming = 1;

template <int V, int POL> __device__ __forceinline__ Vec<V> load_vec(const float *p) {
    Vec<V> r;
    if constexpr (V == 1) {
        r.v[0] = POL == kCacheStreaming ? __ldcs(p) : *p;
    } else if constexpr (V == 2) {
        const float2 t = POL == kCacheStreaming ? __ldcs(reinterpret_cast<const float2 *>(p))
                                                : *reinterpret_cast<const float2 *>(p);
        r.v[0] = t.x; r.v[1] = t.y;
    } else {
        const float4 t = POL == kCacheStreaming ? __ldcs(reinterpret_cast<const float4 *>(p))
                                                : *reinterpret_cast<const float4 *>(p);
        r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w;
    }
    return r;
}
template <int V, int POL> __device__ __forceinline__ void store_vec(float *p, const Vec<V> &a) {
    if constexpr (V == 1) {
        if (POL == kCacheStreaming) __stcs(p, a.v[0]); else *p = a.v[0];
    } else if constexpr (V == 2) {
        const float2 t = make_float2(a.v[0], a.v[1]);
        if (POL == kCacheStreaming) __stcs(reinterpret_cast<float2 *>(p), t);
        else *reinterpret_cast<float2 *>(p) = t;
    } else {
        const float4 t = make_float4(a.v[0], a.v[1], a.v[2], a.v[3]);
        if (POL == kCacheStreaming) __stcs(reinterpret_cast<float4 *>(p), t);
        else *reinterpret_cast<float4 *>(p) = t;
    }
}

struct StepArgs {
    float *x;            // [n]      local coordinates of the model
    const float *g;      // [W, ld]
    float *e;            // [W, ld]
    float *m;            // [W, ld] or nullptr
    float *z;            // [W, ld] next detach points x_{t+1} - lambda e_{t+1}, or nullptr
    float *block_sum;    // [k] or nullptr: if set, the workers' sum of C(p) on block coordinate
                         // (s + i) mod d goes to block_sum[i] and x is only read (rows sharded
                         // over GPUs: the caller all-reduces block_sum, then applies it)
    int64_t n;           // local coordinates
    int64_t ld;          // row stride in floats
    int64_t d;           // model size the block is drawn over
    int64_t j0;          // model coordinate of local coordinate 0
    int64_t k;           // block length
    int32_t W;           // workers
    float eta;           // learning rate
    float mu;            // momentum constant
    float W_float;       // (float)W, the divisor of the average over workers
    float lambda;        // detach coefficient (used only when z is written)
    float delta;         // factor of the scaling compressor C(v) = delta v (used only by it)
    uint64_t seed, step; // the block start is drawn from these
    int32_t chunk;       // stream kernel, chunked order: CTAs per row segment (see kOrderChunked)
};

// The start of this step's block, computed by one thread of the CTA and handed to the
// others through shared memory (the ten Philox rounds are a serial chain of ~100
// instructions: once per CTA they cost nothing, once per thread they would show).
__device__ __forceinline__ int64_t cta_block_start(const StepArgs &a) {
    __shared__ int64_t s_shared;
    if (threadIdx.x == 0) s_shared = block_start(a.seed, a.step, a.d);
    __syncthreads();
    return s_shared;
}

// Programmatic dependent launch, used by the kernel pair of a step.  The kernel that does the tiles
// touching the block (the primary) releases its dependents at its first instruction; the stream
// kernel launched behind it (the secondary) may then start beside it -- the two write disjoint
// floats.  What is enqueued AFTER the pair is ordered behind the secondary only, so the secondary
// grid must not complete before the primary has: one thread of it (thread 0 of CTA 0) ends with
// grid_dependency_wait(), which returns once the primary grid has completed and its writes are
// visible, and a grid is complete only when all of its threads are.  One waiting thread is enough
// for that and keeps one CTA slot busy; with the wait in every thread, finished CTAs would hold
// their slots until the primary ends and the rest of the secondary could not start (measured:
// +2 us on an 80 MB step).  The dependents are released only when every CTA of the primary has
// started, so the wait cannot deadlock; in a kernel that was launched without the programmatic
// attribute both instructions do nothing.
__device__ __forceinline__ void release_dependent_grids() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// One worker's row for V coordinates: Eq. 10 (or Algorithm 1's error-feedback step), then its new error.
// `sent` accumulates C(p) over the workers in call order; `first` starts the sum.
// SCALE selects the scaling compressor C(p) = delta p of the DEF-A paragraph (the case that
// turns the iteration into SGD with iterate averaging, Eq. 11) instead of RBGS.
template <int V, bool MOM, bool SCALE = false>
__device__ __forceinline__ void worker_row(const Vec<V> &g, const Vec<V> &m, const Vec<V> &e,
                                           const bool (&in)[V], float eta, float mu, bool first,
                                           Vec<V> &m_new, Vec<V> &e_new, float (&sent)[V],
                                           float delta = 0.0f) {
#pragma unroll
    for (int i = 0; i < V; ++i) {
        float p;
        if (MOM) {
            m_new.v[i] = __fmaf_rn(mu, m.v[i], g.v[i]);      // m' = mu m + g
            p = __fmaf_rn(eta, m_new.v[i], e.v[i]);          // p = eta m' + e
        } else {
            p = __fmaf_rn(eta, g.v[i], e.v[i]);              // p = eta g + e
        }
        const float c = SCALE ? __fmul_rn(delta, p) : (in[i] ? p : 0.0f);   // C(p)
        e_new.v[i] = __fsub_rn(p, c);                        // e' = p - C(p)
        sent[i] = first ? c : __fadd_rn(sent[i], c);         // running sum over the workers
    }
}

// All W workers of the V coordinates starting at local coordinate `col`, in worker order,
// U rows in flight at a time; then the average and the update on the coordinates that are in the block.
// With DETACH, a second walk over the rows writes the next iteration's gradient points
// z_w = x_{t+1} - lambda e_{w,t+1} (Algorithm 1's detach step); it re-reads the e' this thread has
// just written, which is still in cache.
template <int V, bool MOM, int U, int POL, bool DETACH = false, bool SCALE = false>
__device__ __forceinline__ void column_group(const StepArgs &a, int64_t s, int64_t col) {
    // offset of each coordinate from the block start, mod d; in the block iff < k
    int64_t off = a.j0 + col - s;
    if (off < 0) off += a.d;
    bool in[V];
    bool any = false;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        int64_t o = off + i;
        if (o >= a.d) o -= a.d;
        in[i] = SCALE || o < a.k;                           // the scaling compressor sends every coordinate
        any |= in[i];
    }
    float sent[V];
#pragma unroll
    for (int i = 0; i < V; ++i) sent[i] = 0.0f;
    const size_t ld = (size_t)a.ld;
    const float *gp = a.g + col;
    float *ep = a.e + col;
    float *mp = MOM ? a.m + col : nullptr;
    for (int w = 0; w < a.W; w += U) {
        Vec<V> g[U], e[U], m[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {                      // issue every load of the chunk first
            if (w + u < a.W) {
                const size_t row = (size_t)(w + u) * ld;
                g[u] = load_vec<V, POL>(gp + row);
                e[u] = load_vec<V, POL>(ep + row);
                if (MOM) m[u] = load_vec<V, POL>(mp + row);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {                      // then compute and store in worker order
            if (w + u < a.W) {
                const size_t row = (size_t)(w + u) * ld;
                Vec<V> m_new, e_new;
                worker_row<V, MOM, SCALE>(g[u], m[u], e[u], in, a.eta, a.mu, w + u == 0, m_new, e_new, sent, a.delta);
                if (MOM) store_vec<V, POL>(mp + row, m_new);
                store_vec<V, POL>(ep + row, e_new);
            }
        }
    }
    if (!DETACH) {
        if (any) {                                          // x -= (sum over workers) / W
#pragma unroll
            for (int i = 0; i < V; ++i) {
                if (in[i]) {
                    if (a.block_sum) {                      // the sum is finished by an all-reduce
                        int64_t o = off + i;
                        if (o >= a.d) o -= a.d;
                        a.block_sum[o] = sent[i];
                    } else {
                        const float C_pt = __fdiv_rn(sent[i], a.W_float);
                        a.x[col + i] = __fsub_rn(a.x[col + i], C_pt);
                    }
                }
            }
        }
        return;
    }
    Vec<V> x = load_vec<V, kCacheDefault>(a.x + col);
#pragma unroll
    for (int i = 0; i < V; ++i) {
        if (in[i]) {
            if (a.block_sum) {                              // rows sharded over GPUs: x_{t+1} is not known yet on a
                int64_t o = off + i;                        // block coordinate; z gets x_t there for now and the
                if (o >= a.d) o -= a.d;                     // apply kernel overwrites it after the all-reduce
                a.block_sum[o] = sent[i];
            } else {
                x.v[i] = __fsub_rn(x.v[i], __fdiv_rn(sent[i], a.W_float));
                a.x[col + i] = x.v[i];
            }
        }
    }
    float *zp = a.z + col;
    for (int w = 0; w < a.W; w += U) {
        Vec<V> e[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (w + u < a.W) e[u] = load_vec<V, kCacheDefault>(ep + (size_t)(w + u) * ld);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (w + u < a.W) {
                Vec<V> z;
#pragma unroll
                for (int i = 0; i < V; ++i) z.v[i] = __fmaf_rn(-a.lambda, e[u].v[i], x.v[i]);
                store_vec<V, POL>(zp + (size_t)(w + u) * ld, z);
            }
        }
    }
}

// General kernel: every thread owns V coordinates and walks all W rows.  Used for rows that
// are only 4- or 8-byte aligned (V = 1, 2) and for the n % 4 tail.  Rows must be aligned
// for V-wide access: x, g, e, m aligned to 4V bytes and ld % V == 0.
template <int V, bool MOM, int U, bool DETACH = false, bool SCALE = false>
__global__ void __launch_bounds__(256)
def_step_kernel(const StepArgs a) {
    const int64_t s = cta_block_start(a);
    const int64_t groups = a.n / V;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t grp = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < groups; grp += stride)
        column_group<V, MOM, U, kCacheDefault, DETACH, SCALE>(a, s, grp * V);
}

// Kernels for 16-byte aligned rows.  The n local coordinates are cut into tiles of
// TILE = kTileThreads * 4 coordinates.  A tile "touches the block" if any of its coordinates
// is one of the k block coordinates; every CTA decides that from the block start.
constexpr int kTileThreads = 256;
constexpr int64_t kTile = (int64_t)kTileThreads * 4;

// The tiles of the local range [j0, j0 + n) that touch the block {(s + i) mod d : i < k}.  The
// block is at most two runs of local coordinates (it may wrap past d, and the local range may cut
// it): run A = [s, min(s + k, d)) and, if the block wraps, run B = [0, s + k - d), both clipped to
// the local range.  B ends before s, so its tiles lie at or before A's first tile; a tile both
// runs reach counts for A.  Touched tiles are therefore tiles [0, b_count) and
// [a_first, a_first + a_count), disjoint and in this order.  (Host and device: the host sizes the
// grids from the same arithmetic.)
struct TouchedTiles {
    int64_t a_first, a_count, b_count;
};

__host__ __device__ __forceinline__ TouchedTiles touched_tiles(const StepArgs &a, int64_t s) {
    const int64_t lo = a.j0, hi = a.j0 + a.n;
    const int64_t a0 = s > lo ? s : lo;
    int64_t a1 = s + a.k < a.d ? s + a.k : a.d;
    a1 = a1 < hi ? a1 : hi;
    int64_t b1 = s + a.k - a.d;                                  // <= s; > 0 only if the block wraps
    b1 = b1 < hi ? b1 : hi;
    TouchedTiles t;
    t.a_first = 0; t.a_count = 0; t.b_count = 0;
    if (a1 > a0) {
        t.a_first = (a0 - lo) / kTile;
        t.a_count = (a1 - 1 - lo) / kTile - t.a_first + 1;
    }
    if (b1 > lo) {
        t.b_count = (b1 - 1 - lo) / kTile + 1;
        if (t.a_count > 0 && t.b_count > t.a_first) t.b_count = t.a_first;
    }
    return t;
}

// The u-th tile (in increasing order) that does NOT touch the block: skip the two runs.
__host__ __device__ __forceinline__ int64_t untouched_tile(const TouchedTiles &t, int64_t u) {
    int64_t tile = u + t.b_count;
    if (t.a_count > 0 && tile >= t.a_first) tile += t.a_count;
    return tile;
}

// Tiles that do not touch the block (all but about k / TILE + 2 of them) have nothing to
// sum: C(p) = 0 and e' = p.  CTA (i, w) does worker w's row of the i-th such tiles: three 16-byte
// loads and two stores per thread, few registers, full occupancy.  The grid holds CTAs for these
// tiles only -- the host sizes it from the same block start -- so no CTA is launched just to
// find that its tile belongs to the other kernel (with k = d/8 those were an eighth of the
// grid and cost 2 % of the step).  Consecutive CTAs sweep one row after the other, so the memory
// system sees a handful of long sequential streams.
// With DETACH the kernel also writes z_w = x - lambda e'_w for its row (x is unchanged outside
// the block), which makes x a sixth stream that every worker's CTA of a tile reads.  ORDER
// chooses how CTAs are numbered, i.e. what runs together:
//   kOrderRows     grid (tile slots, W): row after row, the flat stream.  (With DETACH, x would be
//                  re-read from HBM for every row: it is far larger than the L2.)
//   kOrderChunked  1-D grid: a.chunk consecutive CTAs sweep a segment of row 0, the next a.chunk
//                  the same segment of row 1, ...; then the next segment.  Long sequential
//                  streams, and the segment of x stays in the L2 until the last row has used it.
// TILES CTAs' worth of tiles share one CTA of TILES * kTileThreads threads (each group of
// kTileThreads threads still owns one tile).
constexpr int kOrderRows = 0, kOrderChunked = 1;

template <bool MOM, int POL, bool DETACH = false, int ORDER = kOrderRows, int TILES = 1>
__global__ void __launch_bounds__(kTileThreads * TILES)
def_step_stream_kernel(const StepArgs a) {
    int64_t first;
    unsigned w;
    if (ORDER == kOrderRows) {
        first = blockIdx.x; w = blockIdx.y;
    } else {
        const int64_t per_segment = (int64_t)a.W * a.chunk;
        const int64_t segment = (int64_t)blockIdx.x / per_segment;
        const int64_t rem = (int64_t)blockIdx.x - segment * per_segment;
        w = (unsigned)(rem / a.chunk);
        first = segment * a.chunk + rem % a.chunk;
    }
    // One thread draws the block start and works out which tiles touch the block; the others wait
    // for the three numbers.  (Every thread doing that arithmetic itself after the hand-over of s
    // cost the step without momentum, whose CTAs live shortest, 5 %, and the step with momentum
    // 0.4 % at four tiles per CTA.  Issuing the loads before
    // the hand-over is not possible here -- which tile a thread owns depends on it -- and was
    // slower when it was: see the design-variants program.)
    __shared__ TouchedTiles touched_shared;
    if (threadIdx.x == 0) touched_shared = touched_tiles(a, block_start(a.seed, a.step, a.d));
    __syncthreads();
    const TouchedTiles touched = touched_shared;
    const int64_t tile = untouched_tile(touched, first * TILES + (int64_t)(threadIdx.x / kTileThreads));
    const int64_t col = tile * kTile + (int64_t)(threadIdx.x % kTileThreads) * 4;
    if (col < a.n) {                                   // (slots past the last untouched tile land beyond n)
        const size_t at = (size_t)w * (size_t)a.ld + (size_t)col;
        const Vec<4> g = load_vec<4, POL>(a.g + at);
        const Vec<4> e = load_vec<4, POL>(a.e + at);
        Vec<4> m, x;
        if (MOM) m = load_vec<4, POL>(a.m + at);
        if (DETACH) x = load_vec<4, kCacheDefault>(a.x + col);
        Vec<4> m_new, e_new;
        const bool none[4] = {false, false, false, false};
        float unused[4];
        worker_row<4, MOM>(g, m, e, none, a.eta, a.mu, true, m_new, e_new, unused);
        if (MOM) store_vec<4, POL>(a.m + at, m_new);
        store_vec<4, POL>(a.e + at, e_new);
        if (DETACH) {
            Vec<4> z;
#pragma unroll
            for (int i = 0; i < 4; ++i) z.v[i] = __fmaf_rn(-a.lambda, e_new.v[i], x.v[i]);
            store_vec<4, POL>(a.z + at, z);
        }
    }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) grid_dependency_wait();
}

// Tiles that touch the block: one CTA per tile walks the W rows in order (column_group).
// A run of length L touches at most L / TILE + 2 tiles, so a grid of k / TILE + 4 CTAs covers
// every case.  CTA i takes the i-th touched tile: first those of run A, then those of run B.
// CTAs beyond the last touched tile leave.
// MINB: CTAs per SM the compiler is asked to make room for (it caps the registers accordingly).
template <bool MOM, int U, int POL, bool DETACH = false, int MINB = 3>
__global__ void __launch_bounds__(kTileThreads, MINB)
def_step_block_kernel(const StepArgs a) {
    // The stream kernel that follows in the stream works on other tiles and needs nothing from
    // this kernel: when it was launched with programmatic stream serialization, let its CTAs
    // start now instead of after this grid has drained (a no-op otherwise).
    release_dependent_grids();
    const int64_t s = cta_block_start(a);
    const TouchedTiles touched = touched_tiles(a, s);
    int64_t tile;
    if ((int64_t)blockIdx.x < touched.a_count) {
        tile = touched.a_first + blockIdx.x;
    } else {
        tile = (int64_t)blockIdx.x - touched.a_count;
        if (tile >= touched.b_count) return;
    }
    const int64_t col = tile * kTile + (int64_t)threadIdx.x * 4;
    if (col < a.n) column_group<4, MOM, U, POL, DETACH>(a, s, col);
}

// ---------------------------------------------------------------------------
// Contiguous [W, n] tensors whose rows are NOT 16-byte aligned (n % 4 != 0) but whose bases
// are: the part outside the block is still a plain stream, so it is run flat over the W * n
// floats with 16-byte accesses that ignore the row boundaries; every float finds its own
// (worker, coordinate) and skips itself if the coordinate is in the block.  The block
// coordinates -- exactly k of them -- are done beforehand by def_step_block_columns_kernel,
// one thread per coordinate walking the W rows in order with 4-byte accesses.  Both kernels
// have a DETACH variant that also writes the next detach points z = x_{t+1} - lambda e'.
// ---------------------------------------------------------------------------
constexpr int kFlatThreads = 512;
constexpr int64_t kFlatTile = (int64_t)kFlatThreads * 4;     // floats per CTA; needs n >= kFlatTile

template <bool MOM, int U, int POL, bool DETACH = false>
__global__ void __launch_bounds__(256)
def_step_block_columns_kernel(const StepArgs a) {
    // the flat kernel that follows touches no float of a block coordinate: let it start now
    // when it was launched with programmatic stream serialization
    release_dependent_grids();
    const int64_t s = cta_block_start(a);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // i-th block coordinate
    if (i >= a.k) return;
    int64_t j = s + i;
    if (j >= a.d) j -= a.d;
    const int64_t col = j - a.j0;
    if (col >= 0 && col < a.n) column_group<1, MOM, U, POL, DETACH>(a, s, col);
}

// The floats of one flat group of four, done one at a time: those that are not block coordinates
// and lie inside the tensor.  c is the coordinate of float f (the group may run on into the next row).
template <bool MOM, bool DETACH>
__device__ __forceinline__ void flat_group_by_floats(const StepArgs &a, int64_t f, int64_t c, int64_t total, const bool (&in)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (in[i] || f + i >= total) continue;
        Vec<1> g, e, m, m_new, e_new;
        g.v[0] = a.g[f + i];
        e.v[0] = a.e[f + i];
        if (MOM) m.v[0] = a.m[f + i];
        const bool no[1] = {false};
        float u1[1];
        worker_row<1, MOM>(g, m, e, no, a.eta, a.mu, true, m_new, e_new, u1);
        if (MOM) a.m[f + i] = m_new.v[0];
        a.e[f + i] = e_new.v[0];
        if (DETACH) {                                     // not a block coordinate: x does not change in this step
            int64_t ci = c + i;
            if (ci >= a.n) ci -= a.n;
            a.z[f + i] = __fmaf_rn(-a.lambda, e_new.v[0], a.x[ci]);
        }
    }
}

// x at the four coordinates of a flat group that starts at coordinate c (it may run on into the
// next row, i.e. wrap to coordinate 0): one 16-byte load where the group is aligned in x and whole.
__device__ __forceinline__ Vec<4> flat_group_x(const StepArgs &a, int64_t c) {
    Vec<4> x;
    if ((c & 3) == 0 && c + 4 <= a.n) return load_vec<4, kCacheDefault>(a.x + c);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int64_t ci = c + i;
        if (ci >= a.n) ci -= a.n;
        x.v[i] = a.x[ci];
    }
    return x;
}

// How many of the local coordinates [lo, hi) are block coordinates (runs A and B of touched_tiles,
// in local coordinates).
__device__ __forceinline__ int64_t block_coordinates_in(const StepArgs &a, int64_t s, int64_t lo, int64_t hi) {
    const int64_t end = a.j0 + a.n;
    int64_t a0 = (s > a.j0 ? s : a.j0) - a.j0;
    int64_t a1 = s + a.k < a.d ? s + a.k : a.d;
    a1 = (a1 < end ? a1 : end) - a.j0;
    int64_t b1 = s + a.k - a.d;
    b1 = (b1 < end ? b1 : end) - a.j0;
    int64_t count = 0;
    const int64_t al = lo > a0 ? lo : a0, ah = hi < a1 ? hi : a1;
    if (ah > al) count += ah - al;
    const int64_t bh = hi < b1 ? hi : b1;
    if (bh > lo) count += bh - lo;
    return count;
}

// One thread of the CTA draws the block start and sorts the CTA's kFlatTile floats into one of
// three kinds: none of them a block coordinate's (nearly every CTA: a plain 16-byte stream with no
// per-thread bookkeeping), all of them (nothing to do), or mixed (every float checked).
constexpr int kFlatPlain = 0, kFlatMixed = 1, kFlatIdle = 2;

// With DETACH the kernel also writes z = x - lambda e' for its floats (x does not change outside the
// block), which makes x a stream that every row reads.  The CTAs are then numbered so that x stays
// in the L2: the coordinates are cut into segments of kFlatSegment; grid (W * a.chunk, segments);
// CTA (r, seg) is the (r % a.chunk)-th of the flat CTAs whose first float lies in row r / a.chunk
// within segment seg.  Every flat CTA's first float lies in exactly one (row, segment), so each
// is done once; a (row, segment) holds a.chunk - 1 or a.chunk of them, the spare slot idles.
constexpr int64_t kFlatSegment = (int64_t)1 << 20;            // coordinates: 4 MB of x and of every row

template <bool MOM, int POL, bool DETACH = false>
__global__ void __launch_bounds__(kFlatThreads)
def_step_flat_kernel(const StepArgs a) {
    __shared__ int64_t shared[4];
    const int64_t total = (int64_t)a.W * a.n;                 // rows are contiguous: ld == n
    if (threadIdx.x == 0) {
        int64_t cta = blockIdx.x;                             // which run of kFlatTile floats
        int64_t kind = kFlatMixed;
        if (DETACH) {
            const int64_t w = (int64_t)blockIdx.x / a.chunk, i = (int64_t)blockIdx.x % a.chunk;
            const int64_t c_lo = (int64_t)blockIdx.y * kFlatSegment;
            const int64_t c_hi = c_lo + kFlatSegment < a.n ? c_lo + kFlatSegment : a.n;
            const int64_t first = (w * a.n + c_lo + kFlatTile - 1) / kFlatTile;
            const int64_t last = (w * a.n + c_hi + kFlatTile - 1) / kFlatTile;
            cta = first + i;
            if (cta >= last) kind = kFlatIdle;                // the spare slot of this (row, segment)
        }
        const int64_t base = cta * kFlatTile;
        const int64_t s = block_start(a.seed, a.step, a.d);
        const int64_t w0 = base / a.n;                        // worker of the CTA's first float
        const int64_t c0 = base - w0 * a.n;                   // and its coordinate
        if (kind != kFlatIdle && base + kFlatTile <= total) { // (the last, ragged CTA stays mixed)
            // the CTA's floats are coordinates [c0, c0 + kFlatTile) of one row, or -- n >= kFlatTile --
            // [c0, n) of one row and [0, c0 + kFlatTile - n) of the next
            const int64_t end = c0 + kFlatTile;
            int64_t inside = block_coordinates_in(a, s, c0, end < a.n ? end : a.n);
            if (end > a.n) inside += block_coordinates_in(a, s, 0, end - a.n);
            kind = inside == 0 ? kFlatPlain : inside == kFlatTile ? kFlatIdle : kFlatMixed;
        }
        shared[0] = s; shared[1] = c0; shared[2] = kind; shared[3] = base;
    }
    __syncthreads();
    const int64_t kind = shared[2];
    const int64_t f = shared[3] + (int64_t)threadIdx.x * 4;
    if (kind == kFlatPlain) {
        const bool none[4] = {false, false, false, false};
        float unused[4];
        const Vec<4> g = load_vec<4, POL>(a.g + f);
        const Vec<4> e = load_vec<4, POL>(a.e + f);
        Vec<4> m, m_new, e_new, x;
        if (MOM) m = load_vec<4, POL>(a.m + f);
        if (DETACH) {
            int64_t c = shared[1] + (int64_t)threadIdx.x * 4;
            if (c >= a.n) c -= a.n;
            x = flat_group_x(a, c);
        }
        worker_row<4, MOM>(g, m, e, none, a.eta, a.mu, true, m_new, e_new, unused);
        if (MOM) store_vec<4, POL>(a.m + f, m_new);
        store_vec<4, POL>(a.e + f, e_new);
        if (DETACH) {
            Vec<4> z;
#pragma unroll
            for (int i = 0; i < 4; ++i) z.v[i] = __fmaf_rn(-a.lambda, e_new.v[i], x.v[i]);
            store_vec<4, POL>(a.z + f, z);
        }
    } else if (kind == kFlatMixed && f < total) {
        const int64_t s = shared[0];
        int64_t c = shared[1] + (int64_t)threadIdx.x * 4;    // < 2 n because n >= kFlatTile
        if (c >= a.n) c -= a.n;
        bool in[4];
        bool any = false, all = true;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t ci = c + i;                               // coordinate of float f + i (next row after a wrap)
            if (ci >= a.n) ci -= a.n;
            int64_t off = a.j0 + ci - s;
            if (off < 0) off += a.d;
            in[i] = off < a.k;
            any |= in[i];
            all &= in[i];
        }
        if (!any && f + 4 <= total) {
            const bool none[4] = {false, false, false, false};
            float unused[4];
            const Vec<4> g = load_vec<4, POL>(a.g + f);
            const Vec<4> e = load_vec<4, POL>(a.e + f);
            Vec<4> m, m_new, e_new, x;
            if (MOM) m = load_vec<4, POL>(a.m + f);
            if (DETACH) x = flat_group_x(a, c);
            worker_row<4, MOM>(g, m, e, none, a.eta, a.mu, true, m_new, e_new, unused);
            if (MOM) store_vec<4, POL>(a.m + f, m_new);
            store_vec<4, POL>(a.e + f, e_new);
            if (DETACH) {
                Vec<4> z;
#pragma unroll
                for (int i = 0; i < 4; ++i) z.v[i] = __fmaf_rn(-a.lambda, e_new.v[i], x.v[i]);
                store_vec<4, POL>(a.z + f, z);
            }
        } else if (!all) {
            // a group that straddles an edge of the block, or the last W * n % 4 floats: float by
            // float, touching nothing that is in the block (whose floats belong to the other kernel)
            flat_group_by_floats<MOM, DETACH>(a, f, c, total, in);
        }
    }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) grid_dependency_wait();
}

// Second half of a row-sharded step (Algorithm 1's update after the all-reduce):
// x[(s + i) mod d] -= block_sum[i] / W_total for the k block coordinates.  With z set it also
// writes the next detach point of the W_local local workers there: e' = +0 on a block
// coordinate, so z[w, j] = x_{t+1}[j] for every w.
__global__ void __launch_bounds__(256)
def_apply_block_kernel(float *__restrict__ x, const float *__restrict__ block_sum, float *__restrict__ z,
                       int W_local, StepArgs a) {
    const int64_t s = cta_block_start(a);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.k) return;
    int64_t j = s + i;
    if (j >= a.d) j -= a.d;
    const float x_new = __fsub_rn(x[j], __fdiv_rn(block_sum[i], a.W_float));
    x[j] = x_new;
    if (z)
        for (int w = 0; w < W_local; ++w) z[(size_t)w * (size_t)a.ld + (size_t)j] = x_new;
}

}  // namespace defk
