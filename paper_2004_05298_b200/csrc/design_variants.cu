// Timing of design alternatives for the step's kernels on one B200.
//
// Not part of the library: a stand-alone program (built and run by
// paper_2004_05298_b200/design_variants.py) that backs the design decisions with numbers.
// It times, on [W, d] fp32 tensors of the benchmark's size,
//   * the streaming part of the step (m' = mu m + g, p = eta m' + e, e' = p: 3 reads and
//     2 writes of 4 bytes per gradient element) written several ways: a flat 128-bit stream,
//     the same with evict-first cache hints, 256-bit accesses, a persistent grid-stride loop,
//     one thread walking all W rows of its columns, and 1-D bulk asynchronous copies through
//     shared memory;
//   * the library's own stream kernel as shipped, and a stream kernel whose grid covers all tiles
//     (CTAs of tiles that touch the block idle) with the block start obtained in three ways:
//     per CTA before the loads, per CTA after the loads have been issued, and passed in by the
//     host, which is the bound on what hiding that latency can gain;
//   * the library's block kernel (tiles that touch the block) for 2 / 4 / 8 rows in flight and
//     1..4 CTAs per SM requested from the compiler.
// Every kernel here does the arithmetic of the step; none is timed with work left out.
#include "def_kernels.cuh"

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <string>
#include <vector>

namespace {

using defk::StepArgs;
using defk::Vec;

#define CHECK(call)                                                                          \
    do {                                                                                     \
        cudaError_t err_ = (call);                                                           \
        if (err_ != cudaSuccess) {                                                           \
            fprintf(stderr, "%s:%d: %s\n", __FILE__, __LINE__, cudaGetErrorString(err_));    \
            exit(1);                                                                         \
        }                                                                                    \
    } while (0)

// Deterministic small values (no library generator needed): a hash of the index.
__global__ void fill_kernel(float *p, size_t n, uint32_t salt, float scale) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        uint32_t h = (uint32_t)i * 2654435761u ^ salt;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        p[i] = scale * ((float)(h & 0xffff) - 32768.0f) * (1.0f / 32768.0f);
    }
}

__device__ __forceinline__ void stream_math(const float (&g)[4], const float (&e)[4], const float (&m)[4],
                                            float eta, float mu, float (&m_new)[4], float (&e_new)[4]) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_new[i] = __fmaf_rn(mu, m[i], g[i]);
        e_new[i] = __fmaf_rn(eta, m_new[i], e[i]);
    }
}

// ---- flat 128-bit stream, one group of four floats per thread --------------------------------
template <int POL>
__global__ void __launch_bounds__(512)
flat128_kernel(const float *__restrict__ g, float *__restrict__ e, float *__restrict__ m, size_t n, float eta, float mu) {
    const size_t f = ((size_t)blockIdx.x * 512 + threadIdx.x) * 4;
    if (f + 4 > n) return;
    const Vec<4> gv = defk::load_vec<4, POL>(g + f), ev = defk::load_vec<4, POL>(e + f), mv = defk::load_vec<4, POL>(m + f);
    Vec<4> mn, en;
    stream_math(gv.v, ev.v, mv.v, eta, mu, mn.v, en.v);
    defk::store_vec<4, POL>(m + f, mn);
    defk::store_vec<4, POL>(e + f, en);
}

// ---- 256-bit accesses: eight floats per load / store -----------------------------------------
struct alignas(32) F8 { float v[8]; };
__device__ __forceinline__ F8 load256(const float *p) {
    F8 r;
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
                 : "l"(p));
    return r;
}
__device__ __forceinline__ void store256(float *p, const F8 &a) {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(a.v[0]), "f"(a.v[1]), "f"(a.v[2]),
                 "f"(a.v[3]), "f"(a.v[4]), "f"(a.v[5]), "f"(a.v[6]), "f"(a.v[7])
                 : "memory");
}
__global__ void __launch_bounds__(256)
flat256_kernel(const float *__restrict__ g, float *__restrict__ e, float *__restrict__ m, size_t n, float eta, float mu) {
    const size_t f = ((size_t)blockIdx.x * 256 + threadIdx.x) * 8;
    if (f + 8 > n) return;
    const F8 gv = load256(g + f), ev = load256(e + f), mv = load256(m + f);
    F8 mn, en;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        mn.v[i] = __fmaf_rn(mu, mv.v[i], gv.v[i]);
        en.v[i] = __fmaf_rn(eta, mn.v[i], ev.v[i]);
    }
    store256(m + f, mn);
    store256(e + f, en);
}

// ---- persistent grid: a fixed number of CTAs per SM, grid-stride loop --------------------------
__global__ void __launch_bounds__(512)
persistent_kernel(const float *__restrict__ g, float *__restrict__ e, float *__restrict__ m, size_t n, float eta, float mu) {
    const size_t stride = (size_t)gridDim.x * 512 * 4;
    for (size_t f = ((size_t)blockIdx.x * 512 + threadIdx.x) * 4; f + 4 <= n; f += stride) {
        const Vec<4> gv = defk::load_vec<4, 0>(g + f), ev = defk::load_vec<4, 0>(e + f), mv = defk::load_vec<4, 0>(m + f);
        Vec<4> mn, en;
        stream_math(gv.v, ev.v, mv.v, eta, mu, mn.v, en.v);
        defk::store_vec<4, 0>(m + f, mn);
        defk::store_vec<4, 0>(e + f, en);
    }
}

// ---- 1-D bulk asynchronous copies (the TMA engine without a tensor map) -----------------------
// One CTA per chunk of kBulkFloats floats of each tensor: one thread asks for the three chunks
// (global -> shared memory, completion counted in bytes on an mbarrier), every thread computes
// in shared memory, one thread sends m' and e' back (shared -> global).  Every wait is bounded:
// a CTA that gives up records it in *gave_up and leaves without touching its chunk.
constexpr int kBulkThreads = 256;
constexpr int kBulkFloats = 4096;                      // 16 KB per tensor per CTA, 48 KB of shared memory

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(kBulkThreads)
bulk_kernel(const float *__restrict__ g, float *__restrict__ e, float *__restrict__ m, size_t n, float eta, float mu,
            int *gave_up) {
    extern __shared__ __align__(128) float tile[];     // g | e | m, kBulkFloats each
    __shared__ __align__(8) uint64_t bar;
    float *sg = tile, *se = tile + kBulkFloats, *sm = tile + 2 * kBulkFloats;
    const size_t base = (size_t)blockIdx.x * kBulkFloats;
    if (base >= n) return;
    const size_t left = n - base;
    const uint32_t count = (uint32_t)(left < (size_t)kBulkFloats ? left : (size_t)kBulkFloats);   // multiple of 4
    const uint32_t bytes = count * 4u;
    const uint32_t bar_a = smem_addr(&bar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(3u * bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(sg)), "l"(g + base), "r"(bytes), "r"(bar_a) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(se)), "l"(e + base), "r"(bytes), "r"(bar_a) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(sm)), "l"(m + base), "r"(bytes), "r"(bar_a) : "memory");
    }
    uint32_t done = 0;
    for (int spin = 0; spin < (1 << 20) && !done; ++spin)
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done) : "r"(bar_a) : "memory");
    if (!done) {                                       // never seen in practice; no copy is re-issued
        if (threadIdx.x == 0) atomicAdd(gave_up, 1);
        return;
    }
    for (uint32_t i = threadIdx.x * 4; i < count; i += kBulkThreads * 4) {
        const float4 gv = *reinterpret_cast<const float4 *>(sg + i);
        const float4 ev = *reinterpret_cast<const float4 *>(se + i);
        const float4 mv = *reinterpret_cast<const float4 *>(sm + i);
        const float gg[4] = {gv.x, gv.y, gv.z, gv.w}, ee[4] = {ev.x, ev.y, ev.z, ev.w}, mm[4] = {mv.x, mv.y, mv.z, mv.w};
        float mn[4], en[4];
        stream_math(gg, ee, mm, eta, mu, mn, en);
        *reinterpret_cast<float4 *>(sm + i) = make_float4(mn[0], mn[1], mn[2], mn[3]);
        *reinterpret_cast<float4 *>(se + i) = make_float4(en[0], en[1], en[2], en[3]);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stores above, before the engine reads them
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(m + base), "r"(smem_addr(sm)), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(e + base), "r"(smem_addr(se)), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // shared memory must outlive the reads
    }
}

// ---- a stream kernel over ALL tiles, with the block start obtained in three ways ---------------
// Grid (tile pairs, W) over every tile; a CTA whose tile touches the block stores nothing (the
// library's kernel before its grid was cut down to the tiles it works on).
// MODE 0: block start per CTA (Philox by one thread, handed over through shared memory), then loads.
// MODE 1: the three loads are issued before that hand-over.
// MODE 2: the start is a kernel argument (no Philox, no barrier) -- what hiding the latency can gain at most.
__device__ __forceinline__ bool tile_touches_block(const StepArgs &a, int64_t s, int64_t tile) {
    const int64_t tile0 = tile * defk::kTile;
    const int64_t tile_len = (a.n - tile0 < defk::kTile) ? a.n - tile0 : defk::kTile;
    int64_t off0 = a.j0 + tile0 - s;                 // offset of the tile's start from s, mod d
    if (off0 < 0) off0 += a.d;
    return off0 < a.k || off0 + tile_len > a.d;      // starts inside the block, or wraps onto its start
}

template <int MODE>
__global__ void __launch_bounds__(512)
stream_variant_kernel(const StepArgs a, int64_t s_from_host) {
    const int64_t tile = (int64_t)blockIdx.x * 2 + (int64_t)(threadIdx.x / defk::kTileThreads);
    const int64_t col = tile * defk::kTile + (int64_t)(threadIdx.x % defk::kTileThreads) * 4;
    const bool live = col < a.n;
    const size_t at = (size_t)blockIdx.y * (size_t)a.ld + (size_t)col;
    Vec<4> g, e, m;
    if (MODE == 1 && live) {
        g = defk::load_vec<4, 0>(a.g + at); e = defk::load_vec<4, 0>(a.e + at); m = defk::load_vec<4, 0>(a.m + at);
    }
    const int64_t s = MODE == 2 ? s_from_host : defk::cta_block_start(a);
    if (live && !tile_touches_block(a, s, tile)) {
        if (MODE != 1) {
            g = defk::load_vec<4, 0>(a.g + at); e = defk::load_vec<4, 0>(a.e + at); m = defk::load_vec<4, 0>(a.m + at);
        }
        Vec<4> mn, en;
        stream_math(g.v, e.v, m.v, a.eta, a.mu, mn.v, en.v);
        defk::store_vec<4, 0>(a.m + at, mn);
        defk::store_vec<4, 0>(a.e + at, en);
    }
}

// ---- the library's stream kernel with the tile plan handed in by the host: no per-CTA prologue ---
template <int TILES>
__global__ void __launch_bounds__(256 * TILES)
stream_hostplan_kernel(const StepArgs a, const defk::TouchedTiles touched) {
    const int64_t tile = defk::untouched_tile(touched, (int64_t)blockIdx.x * TILES + (int64_t)(threadIdx.x / defk::kTileThreads));
    const int64_t col = tile * defk::kTile + (int64_t)(threadIdx.x % defk::kTileThreads) * 4;
    if (col >= a.n) return;
    const size_t at = (size_t)blockIdx.y * (size_t)a.ld + (size_t)col;
    const Vec<4> g = defk::load_vec<4, 0>(a.g + at), e = defk::load_vec<4, 0>(a.e + at), m = defk::load_vec<4, 0>(a.m + at);
    Vec<4> mn, en;
    stream_math(g.v, e.v, m.v, a.eta, a.mu, mn.v, en.v);
    defk::store_vec<4, 0>(a.m + at, mn);
    defk::store_vec<4, 0>(a.e + at, en);
}

__global__ void empty_kernel() {}

// Device time per launch.  Back to back (one event pair around `reps` launches), or -- with a
// flush buffer larger than the L2 -- every launch from cold caches: the buffer is rewritten before
// each launch and each launch has its own event pair.
struct Timer {
    cudaEvent_t a, b;
    float *flush = nullptr;
    size_t flush_floats = 0;
    Timer() { CHECK(cudaEventCreate(&a)); CHECK(cudaEventCreate(&b)); }
    template <typename F> double ms(F launch, int reps) {
        for (int i = 0; i < 3; ++i) launch();
        CHECK(cudaDeviceSynchronize());
        double total = 0.0;
        if (!flush) {
            CHECK(cudaEventRecord(a));
            for (int i = 0; i < reps; ++i) launch();
            CHECK(cudaEventRecord(b));
            CHECK(cudaEventSynchronize(b));
            float t = 0.f;
            CHECK(cudaEventElapsedTime(&t, a, b));
            total = t;
        } else {
            for (int i = 0; i < reps; ++i) {
                fill_kernel<<<2048, 256>>>(flush, flush_floats, (uint32_t)i, 1.0f);
                CHECK(cudaEventRecord(a));
                launch();
                CHECK(cudaEventRecord(b));
                CHECK(cudaEventSynchronize(b));
                float t = 0.f;
                CHECK(cudaEventElapsedTime(&t, a, b));
                total += t;
            }
        }
        CHECK(cudaGetLastError());
        return total / reps;
    }
};

}  // namespace

template <int U, int MINB>
void launch_block(const StepArgs &a, unsigned grid) {
    defk::def_step_block_kernel<true, U, 0, false, MINB><<<grid, defk::kTileThreads>>>(a);
}

int main(int argc, char **argv) {
    int64_t d = 138357544, ratio = 32;
    int W = 16, reps = 10;
    bool cold = false;
    std::string only;
    for (int i = 1; i < argc; ++i) {
        if (!strcmp(argv[i], "--d") && i + 1 < argc) d = atoll(argv[++i]);
        else if (!strcmp(argv[i], "--W") && i + 1 < argc) W = atoi(argv[++i]);
        else if (!strcmp(argv[i], "--ratio") && i + 1 < argc) ratio = atoll(argv[++i]);
        else if (!strcmp(argv[i], "--reps") && i + 1 < argc) reps = atoi(argv[++i]);
        else if (!strcmp(argv[i], "--only") && i + 1 < argc) only = argv[++i];
        else if (!strcmp(argv[i], "--cold")) cold = true;
        else { fprintf(stderr, "usage: %s [--d D] [--W W] [--ratio R] [--reps N] [--cold] [--only substring]\n", argv[0]); return 2; }
    }
    if (d < 4096 || d % 4 != 0 || W < 1 || W > 64 || ratio < 1 || reps < 1) { fprintf(stderr, "need d %% 4 == 0, d >= 4096, 1 <= W <= 64\n"); return 2; }
    cudaDeviceProp prop;
    CHECK(cudaGetDeviceProperties(&prop, 0));
    if (prop.major != 10) { fprintf(stderr, "needs a compute capability 10.x device\n"); return 1; }
    const size_t n = (size_t)W * (size_t)d;
    const int64_t k = d / ratio > 0 ? d / ratio : 1;
    float *g, *e, *m, *x;
    int *gave_up;
    CHECK(cudaMalloc(&g, n * 4)); CHECK(cudaMalloc(&e, n * 4)); CHECK(cudaMalloc(&m, n * 4)); CHECK(cudaMalloc(&x, (size_t)d * 4));
    CHECK(cudaMalloc(&gave_up, 4)); CHECK(cudaMemset(gave_up, 0, 4));
    fill_kernel<<<2048, 256>>>(g, n, 1u, 0.03f);
    fill_kernel<<<2048, 256>>>(x, (size_t)d, 2u, 0.05f);
    CHECK(cudaMemset(e, 0, n * 4)); CHECK(cudaMemset(m, 0, n * 4));
    CHECK(cudaDeviceSynchronize());
    CHECK(cudaFuncSetAttribute(bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 3 * kBulkFloats * 4));

    const float eta = 0.1f, mu = 0.9f;
    StepArgs a = {};
    a.x = x; a.g = g; a.e = e; a.m = m; a.n = d; a.ld = d; a.d = d; a.j0 = 0; a.k = k; a.W = W;
    a.eta = eta; a.mu = mu; a.W_float = (float)W; a.lambda = 0.3f; a.seed = 5; a.step = 0;
    const int64_t tiles = (d + defk::kTile - 1) / defk::kTile;
    const dim3 pair_grid((unsigned)((tiles + 1) / 2), (unsigned)W);
    const int64_t s0 = defk::block_start(a.seed, a.step, d);
    // bytes the variants move: the streams all of [W, d]; the library's stream kernel all tiles but those touching the block
    const double bytes_all = 20.0 * (double)n;
    int64_t touched = 0;
    for (int64_t t = 0; t < tiles; ++t) {
        int64_t off = t * defk::kTile - s0; if (off < 0) off += d;
        const int64_t len = d - t * defk::kTile < defk::kTile ? d - t * defk::kTile : defk::kTile;
        if (off < k || off + len > d) touched += len;
    }
    const double bytes_stream = 20.0 * (double)W * (double)(d - touched);
    const double bytes_block = 20.0 * (double)W * (double)touched + 8.0 * (double)k;
    const defk::TouchedTiles tt = defk::touched_tiles(a, s0);
    const unsigned block_grid = (unsigned)(tt.a_count + tt.b_count > 0 ? tt.a_count + tt.b_count : 1);
    const dim3 stream_grid((unsigned)((tiles - tt.a_count - tt.b_count + 3) / 4 > 0 ? (tiles - tt.a_count - tt.b_count + 3) / 4 : 1), (unsigned)W);

    Timer timer;
    if (cold) {                                        // 384 MB, three times the L2
        timer.flush_floats = (size_t)96 << 20;
        CHECK(cudaMalloc(&timer.flush, timer.flush_floats * 4));
    }
    printf("device: %s, %d SMs; W = %d, d = %lld, k = d/%lld = %lld, %d launches per figure, %s\n\n", prop.name,
           prop.multiProcessorCount, W, (long long)d, (long long)ratio, (long long)k, reps,
           cold ? "each launch from cold caches (384 MB rewritten before it, own event pair)" : "launches back to back");
    printf("| variant | ms | GB/s | bytes per launch |\n|---|---|---|---|\n");
    auto row = [&](const char *name, double bytes, auto launch) {
        if (!only.empty() && std::string(name).find(only) == std::string::npos) return;
        const double t = timer.ms(launch, reps);
        printf("| %s | %.4f | %.0f | %.3e |\n", name, t, bytes / (t * 1e-3) / 1e9, bytes);
        fflush(stdout);
    };
    row("empty kernel (what a launch costs by itself)", 0.0, [&] { empty_kernel<<<1, 32>>>(); });
    const unsigned g512 = (unsigned)((n / 4 + 511) / 512), g256x8 = (unsigned)((n / 8 + 255) / 256);
    row("flat stream, 128-bit, default caching, one group per thread", bytes_all, [&] { flat128_kernel<0><<<g512, 512>>>(g, e, m, n, eta, mu); });
    for (int per_sm : {3, 2, 1}) {                     // fewer resident CTAs: dynamic shared memory nobody uses caps them
        char name[112];
        snprintf(name, sizeof(name), "flat stream, 128-bit, at most %d CTAs of 512 per SM (instead of 4)", per_sm);
        const int smem = per_sm == 3 ? 60 * 1024 : per_sm == 2 ? 90 * 1024 : 120 * 1024;
        CHECK(cudaFuncSetAttribute(flat128_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        row(name, bytes_all, [&] { flat128_kernel<0><<<g512, 512, smem>>>(g, e, m, n, eta, mu); });
    }
    row("flat stream, 128-bit, ld.cs / st.cs", bytes_all, [&] { flat128_kernel<1><<<g512, 512>>>(g, e, m, n, eta, mu); });
    row("flat stream, 256-bit accesses", bytes_all, [&] { flat256_kernel<<<g256x8, 256>>>(g, e, m, n, eta, mu); });
    for (int per_sm : {2, 4}) {
        char name[96];
        snprintf(name, sizeof(name), "persistent grid-stride stream, %d CTAs of 512 per SM", per_sm);
        const unsigned grid = (unsigned)(prop.multiProcessorCount * per_sm);
        row(name, bytes_all, [&] { persistent_kernel<<<grid, 512>>>(g, e, m, n, eta, mu); });
    }
    {   // one thread walks all W rows of its four columns (the library's general kernel), nothing in the block
        StepArgs c = a; c.k = 1;
        const unsigned grid = (unsigned)((d / 4 + 255) / 256);
        row("column walk: one thread, all W rows of its 4 columns (def_step_kernel)", bytes_all,
            [&] { defk::def_step_kernel<4, true, 4><<<grid, 256>>>(c); });
    }
    row("1-D bulk async copies through shared memory (16 KB chunks)", bytes_all,
        [&] { bulk_kernel<<<(unsigned)((n + kBulkFloats - 1) / kBulkFloats), kBulkThreads, 3 * kBulkFloats * 4>>>(g, e, m, n, eta, mu, gave_up); });
    row("library stream kernel as shipped (tiles outside the block only, CTAs of 1024 threads)", bytes_stream,
        [&] { defk::def_step_stream_kernel<true, 0, false, defk::kOrderRows, 4><<<stream_grid, 1024>>>(a); });
    {   // CTA size x resident CTAs, for the library kernel (prologue per CTA) and for the host-plan kernel (none)
        const int64_t stream_tiles = tiles - tt.a_count - tt.b_count;
#define LIB_SHAPE(T, P) { auto k_ = defk::def_step_stream_kernel<true, 0, false, defk::kOrderRows, T>; \
        const int threads_ = 256 * T; int smem_ = 0; if (P < 2048 / threads_) smem_ = (227 * 1024 / (P + 1) + 1024) / 1024 * 1024; \
        if (smem_) CHECK(cudaFuncSetAttribute(k_, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_)); \
        char name_[128]; snprintf(name_, sizeof(name_), "library stream kernel, CTAs of %d threads, %d per SM", threads_, P); \
        const dim3 grid_((unsigned)((stream_tiles + T - 1) / T), (unsigned)W); \
        row(name_, bytes_stream, [&] { k_<<<grid_, threads_, smem_>>>(a); }); }
#define HOST_SHAPE(T, P) { auto k_ = stream_hostplan_kernel<T>; \
        const int threads_ = 256 * T; int smem_ = 0; if (P < 2048 / threads_) smem_ = (227 * 1024 / (P + 1) + 1024) / 1024 * 1024; \
        if (smem_) CHECK(cudaFuncSetAttribute(k_, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_)); \
        char name_[128]; snprintf(name_, sizeof(name_), "stream kernel with the tile plan from the host (no prologue), CTAs of %d threads, %d per SM", threads_, P); \
        const dim3 grid_((unsigned)((stream_tiles + T - 1) / T), (unsigned)W); \
        row(name_, bytes_stream, [&] { k_<<<grid_, threads_, smem_>>>(a, tt); }); }
        LIB_SHAPE(1, 8) LIB_SHAPE(1, 7) LIB_SHAPE(1, 6) LIB_SHAPE(2, 4) LIB_SHAPE(2, 3) LIB_SHAPE(3, 2) LIB_SHAPE(4, 2)
        HOST_SHAPE(1, 8) HOST_SHAPE(1, 7) HOST_SHAPE(1, 6) HOST_SHAPE(1, 5) HOST_SHAPE(2, 4) HOST_SHAPE(2, 3) HOST_SHAPE(3, 2) HOST_SHAPE(4, 2) HOST_SHAPE(4, 1)
#undef LIB_SHAPE
#undef HOST_SHAPE
    }
    row("stream kernel over all tiles, block start per CTA, then loads", bytes_stream,
        [&] { stream_variant_kernel<0><<<pair_grid, 512>>>(a, s0); });
    row("stream kernel over all tiles, loads issued before the block start is known", bytes_stream,
        [&] { stream_variant_kernel<1><<<pair_grid, 512>>>(a, s0); });
    row("stream kernel over all tiles, block start passed in by the host (bound)", bytes_stream,
        [&] { stream_variant_kernel<2><<<pair_grid, 512>>>(a, s0); });
    row("library block kernel, U = 2 rows in flight, min 1 CTA/SM", bytes_block, [&] { launch_block<2, 1>(a, block_grid); });
    row("library block kernel, U = 2, min 4 CTAs/SM", bytes_block, [&] { launch_block<2, 4>(a, block_grid); });
    row("library block kernel, U = 4, min 1 CTA/SM", bytes_block, [&] { launch_block<4, 1>(a, block_grid); });
    row("library block kernel, U = 4, min 3 CTAs/SM", bytes_block, [&] { launch_block<4, 3>(a, block_grid); });
    row("library block kernel, U = 4, min 4 CTAs/SM", bytes_block, [&] { launch_block<4, 4>(a, block_grid); });
    row("library block kernel, U = 8, min 1 CTA/SM", bytes_block, [&] { launch_block<8, 1>(a, block_grid); });
    row("library block kernel, U = 8, min 2 CTAs/SM", bytes_block, [&] { launch_block<8, 2>(a, block_grid); });
    int h = 0;
    CHECK(cudaMemcpy(&h, gave_up, 4, cudaMemcpyDeviceToHost));
    if (h) { fprintf(stderr, "bulk variant: %d CTAs gave up waiting\n", h); return 1; }
    CHECK(cudaFree(g)); CHECK(cudaFree(e)); CHECK(cudaFree(m)); CHECK(cudaFree(x)); CHECK(cudaFree(gave_up));
    return 0;
}
