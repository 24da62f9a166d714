// C boundary of the DEF / DEF-A / EF step library (see include/def.h): argument
// validation, kernel selection and launch, and the host-memory streaming path.
#include "../../include/def.h"
#include "def_kernels.cuh"
#include "def_aux_kernels.cuh"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

namespace {

thread_local char g_last_error[512] = "";

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t err, const char *what) {
    return fail(DEF_ERR_CUDA, "%s: %s", what, cudaGetErrorString(err));
}

constexpr int kThreads = 256;
constexpr int kHostSlots = 3;  // staging slots of the host-memory path

struct HostSlot {
    float *x = nullptr, *g = nullptr, *e = nullptr, *m = nullptr;
    cudaEvent_t loaded = nullptr, computed = nullptr, drained = nullptr;
    bool used = false;
};

}  // namespace

struct def_ctx {
    int64_t d = 0, k = 0;
    int32_t W = 0, variant = 0;
    float lr = 0.f, momentum = 0.f, lambda = 0.3f;
    cudaStream_t stream = nullptr;
    int64_t launches = 0;
    int64_t small_step_bytes = 0;  // set by def_create (kSmallStepBytesDefault)
    int32_t pair_overlap = DEF_OVERLAP_AUTO;
    int32_t compressor = DEF_COMPRESSOR_RBGS;
    float delta = 0.f;             // factor of DEF_COMPRESSOR_SCALE
    // per-kernel device times (profiling aid, off by default)
    bool timing = false;
    cudaEvent_t t_begin = nullptr, t_end = nullptr;
    double kernel_ms[DEF_KERNEL_KINDS] = {0.0, 0.0, 0.0};
    int64_t kernel_launches[DEF_KERNEL_KINDS] = {0, 0, 0};
    // device facts, filled by the first launching call
    bool device_checked = false;
    int device = -1;
    int sm_count = 0;
    // def_stats: per-CTA partial sums (allocated by the first def_stats call)
    double *stats_scratch = nullptr;
    // row-sharded step: the caller's side stream for the block kernel, the all-reduce and the
    // update (def_set_rows_stream), the events that fork it from and join it to `stream`, and
    // whether the last local half left block sums behind on `stream` itself
    cudaStream_t rows_stream = nullptr;
    cudaEvent_t rows_fork = nullptr, rows_join = nullptr;
    bool sums_on_main = false;
    // host-memory path
    bool host_ready = false;
    int64_t host_chunk = 0;  // coordinates per staging slot (multiple of 4)
    HostSlot slots[kHostSlots];
    cudaStream_t s_h2d = nullptr, s_run = nullptr, s_d2h = nullptr;
};

namespace {

int check_device(def_ctx *ctx) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return fail(DEF_ERR_DEVICE, "no usable CUDA device: %s", cudaGetErrorString(err));
    }
    if (ctx->device_checked && ctx->device == dev) return DEF_OK;
    cudaDeviceProp prop;
    err = cudaGetDeviceProperties(&prop, dev);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return fail(DEF_ERR_DEVICE, "cannot query device %d: %s", dev, cudaGetErrorString(err));
    }
    if (prop.major != 10)
        return fail(DEF_ERR_DEVICE, "device %d is compute capability %d.%d; this library is built for 10.x (sm_100a)",
                    dev, prop.major, prop.minor);
    ctx->device = dev;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->device_checked = true;
    return DEF_OK;
}

bool overlaps(const void *a, size_t a_bytes, const void *b, size_t b_bytes) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

// Bytes spanned by a [W, n] view with row stride ld, and by x[n].
size_t span_rows(int64_t W, int64_t n, int64_t ld) {
    return ((size_t)(W - 1) * (size_t)ld + (size_t)n) * sizeof(float);
}

int validate_tensors(const def_ctx *ctx, int64_t n, int64_t ld, const float *x, const float *g,
                     const float *e, const float *m) {
    if (!x || !g || !e) return fail(DEF_ERR_NULL, "params, grads and errors must not be NULL");
    if (ctx->momentum != 0.f && !m)
        return fail(DEF_ERR_NULL, "mom must not be NULL when momentum != 0");
    if (ctx->momentum == 0.f && m)
        return fail(DEF_ERR_ARG, "mom must be NULL when momentum == 0");
    const void *ptrs[4] = {x, g, e, m};
    const char *names[4] = {"params", "grads", "errors", "mom"};
    for (int i = 0; i < 4; ++i)
        if (ptrs[i] && ((uintptr_t)ptrs[i] & 3u))
            return fail(DEF_ERR_ALIGN, "%s is not 4-byte aligned", names[i]);
    const size_t bytes[4] = {(size_t)n * sizeof(float), span_rows(ctx->W, n, ld),
                             span_rows(ctx->W, n, ld), span_rows(ctx->W, n, ld)};
    for (int i = 0; i < 4; ++i)
        for (int j = i + 1; j < 4; ++j)
            if (ptrs[i] && ptrs[j] && overlaps(ptrs[i], bytes[i], ptrs[j], bytes[j]))
                return fail(DEF_ERR_ALIAS, "%s and %s overlap", names[i], names[j]);
    return DEF_OK;
}

// The optional detach output of a step: 4-byte aligned, overlapping none of the step's tensors.
int validate_detach_out(const def_ctx *ctx, int64_t n, int64_t ld, const float *z, const float *x,
                        const float *g, const float *e, const float *m) {
    if (!z) return fail(DEF_ERR_NULL, "detached_out must not be NULL");
    if ((uintptr_t)z & 3u) return fail(DEF_ERR_ALIGN, "detached_out is not 4-byte aligned");
    const size_t rows_b = span_rows(ctx->W, n, ld);
    if (overlaps(z, rows_b, x, (size_t)n * sizeof(float)) || overlaps(z, rows_b, g, rows_b) ||
        overlaps(z, rows_b, e, rows_b) || (m && overlaps(z, rows_b, m, rows_b)))
        return fail(DEF_ERR_ALIAS, "detached_out overlaps another tensor");
    return DEF_OK;
}

// Widest access every row of the view supports.
int vector_width(int64_t ld, const float *x, const float *g, const float *e, const float *m,
                 const float *z = nullptr) {
    uintptr_t bits = (uintptr_t)x | (uintptr_t)g | (uintptr_t)e | (uintptr_t)m | (uintptr_t)z;
    if ((bits & 15u) == 0 && ld % 4 == 0) return 4;
    if ((bits & 7u) == 0 && ld % 2 == 0) return 2;
    return 1;
}

// Rows in flight per thread on the tiles that touch the block (4 keeps the block kernel under
// 96 registers, two CTAs per SM; 8 rows measured no faster and costs a CTA of occupancy), and
// the cache policy of the [W, d] traffic (default caching measured 1.5 % faster than ld.cs/st.cs).
constexpr int kBlockRows = 4;
constexpr int kPolicy = defk::kCacheDefault;

// Runs `launch` (one kernel launch on `stream`), counts it, and in timing mode brackets it
// with events and waits for it so that its device time can be added to the kernel's total.
template <typename Launch>
cudaError_t counted_launch(def_ctx *ctx, int kind, cudaStream_t stream, Launch launch) {
    if (ctx->timing) {
        cudaError_t err = cudaEventRecord(ctx->t_begin, stream);
        if (err != cudaSuccess) return err;
    }
    launch();
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    ctx->launches += 1;
    if (ctx->timing) {
        float ms = 0.f;
        if ((err = cudaEventRecord(ctx->t_end, stream)) != cudaSuccess) return err;
        if ((err = cudaEventSynchronize(ctx->t_end)) != cudaSuccess) return err;
        if ((err = cudaEventElapsedTime(&ms, ctx->t_begin, ctx->t_end)) != cudaSuccess) return err;
        ctx->kernel_ms[kind] += ms;
        ctx->kernel_launches[kind] += 1;
    }
    return cudaSuccess;
}

// Launch of the stream kernel right after the block kernel of the same step.  The two work on
// disjoint tiles, so the stream kernel is allowed to start while the block kernel still runs
// (programmatic stream serialization; the block kernel releases its dependents at once).  That
// hides the block kernel's latency-bound run on small and mid-sized models.  One thread of the
// stream kernel ends with a wait for the block kernel's grid, so whatever is enqueued later, being
// ordered behind the stream kernel, is ordered behind both.  Not used in timing mode, where each
// kernel is measured alone, under DEF_OVERLAP_NEVER, nor when the block kernel went to another
// stream (`beside` false: the two then overlap as work on two streams does).  DEF_OVERLAP_AUTO
// overlaps at every size: side by side was at least as fast as one after the other wherever it
// was measured (1 MB to 44 GB per step, k from d/1000 to d/8).
template <typename Kernel>
cudaError_t launch_beside_block_kernel(const def_ctx *ctx, Kernel kernel, dim3 grid, unsigned threads,
                                       cudaStream_t stream, const defk::StepArgs &a, bool beside = true) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed =
        (ctx->timing || !beside || ctx->pair_overlap == DEF_OVERLAP_NEVER) ? 0 : 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

// With the fused detach output x becomes a stream every worker's CTA of a tile reads.  The
// stream kernel then runs in chunked order: 256 CTAs (four tiles each with momentum: 4 MB of
// every row and of x) sweep a segment of row 0, the next 256 the same segment of row 1, and so
// on, so the streams stay long and sequential while the segment of x stays in the L2 for all W
// rows.  Measured on the VGG-16-sized workload: 7.91 ms, against 8.78 ms with the W CTAs of a
// tile adjacent and 8.97 ms row after row (x re-read from HBM for every row).
constexpr int kDetachChunkCtas = 256;

// Steps that move fewer bytes than this run as ONE launch of the general kernel instead of the
// kernel pair.  From cold caches (L2 flushed before every step) the single launch is 1 us ahead up
// to about 20 MB (8.2 vs 9.2 us at 1-5 MB, 10.2 vs 11.3 at 21 MB), level at 80 MB (19.4 us both)
// and behind from the 137 MB ResNet-56-sized workload on (28.7 vs 27.6 us; 55.3 vs 54.3 at
// 320 MB); stepped back to back out of the L2, where the launches themselves are the bound, it
// leads up to 137 MB (6.2 vs 8.2 us at 1 MB, 10.4 vs 10.5 at 80 MB, 14.6 vs 16.4 at 137 MB) and
// trails from 320 MB (52.7 vs 49.5 us).  Hence 128 MiB.
// def_set_small_step_bytes changes it per context.
constexpr int64_t kSmallStepBytesDefault = (int64_t)128 << 20;

// `block_stream`: where the kernel of the tiles that touch the block goes when the step runs as a
// pair (the row-sharded step puts it on a side stream so that the all-reduce of the block sums
// can follow it there while the stream kernel runs); equal to `stream` otherwise.
template <int V, bool MOM, bool DETACH>
cudaError_t launch_one(def_ctx *ctx, const defk::StepArgs &a, cudaStream_t stream, cudaStream_t block_stream) {
    const int64_t groups = a.n / V;
    if (groups == 0) return cudaSuccess;
    if (ctx->compressor == DEF_COMPRESSOR_SCALE) {   // dense: every coordinate is sent and updated
        const int64_t want = (groups + kThreads - 1) / kThreads;
        if (want > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
        return counted_launch(ctx, DEF_KERNEL_GENERAL, stream, [&] {
            defk::def_step_kernel<V, MOM, 4, DETACH, true><<<(unsigned)want, kThreads, 0, stream>>>(a);
        });
    }
    if (V == 4 && 20 * (int64_t)a.W * a.n >= ctx->small_step_bytes) {
        const int64_t tiles = (a.n + defk::kTile - 1) / defk::kTile;
        if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
        // Each kernel gets CTAs for its own tiles only.  The host draws the block start with the
        // same function the kernels use (they still draw it themselves) to count them.
        const defk::TouchedTiles touched = defk::touched_tiles(a, defk::block_start(a.seed, a.step, a.d));
        const int64_t block_ctas = touched.a_count + touched.b_count;
        const int64_t stream_tiles = tiles - block_ctas;
        // the few tiles that touch the block first, then the stream over all the others
        const unsigned block_grid = (unsigned)(block_ctas > 0 ? block_ctas : 1);
        const bool beside = block_stream == stream;
        cudaError_t err = counted_launch(ctx, DEF_KERNEL_BLOCK, block_stream, [&] {
            defk::def_step_block_kernel<MOM, kBlockRows, kPolicy, DETACH><<<block_grid, defk::kTileThreads, 0, block_stream>>>(a);
        });
        if (err != cudaSuccess) return err;
        // Tiles per CTA of the stream kernel, i.e. CTAs of 256 times this many threads, two or four
        // of them resident per SM.  With momentum (3 loads, 2 stores per thread) CTAs of 1024
        // threads ran the VGG-16-, ResNet-50- and ResNet-18-sized steps 1.2 / 0.9 / 0.7 % faster than
        // CTAs of 512, and the step with the detach output 0.9 %; without momentum (2 loads, 1 store)
        // they ran it 5 % slower, and CTAs of 768 threads 15 % slower.
        constexpr int kStreamTiles = MOM ? 4 : 2;
        int64_t slots = (stream_tiles + kStreamTiles - 1) / kStreamTiles;
        if (slots < 1) slots = 1;                       // k = d: nothing to stream; one idle CTA keeps the pair a pair
        if constexpr (DETACH) {
            const int64_t segments = (slots + kDetachChunkCtas - 1) / kDetachChunkCtas;
            const int64_t ctas = segments * kDetachChunkCtas * a.W;
            if (ctas > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
            defk::StepArgs c = a;
            c.chunk = kDetachChunkCtas;
            return counted_launch(ctx, DEF_KERNEL_STREAM, stream, [&] {
                launch_beside_block_kernel(ctx, defk::def_step_stream_kernel<MOM, kPolicy, true, defk::kOrderChunked, kStreamTiles>,
                                           dim3((unsigned)ctas), defk::kTileThreads * kStreamTiles, stream, c, beside);
            });
        }
        else {
            const dim3 grid((unsigned)slots, (unsigned)a.W);
            return counted_launch(ctx, DEF_KERNEL_STREAM, stream, [&] {
                launch_beside_block_kernel(ctx, defk::def_step_stream_kernel<MOM, kPolicy, false, defk::kOrderRows, kStreamTiles>,
                                           grid, defk::kTileThreads * kStreamTiles, stream, a, beside);
            });
        }
    }
    // One group of V coordinates per thread; the grid-stride loop only covers the case of
    // more groups than one grid can hold.
    const int64_t want = (groups + kThreads - 1) / kThreads;
    const int64_t cap = 0x7fffffffLL;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    if (a.block_sum) ctx->sums_on_main = true;
    return counted_launch(ctx, DEF_KERNEL_GENERAL, stream, [&] {
        defk::def_step_kernel<V, MOM, 4, DETACH><<<grid, kThreads, 0, stream>>>(a);
    });
}

template <int V>
cudaError_t launch_v(def_ctx *ctx, const defk::StepArgs &a, cudaStream_t stream, cudaStream_t block_stream) {
    if (a.z) return a.m ? launch_one<V, true, true>(ctx, a, stream, block_stream) : launch_one<V, false, true>(ctx, a, stream, block_stream);
    return a.m ? launch_one<V, true, false>(ctx, a, stream, block_stream) : launch_one<V, false, false>(ctx, a, stream, block_stream);
}

// Enqueue the step on local coordinates [0, n) of a view; counts launches.
int enqueue_columns(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *x, const float *g,
                    float *e, float *m, uint64_t step, uint64_t seed, cudaStream_t stream,
                    float *z = nullptr, float *block_sum = nullptr, cudaStream_t block_stream = nullptr) {
    if (n == 0) return DEF_OK;
    if (!block_sum || !block_stream) block_stream = stream;
    defk::StepArgs a;
    a.x = x; a.g = g; a.e = e; a.m = m; a.z = z; a.block_sum = block_sum; a.lambda = ctx->lambda; a.delta = ctx->delta;
    a.n = n; a.ld = ld; a.d = ctx->d; a.j0 = j0; a.k = ctx->k; a.W = ctx->W;
    a.eta = ctx->lr; a.mu = ctx->momentum; a.W_float = (float)ctx->W;
    a.seed = seed; a.step = step; a.chunk = 0;
    const int V = vector_width(ld, x, g, e, m, z);
    cudaError_t err = cudaSuccess;
    // Contiguous rows that are not 16-byte aligned but whose bases are: block coordinates by one
    // kernel, everything else as a flat stream that ignores the row boundaries.
    const bool flat_ok = V < 4 && ld == n && n >= defk::kFlatTile &&
                         ctx->compressor == DEF_COMPRESSOR_RBGS &&
                         (((uintptr_t)g | (uintptr_t)e | (uintptr_t)m | (uintptr_t)z | (uintptr_t)(z ? x : nullptr)) & 15u) == 0 &&
                         20 * (int64_t)ctx->W * n >= ctx->small_step_bytes;
    if (flat_ok) {
        const int64_t block_grid = (ctx->k + 255) / 256;
        const int64_t flat_ctas = ((int64_t)ctx->W * n + defk::kFlatTile - 1) / defk::kFlatTile;
        dim3 flat_grid((unsigned)flat_ctas);
        if (z) {   // chunked order: (row, segment of coordinates) by (slot in it), so that x stays in the L2
            const int64_t segment = n < defk::kFlatSegment ? n : defk::kFlatSegment;
            const int64_t slots = (segment + defk::kFlatTile - 1) / defk::kFlatTile;
            const int64_t segments = (n + defk::kFlatSegment - 1) / defk::kFlatSegment;
            if (segments > 65535 || slots * ctx->W > 0x7fffffffLL) return fail(DEF_ERR_ARG, "problem too large for one grid");
            a.chunk = (int32_t)slots;
            flat_grid = dim3((unsigned)(slots * ctx->W), (unsigned)segments);
        }
        if (block_grid > 0x7fffffffLL || flat_ctas > 0x7fffffffLL) return fail(DEF_ERR_ARG, "problem too large for one grid");
        const bool beside = block_stream == stream;
        err = counted_launch(ctx, DEF_KERNEL_BLOCK, block_stream, [&] {
            const unsigned grid = (unsigned)block_grid;
            if (m && z) defk::def_step_block_columns_kernel<true, 8, kPolicy, true><<<grid, 256, 0, block_stream>>>(a);
            else if (m) defk::def_step_block_columns_kernel<true, 8, kPolicy, false><<<grid, 256, 0, block_stream>>>(a);
            else if (z) defk::def_step_block_columns_kernel<false, 8, kPolicy, true><<<grid, 256, 0, block_stream>>>(a);
            else defk::def_step_block_columns_kernel<false, 8, kPolicy, false><<<grid, 256, 0, block_stream>>>(a);
        });
        if (err != cudaSuccess) return cuda_fail(err, "def_step block-columns kernel launch");
        err = counted_launch(ctx, DEF_KERNEL_STREAM, stream, [&] {
            if (m && z) launch_beside_block_kernel(ctx, defk::def_step_flat_kernel<true, kPolicy, true>, flat_grid, defk::kFlatThreads, stream, a, beside);
            else if (m) launch_beside_block_kernel(ctx, defk::def_step_flat_kernel<true, kPolicy, false>, flat_grid, defk::kFlatThreads, stream, a, beside);
            else if (z) launch_beside_block_kernel(ctx, defk::def_step_flat_kernel<false, kPolicy, true>, flat_grid, defk::kFlatThreads, stream, a, beside);
            else launch_beside_block_kernel(ctx, defk::def_step_flat_kernel<false, kPolicy, false>, flat_grid, defk::kFlatThreads, stream, a, beside);
        });
        if (err != cudaSuccess) return cuda_fail(err, "def_step flat kernel launch");
        return DEF_OK;
    }
    const int64_t body = n - n % V;
    if (body > 0) {
        a.n = body;
        err = V == 4 ? launch_v<4>(ctx, a, stream, block_stream) : V == 2 ? launch_v<2>(ctx, a, stream, block_stream)
                                                                            : launch_v<1>(ctx, a, stream, block_stream);
        if (err != cudaSuccess) return cuda_fail(err, "def_step kernel launch");
    }
    if (body < n) {  // the last n % V coordinates, one float at a time
        defk::StepArgs t = a;
        t.x = x + body; t.g = g + body; t.e = e + body; t.m = m ? m + body : nullptr;
        t.z = z ? z + body : nullptr;
        t.n = n - body; t.j0 = j0 + body;
        err = launch_v<1>(ctx, t, stream, block_stream);
        if (err != cudaSuccess) return cuda_fail(err, "def_step tail kernel launch");
    }
    return DEF_OK;
}

void free_host_path(def_ctx *ctx) {
    for (HostSlot &s : ctx->slots) {
        if (s.x) cudaFree(s.x);
        if (s.g) cudaFree(s.g);
        if (s.e) cudaFree(s.e);
        if (s.m) cudaFree(s.m);
        if (s.loaded) cudaEventDestroy(s.loaded);
        if (s.computed) cudaEventDestroy(s.computed);
        if (s.drained) cudaEventDestroy(s.drained);
        s = HostSlot();
    }
    if (ctx->s_h2d) cudaStreamDestroy(ctx->s_h2d);
    if (ctx->s_run) cudaStreamDestroy(ctx->s_run);
    if (ctx->s_d2h) cudaStreamDestroy(ctx->s_d2h);
    ctx->s_h2d = ctx->s_run = ctx->s_d2h = nullptr;
    ctx->host_ready = false;
}

int prepare_host_path(def_ctx *ctx) {
    if (ctx->host_ready) return DEF_OK;
    size_t free_b = 0, total_b = 0;
    cudaError_t err = cudaMemGetInfo(&free_b, &total_b);
    if (err != cudaSuccess) return cuda_fail(err, "cudaMemGetInfo");
    // One slot holds x plus g, e (and m) for `chunk` coordinates.  Aim at 512 MiB of row data per
    // slot (on the VGG-16-sized model: 0.53 s per step, against 0.56 s with 128 MiB pieces, 0.58 with
    // 64 MiB, 0.53 with 1 GiB and 0.54 with 2 GiB), but at an eighth of the model at most, so that
    // smaller models are still cut into enough pieces for the copies and the kernels to overlap, at
    // 16 MiB at least, and never at more than a quarter of the free memory in total.
    const int rows = ctx->W * (ctx->momentum != 0.f ? 3 : 2) + 1;
    const size_t per_coordinate = sizeof(float) * (size_t)rows;
    size_t piece_bytes = (size_t)ctx->d * per_coordinate / 8;
    if (piece_bytes > ((size_t)512 << 20)) piece_bytes = (size_t)512 << 20;
    if (piece_bytes < ((size_t)16 << 20)) piece_bytes = (size_t)16 << 20;
    int64_t chunk = (int64_t)(piece_bytes / per_coordinate);
    const int64_t by_memory = (int64_t)(free_b / 4 / kHostSlots / (sizeof(float) * (size_t)rows));
    if (chunk > by_memory) chunk = by_memory;
    if (chunk > ctx->d) chunk = ctx->d;
    chunk = (chunk + 3) / 4 * 4;
    if (chunk < 4) return fail(DEF_ERR_CUDA, "not enough free device memory for staging buffers");
    const size_t row_bytes = (size_t)chunk * sizeof(float);
    for (HostSlot &s : ctx->slots) {
        if ((err = cudaMalloc(&s.x, row_bytes)) != cudaSuccess ||
            (err = cudaMalloc(&s.g, row_bytes * ctx->W)) != cudaSuccess ||
            (err = cudaMalloc(&s.e, row_bytes * ctx->W)) != cudaSuccess ||
            (ctx->momentum != 0.f && (err = cudaMalloc(&s.m, row_bytes * ctx->W)) != cudaSuccess) ||
            (err = cudaEventCreateWithFlags(&s.loaded, cudaEventDisableTiming)) != cudaSuccess ||
            (err = cudaEventCreateWithFlags(&s.computed, cudaEventDisableTiming)) != cudaSuccess ||
            (err = cudaEventCreateWithFlags(&s.drained, cudaEventDisableTiming)) != cudaSuccess) {
            free_host_path(ctx);
            return cuda_fail(err, "allocating staging buffers");
        }
    }
    if ((err = cudaStreamCreateWithFlags(&ctx->s_h2d, cudaStreamNonBlocking)) != cudaSuccess ||
        (err = cudaStreamCreateWithFlags(&ctx->s_run, cudaStreamNonBlocking)) != cudaSuccess ||
        (err = cudaStreamCreateWithFlags(&ctx->s_d2h, cudaStreamNonBlocking)) != cudaSuccess) {
        free_host_path(ctx);
        return cuda_fail(err, "creating streams");
    }
    ctx->host_chunk = chunk;
    ctx->host_ready = true;
    return DEF_OK;
}

}  // namespace

extern "C" {

const char *def_last_error(void) { return g_last_error; }

def_ctx *def_create(int64_t d, int32_t W, int64_t k, int32_t variant, float lr, float momentum,
                    const float *coeffs) {
    g_last_error[0] = 0;
    if (d < 1) { fail(DEF_ERR_ARG, "d must be >= 1 (got %lld)", (long long)d); return nullptr; }
    if (W < 1 || W > DEF_MAX_WORKERS) {
        fail(DEF_ERR_ARG, "W must be in 1..%d (got %d)", DEF_MAX_WORKERS, W);
        return nullptr;
    }
    if (k < 1 || k > d) {
        fail(DEF_ERR_ARG, "k must be in 1..d (got k=%lld, d=%lld)", (long long)k, (long long)d);
        return nullptr;
    }
    if (variant != DEF_VARIANT_DEF && variant != DEF_VARIANT_DEF_A && variant != DEF_VARIANT_EF) {
        fail(DEF_ERR_ARG, "unknown variant %d", variant);
        return nullptr;
    }
    if (!std::isfinite(lr)) { fail(DEF_ERR_ARG, "lr must be finite"); return nullptr; }
    if (!(momentum >= 0.f && momentum < 1.f)) {
        fail(DEF_ERR_ARG, "momentum must be in [0, 1)");
        return nullptr;
    }
    float lambda = 0.3f;
    if (coeffs) {
        lambda = coeffs[0];
        if (!(lambda >= 0.f && lambda <= 1.f)) {
            fail(DEF_ERR_ARG, "coeffs[0] (lambda) must be in [0, 1]");
            return nullptr;
        }
        if (coeffs[1] != 0.f) {
            fail(DEF_ERR_UNSUPPORTED, "coeffs[1] (weight decay) must be 0: fold weight decay into the gradients");
            return nullptr;
        }
    }
    if (variant == DEF_VARIANT_EF) lambda = 0.f;
    def_ctx *ctx = new (std::nothrow) def_ctx();
    if (!ctx) { fail(DEF_ERR_ARG, "out of host memory"); return nullptr; }
    ctx->d = d; ctx->W = W; ctx->k = k; ctx->variant = variant;
    ctx->lr = lr; ctx->momentum = momentum; ctx->lambda = lambda;
    ctx->small_step_bytes = kSmallStepBytesDefault;
    return ctx;
}

int def_destroy(def_ctx *ctx) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    free_host_path(ctx);
    if (ctx->stats_scratch) cudaFree(ctx->stats_scratch);
    if (ctx->rows_fork) cudaEventDestroy(ctx->rows_fork);
    if (ctx->rows_join) cudaEventDestroy(ctx->rows_join);
    if (ctx->t_begin) cudaEventDestroy(ctx->t_begin);
    if (ctx->t_end) cudaEventDestroy(ctx->t_end);
    delete ctx;
    return DEF_OK;
}

int def_set_stream(def_ctx *ctx, void *cuda_stream) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (ctx->rows_stream && (void *)ctx->rows_stream == cuda_stream)
        return fail(DEF_ERR_ARG, "the context's stream must differ from its side stream");
    ctx->stream = (cudaStream_t)cuda_stream;
    return DEF_OK;
}

int def_set_lr(def_ctx *ctx, float lr) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (!std::isfinite(lr)) return fail(DEF_ERR_ARG, "lr must be finite");
    ctx->lr = lr;
    return DEF_OK;
}

int def_block_start(const def_ctx *ctx, uint64_t step, uint64_t seed, int64_t *start_out) {
    if (!ctx || !start_out) return fail(DEF_ERR_NULL, "ctx and start_out must not be NULL");
    *start_out = defk::block_start(seed, step, ctx->d);
    return DEF_OK;
}

int def_block_start_device(const uint64_t *seeds, const uint64_t *steps, const int64_t *ds,
                           int64_t n, int64_t *starts_out, void *cuda_stream) {
    if (!seeds || !steps || !ds || !starts_out) return fail(DEF_ERR_NULL, "NULL array");
    if (n < 0) return fail(DEF_ERR_ARG, "n must be >= 0");
    if (n == 0) return DEF_OK;
    const int64_t blocks = (n + 255) / 256;
    if (blocks > 0x7fffffffLL) return fail(DEF_ERR_ARG, "n too large");
    defk::block_start_batch_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(
        seeds, steps, ds, n, starts_out);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "block start kernel launch");
    return DEF_OK;
}

int def_tile_plan(const def_ctx *ctx, int64_t j0, int64_t n, uint64_t step, uint64_t seed, int64_t plan_out[4]) {
    if (!ctx || !plan_out) return fail(DEF_ERR_NULL, "ctx and plan_out must not be NULL");
    if (j0 < 0 || n < 1 || j0 > ctx->d || n > ctx->d - j0)
        return fail(DEF_ERR_ARG, "column range [%lld, %lld) is outside [0, %lld) or empty", (long long)j0,
                    (long long)(j0 + n), (long long)ctx->d);
    defk::StepArgs a = {};
    a.n = n; a.d = ctx->d; a.j0 = j0; a.k = ctx->k;
    const defk::TouchedTiles t = defk::touched_tiles(a, defk::block_start(seed, step, ctx->d));
    plan_out[0] = t.a_first; plan_out[1] = t.a_count; plan_out[2] = t.b_count;
    plan_out[3] = (n + defk::kTile - 1) / defk::kTile - t.a_count - t.b_count;
    return DEF_OK;
}

int def_launch_count(const def_ctx *ctx, int64_t *count_out) {
    if (!ctx || !count_out) return fail(DEF_ERR_NULL, "ctx and count_out must not be NULL");
    *count_out = ctx->launches;
    return DEF_OK;
}

int def_set_compressor(def_ctx *ctx, int32_t compressor, float delta) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (compressor == DEF_COMPRESSOR_RBGS) {
        ctx->compressor = compressor;
        return DEF_OK;
    }
    if (compressor != DEF_COMPRESSOR_SCALE) return fail(DEF_ERR_ARG, "unknown compressor %d", compressor);
    if (!(delta > 0.f && delta < 1.f)) return fail(DEF_ERR_ARG, "delta must be in (0, 1)");
    ctx->compressor = compressor;
    ctx->delta = delta;
    return DEF_OK;
}

int def_set_small_step_bytes(def_ctx *ctx, int64_t bytes) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (bytes < 0) return fail(DEF_ERR_ARG, "bytes must be >= 0");
    ctx->small_step_bytes = bytes;
    return DEF_OK;
}

int def_set_pair_overlap(def_ctx *ctx, int32_t mode) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (mode != DEF_OVERLAP_AUTO && mode != DEF_OVERLAP_NEVER && mode != DEF_OVERLAP_ALWAYS)
        return fail(DEF_ERR_ARG, "unknown overlap mode %d", mode);
    ctx->pair_overlap = mode;
    return DEF_OK;
}

int def_set_kernel_timing(def_ctx *ctx, int enable) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (enable && !ctx->t_begin) {
        int rc = check_device(ctx);
        if (rc != DEF_OK) return rc;
        cudaError_t err = cudaEventCreate(&ctx->t_begin);
        if (err == cudaSuccess) err = cudaEventCreate(&ctx->t_end);
        if (err != cudaSuccess) return cuda_fail(err, "creating timing events");
    }
    ctx->timing = enable != 0;
    return DEF_OK;
}

int def_kernel_time(const def_ctx *ctx, int kernel, double *total_ms_out, int64_t *launches_out) {
    if (!ctx || !total_ms_out || !launches_out) return fail(DEF_ERR_NULL, "NULL argument");
    if (kernel < 0 || kernel >= DEF_KERNEL_KINDS) return fail(DEF_ERR_ARG, "unknown kernel kind %d", kernel);
    *total_ms_out = ctx->kernel_ms[kernel];
    *launches_out = ctx->kernel_launches[kernel];
    return DEF_OK;
}

namespace {

// Shared checks of the per-coordinate helpers: a column view of n coordinates with row stride ld.
int check_view(const def_ctx *ctx, int64_t n, int64_t ld) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (n < 0 || n > ctx->d) return fail(DEF_ERR_ARG, "n=%lld is outside [0, d=%lld]", (long long)n, (long long)ctx->d);
    if (ld < n) return fail(DEF_ERR_ARG, "row stride ld=%lld is smaller than n=%lld", (long long)ld, (long long)n);
    return DEF_OK;
}

// Grid of the partial-sums kernel of def_stats: one CTA per 256 coordinate groups while that stays
// within the scratch (kStatsMaxCtas slots); beyond, a whole number of waves of resident CTAs
// (three of 256 threads per SM at its 64-80 registers), so that the tile-stride loop gives every
// SM the same work and there is no ragged last wave.
int64_t stats_grid(int64_t groups, int sm_count) {
    int64_t ctas = (groups + defk::kStatsThreads - 1) / defk::kStatsThreads;
    if (ctas > defk::kStatsMaxCtas) {
        const int64_t wave = (int64_t)(sm_count > 0 ? sm_count : 1) * 3;
        ctas = defk::kStatsMaxCtas / wave * wave;
        if (ctas < 1) ctas = defk::kStatsMaxCtas;
    }
    return ctas < 1 ? 1 : ctas;
}

// The two kernels of def_stats / def_stats_static: per-CTA partial sums into `scratch`, then one
// CTA that adds them.  The second is launched with programmatic stream serialization: it is set
// up while the first runs and waits (griddepcontrol.wait) for that grid to complete before it
// reads a partial sum, which takes its launch latency out of the call.
int launch_stats(const float *errors, int64_t n, int64_t ld, int W, float lambda, int V, int64_t ctas,
                 double *scratch, double *stats_out, cudaStream_t stream) {
    if (V == 4) defk::def_stats_partial_kernel<4, 8><<<(unsigned)ctas, defk::kStatsThreads, 0, stream>>>(errors, n, ld, W, scratch);
    else if (V == 2) defk::def_stats_partial_kernel<2, 8><<<(unsigned)ctas, defk::kStatsThreads, 0, stream>>>(errors, n, ld, W, scratch);
    else defk::def_stats_partial_kernel<1, 8><<<(unsigned)ctas, defk::kStatsThreads, 0, stream>>>(errors, n, ld, W, scratch);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "def_stats kernel launch");
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(defk::kStatsThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    err = cudaLaunchKernelEx(&cfg, defk::def_stats_final_kernel, (const double *)scratch, (int)ctas, W, lambda, stats_out);
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "def_stats final kernel launch");
    return DEF_OK;
}

int width_of(int64_t ld, const void *a, const void *b, const void *c) {
    const uintptr_t bits = (uintptr_t)a | (uintptr_t)b | (uintptr_t)c;
    if ((bits & 15u) == 0 && ld % 4 == 0) return 4;
    if ((bits & 7u) == 0 && ld % 2 == 0) return 2;
    return 1;
}

}  // namespace

int def_detach(def_ctx *ctx, int64_t n, int64_t ld, const float *params, const float *errors,
               float *detached_out) {
    int rc = check_view(ctx, n, ld);
    if (rc != DEF_OK) return rc;
    if (!params || !errors || !detached_out) return fail(DEF_ERR_NULL, "params, errors and detached_out must not be NULL");
    if (((uintptr_t)params | (uintptr_t)errors | (uintptr_t)detached_out) & 3u) return fail(DEF_ERR_ALIGN, "a pointer is not 4-byte aligned");
    const size_t rows_b = span_rows(ctx->W, n, ld), x_b = (size_t)n * sizeof(float);
    if (overlaps(detached_out, rows_b, errors, rows_b) || overlaps(detached_out, rows_b, params, x_b))
        return fail(DEF_ERR_ALIAS, "detached_out overlaps an input");
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    if (n == 0) return DEF_OK;
    const int V = width_of(ld, params, errors, detached_out);
    const int64_t groups = (n + V - 1) / V;
    const int64_t blocks = (groups + 255) / 256;
    if (blocks > 0x7fffffffLL) return fail(DEF_ERR_ARG, "n too large");
    if (V == 4) defk::def_detach_kernel<4, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, detached_out, n, ld, ctx->W, ctx->lambda);
    else if (V == 2) defk::def_detach_kernel<2, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, detached_out, n, ld, ctx->W, ctx->lambda);
    else defk::def_detach_kernel<1, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, detached_out, n, ld, ctx->W, ctx->lambda);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "def_detach kernel launch");
    ctx->launches += 1;
    return DEF_OK;
}

int def_output(def_ctx *ctx, int64_t n, int64_t ld, const float *params, const float *errors,
               float *model_out) {
    int rc = check_view(ctx, n, ld);
    if (rc != DEF_OK) return rc;
    if (!params || !model_out) return fail(DEF_ERR_NULL, "params and model_out must not be NULL");
    const bool averaged = ctx->variant == DEF_VARIANT_DEF;
    if (averaged && !errors) return fail(DEF_ERR_NULL, "errors must not be NULL for DEF_VARIANT_DEF");
    if (((uintptr_t)params | (uintptr_t)(averaged ? errors : nullptr) | (uintptr_t)model_out) & 3u)
        return fail(DEF_ERR_ALIGN, "a pointer is not 4-byte aligned");
    const size_t x_b = (size_t)n * sizeof(float);
    if (overlaps(model_out, x_b, params, x_b) || (averaged && overlaps(model_out, x_b, errors, span_rows(ctx->W, n, ld))))
        return fail(DEF_ERR_ALIAS, "model_out overlaps an input");
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    if (n == 0) return DEF_OK;
    if (!averaged) {   // DEF-A and EF return x_T itself
        cudaError_t err = cudaMemcpyAsync(model_out, params, x_b, cudaMemcpyDeviceToDevice, ctx->stream);
        if (err != cudaSuccess) return cuda_fail(err, "def_output copy");
        return DEF_OK;
    }
    const int V = width_of(ld, params, errors, model_out);
    const int64_t groups = (n + V - 1) / V;
    const int64_t blocks = (groups + 255) / 256;
    if (blocks > 0x7fffffffLL) return fail(DEF_ERR_ARG, "n too large");
    const float Wf = (float)ctx->W;
    if (V == 4) defk::def_output_kernel<4, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, model_out, n, ld, ctx->W, Wf);
    else if (V == 2) defk::def_output_kernel<2, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, model_out, n, ld, ctx->W, Wf);
    else defk::def_output_kernel<1, 8><<<(unsigned)blocks, 256, 0, ctx->stream>>>(params, errors, model_out, n, ld, ctx->W, Wf);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "def_output kernel launch");
    ctx->launches += 1;
    return DEF_OK;
}

int def_stats(def_ctx *ctx, int64_t n, int64_t ld, const float *errors, double *stats_out) {
    int rc = check_view(ctx, n, ld);
    if (rc != DEF_OK) return rc;
    if (!errors || !stats_out) return fail(DEF_ERR_NULL, "errors and stats_out must not be NULL");
    if (((uintptr_t)errors & 3u) || ((uintptr_t)stats_out & 7u)) return fail(DEF_ERR_ALIGN, "errors must be 4-byte and stats_out 8-byte aligned");
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    if (!ctx->stats_scratch) {
        cudaError_t err = cudaMalloc(&ctx->stats_scratch, sizeof(double) * 2 * defk::kStatsMaxCtas);
        if (err != cudaSuccess) return cuda_fail(err, "allocating def_stats scratch");
    }
    const int V = width_of(ld, errors, nullptr, nullptr);
    const int64_t groups = (n + V - 1) / V;
    const int64_t ctas = stats_grid(groups, ctx->sm_count);
    rc = launch_stats(errors, n, ld, ctx->W, ctx->lambda, V, ctas, ctx->stats_scratch, stats_out, ctx->stream);
    if (rc == DEF_OK) ctx->launches += 2;
    return rc;
}

int def_step_columns(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *params,
                     const float *grads, float *errors, float *mom, uint64_t step,
                     uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (j0 < 0 || n < 0 || j0 > ctx->d || n > ctx->d - j0)
        return fail(DEF_ERR_ARG, "column range [%lld, %lld) is outside [0, %lld)", (long long)j0,
                    (long long)(j0 + n), (long long)ctx->d);
    if (ld < n) return fail(DEF_ERR_ARG, "row stride ld=%lld is smaller than n=%lld", (long long)ld, (long long)n);
    if (n == 0) return DEF_OK;   // an empty column range (a rank with no columns) is a no-op
    int rc = validate_tensors(ctx, n, ld, params, grads, errors, mom);
    if (rc != DEF_OK) return rc;
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    return enqueue_columns(ctx, j0, n, ld, params, grads, errors, mom, step, seed, ctx->stream);
}

int def_step(def_ctx *ctx, float *params, const float *grads, float *errors, float *mom,
             uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    return def_step_columns(ctx, 0, ctx->d, ctx->d, params, grads, errors, mom, step, seed);
}

int def_step_columns_detach(def_ctx *ctx, int64_t j0, int64_t n, int64_t ld, float *params,
                            const float *grads, float *errors, float *mom, float *detached_out,
                            uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (j0 < 0 || n < 0 || j0 > ctx->d || n > ctx->d - j0)
        return fail(DEF_ERR_ARG, "column range [%lld, %lld) is outside [0, %lld)", (long long)j0,
                    (long long)(j0 + n), (long long)ctx->d);
    if (ld < n) return fail(DEF_ERR_ARG, "row stride ld=%lld is smaller than n=%lld", (long long)ld, (long long)n);
    if (n == 0) return DEF_OK;   // an empty column range (a rank with no columns) is a no-op
    int rc = validate_tensors(ctx, n, ld, params, grads, errors, mom);
    if (rc != DEF_OK) return rc;
    if ((rc = validate_detach_out(ctx, n, ld, detached_out, params, grads, errors, mom)) != DEF_OK) return rc;
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    return enqueue_columns(ctx, j0, n, ld, params, grads, errors, mom, step, seed, ctx->stream, detached_out);
}

int def_step_detach(def_ctx *ctx, float *params, const float *grads, float *errors, float *mom,
                    float *detached_out, uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    return def_step_columns_detach(ctx, 0, ctx->d, ctx->d, params, grads, errors, mom, detached_out, step, seed);
}

}  // extern "C"

namespace {

// First half of a row-sharded step; `params` and `z` are both NULL (plain) or both set (with the
// detach output).
int rows_local(def_ctx *ctx, const float *params, const float *grads, float *errors, float *mom,
               float *block_sum_out, float *z, uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (ctx->compressor != DEF_COMPRESSOR_RBGS)
        return fail(DEF_ERR_UNSUPPORTED, "row-sharded steps support the RBGS compressor only");
    if (!block_sum_out) return fail(DEF_ERR_NULL, "block_sum_out must not be NULL");
    if ((uintptr_t)block_sum_out & 3u) return fail(DEF_ERR_ALIGN, "block_sum_out is not 4-byte aligned");
    if (!grads || !errors) return fail(DEF_ERR_NULL, "grads and errors must not be NULL");
    if (ctx->momentum != 0.f && !mom) return fail(DEF_ERR_NULL, "mom must not be NULL when momentum != 0");
    if (ctx->momentum == 0.f && mom) return fail(DEF_ERR_ARG, "mom must be NULL when momentum == 0");
    if (((uintptr_t)grads | (uintptr_t)errors | (uintptr_t)mom) & 3u) return fail(DEF_ERR_ALIGN, "a tensor is not 4-byte aligned");
    const size_t rows_b = span_rows(ctx->W, ctx->d, ctx->d), bs_b = (size_t)ctx->k * sizeof(float);
    const size_t x_b = (size_t)ctx->d * sizeof(float);
    if (overlaps(grads, rows_b, errors, rows_b) || (mom && (overlaps(mom, rows_b, errors, rows_b) || overlaps(mom, rows_b, grads, rows_b))))
        return fail(DEF_ERR_ALIAS, "grads, errors and mom must not overlap");
    if (overlaps(block_sum_out, bs_b, grads, rows_b) || overlaps(block_sum_out, bs_b, errors, rows_b) ||
        (mom && overlaps(block_sum_out, bs_b, mom, rows_b)))
        return fail(DEF_ERR_ALIAS, "block_sum_out overlaps a tensor");
    if (z) {
        if (!params) return fail(DEF_ERR_NULL, "params must not be NULL");
        if ((uintptr_t)params & 3u) return fail(DEF_ERR_ALIGN, "params is not 4-byte aligned");
        if (overlaps(params, x_b, grads, rows_b) || overlaps(params, x_b, errors, rows_b) ||
            (mom && overlaps(params, x_b, mom, rows_b)) || overlaps(params, x_b, block_sum_out, bs_b))
            return fail(DEF_ERR_ALIAS, "params overlaps another tensor");
        int rc = validate_detach_out(ctx, ctx->d, ctx->d, z, params, grads, errors, mom);
        if (rc != DEF_OK) return rc;
        if (overlaps(z, rows_b, block_sum_out, bs_b)) return fail(DEF_ERR_ALIAS, "detached_out overlaps block_sum_out");
    }
    int rc = check_device(ctx);
    if (rc != DEF_OK) return rc;
    cudaStream_t side = ctx->rows_stream;
    cudaError_t err;
    ctx->sums_on_main = false;
    if (side) {
        // The side stream picks up where `stream` is now: behind the previous step's kernels and
        // whatever produced the gradients.  The block kernel then runs there, beside the stream
        // kernel on `stream`, and the caller's all-reduce can follow it without waiting for the latter.
        if ((err = cudaEventRecord(ctx->rows_fork, ctx->stream)) != cudaSuccess ||
            (err = cudaStreamWaitEvent(side, ctx->rows_fork, 0)) != cudaSuccess)
            return cuda_fail(err, "forking the side stream");
    }
    // Without the detach output x is never dereferenced by the local half (block_sum is set); the
    // errors pointer stands in for the alignment class.
    float *x_arg = z ? const_cast<float *>(params) : errors;
    rc = enqueue_columns(ctx, 0, ctx->d, ctx->d, x_arg, grads, errors, mom, step, seed, ctx->stream, z, block_sum_out, side);
    if (rc != DEF_OK) return rc;
    if (side && ctx->sums_on_main) {   // a kernel on `stream` wrote block sums: the side stream must see them
        if ((err = cudaEventRecord(ctx->rows_fork, ctx->stream)) != cudaSuccess ||
            (err = cudaStreamWaitEvent(side, ctx->rows_fork, 0)) != cudaSuccess)
            return cuda_fail(err, "ordering the side stream behind the step kernel");
    }
    return DEF_OK;
}

int rows_apply(def_ctx *ctx, float *params, const float *block_sum, int32_t W_total, float *z,
               uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (!params || !block_sum) return fail(DEF_ERR_NULL, "params and block_sum must not be NULL");
    if (((uintptr_t)params | (uintptr_t)block_sum | (uintptr_t)z) & 3u) return fail(DEF_ERR_ALIGN, "a pointer is not 4-byte aligned");
    if (W_total < ctx->W) return fail(DEF_ERR_ARG, "W_total=%d is smaller than this context's W=%d", W_total, ctx->W);
    const size_t x_b = (size_t)ctx->d * sizeof(float), bs_b = (size_t)ctx->k * sizeof(float);
    if (overlaps(params, x_b, block_sum, bs_b)) return fail(DEF_ERR_ALIAS, "params and block_sum overlap");
    if (z) {
        const size_t rows_b = span_rows(ctx->W, ctx->d, ctx->d);
        if (overlaps(z, rows_b, params, x_b) || overlaps(z, rows_b, block_sum, bs_b))
            return fail(DEF_ERR_ALIAS, "detached_out overlaps params or block_sum");
    }
    int rc = check_device(ctx);
    if (rc != DEF_OK) return rc;
    defk::StepArgs a = {};
    a.d = ctx->d; a.ld = ctx->d; a.k = ctx->k; a.W = W_total; a.W_float = (float)W_total; a.seed = seed; a.step = step;
    const int64_t blocks = (ctx->k + 255) / 256;
    if (blocks > 0x7fffffffLL) return fail(DEF_ERR_ARG, "k too large");
    cudaStream_t side = ctx->rows_stream;
    cudaStream_t run = side ? side : ctx->stream;
    defk::def_apply_block_kernel<<<(unsigned)blocks, 256, 0, run>>>(params, block_sum, z, ctx->W, a);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return cuda_fail(err, "def_step_rows_apply kernel launch");
    ctx->launches += 1;
    if (side) {   // `stream` goes on only when the side stream's part of the step is done
        if ((err = cudaEventRecord(ctx->rows_join, side)) != cudaSuccess ||
            (err = cudaStreamWaitEvent(ctx->stream, ctx->rows_join, 0)) != cudaSuccess)
            return cuda_fail(err, "joining the side stream");
    }
    return DEF_OK;
}

}  // namespace

extern "C" {

int def_step_rows_local(def_ctx *ctx, const float *grads, float *errors, float *mom,
                        float *block_sum_out, uint64_t step, uint64_t seed) {
    return rows_local(ctx, nullptr, grads, errors, mom, block_sum_out, nullptr, step, seed);
}

int def_step_rows_apply(def_ctx *ctx, float *params, const float *block_sum, int32_t W_total,
                        uint64_t step, uint64_t seed) {
    return rows_apply(ctx, params, block_sum, W_total, nullptr, step, seed);
}

int def_step_rows_local_detach(def_ctx *ctx, const float *params, const float *grads, float *errors,
                               float *mom, float *block_sum_out, float *detached_out, uint64_t step,
                               uint64_t seed) {
    if (!detached_out) return fail(DEF_ERR_NULL, "detached_out must not be NULL");
    if (!params) return fail(DEF_ERR_NULL, "params must not be NULL");
    return rows_local(ctx, params, grads, errors, mom, block_sum_out, detached_out, step, seed);
}

int def_step_rows_apply_detach(def_ctx *ctx, float *params, const float *block_sum, int32_t W_total,
                               float *detached_out, uint64_t step, uint64_t seed) {
    if (!detached_out) return fail(DEF_ERR_NULL, "detached_out must not be NULL");
    return rows_apply(ctx, params, block_sum, W_total, detached_out, step, seed);
}

int def_set_rows_stream(def_ctx *ctx, void *side_stream) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (side_stream && side_stream == (void *)ctx->stream)
        return fail(DEF_ERR_ARG, "the side stream must differ from the context's stream");
    if (side_stream && !ctx->rows_fork) {
        int rc = check_device(ctx);
        if (rc != DEF_OK) return rc;
        cudaError_t err = cudaEventCreateWithFlags(&ctx->rows_fork, cudaEventDisableTiming);
        if (err == cudaSuccess) err = cudaEventCreateWithFlags(&ctx->rows_join, cudaEventDisableTiming);
        if (err != cudaSuccess) return cuda_fail(err, "creating the side stream's events");
    }
    ctx->rows_stream = (cudaStream_t)side_stream;
    return DEF_OK;
}

int def_step_host(def_ctx *ctx, float *params_host, const float *grads_host, float *errors_host,
                  float *mom_host, uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    return def_step_columns_host(ctx, 0, ctx->d, ctx->d, params_host, grads_host, errors_host,
                                 mom_host, step, seed);
}

int def_step_columns_host(def_ctx *ctx, int64_t c0, int64_t cols, int64_t ld, float *params_host,
                          const float *grads_host, float *errors_host, float *mom_host,
                          uint64_t step, uint64_t seed) {
    if (!ctx) return fail(DEF_ERR_NULL, "ctx is NULL");
    if (c0 < 0 || cols < 0 || c0 > ctx->d || cols > ctx->d - c0)
        return fail(DEF_ERR_ARG, "column range [%lld, %lld) is outside [0, %lld)", (long long)c0,
                    (long long)(c0 + cols), (long long)ctx->d);
    if (ld < cols) return fail(DEF_ERR_ARG, "row stride ld=%lld is smaller than n=%lld", (long long)ld, (long long)cols);
    if (cols == 0) return DEF_OK;
    int rc = validate_tensors(ctx, cols, ld, params_host, grads_host, errors_host, mom_host);
    if (rc != DEF_OK) return rc;
    if ((rc = check_device(ctx)) != DEF_OK) return rc;
    if ((rc = prepare_host_path(ctx)) != DEF_OK) return rc;

    const int64_t d = cols, chunk = ctx->host_chunk;   // local coordinates 0..cols-1
    const int W = ctx->W;
    const size_t host_pitch = (size_t)ld * sizeof(float);
    const size_t dev_pitch = (size_t)chunk * sizeof(float);
    cudaError_t err = cudaSuccess;
    int64_t piece = 0;
    for (int64_t j0 = 0; j0 < d; j0 += chunk, ++piece) {
        HostSlot &s = ctx->slots[piece % kHostSlots];
        const int64_t n = (d - j0 < chunk) ? d - j0 : chunk;
        const size_t width = (size_t)n * sizeof(float);
        // the slot's previous piece must have left the device before it is overwritten
        if (s.used && (err = cudaStreamWaitEvent(ctx->s_h2d, s.drained, 0)) != cudaSuccess) break;
        if ((err = cudaMemcpyAsync(s.x, params_host + j0, width, cudaMemcpyHostToDevice, ctx->s_h2d)) != cudaSuccess) break;
        if ((err = cudaMemcpy2DAsync(s.g, dev_pitch, grads_host + j0, host_pitch, width, W, cudaMemcpyHostToDevice, ctx->s_h2d)) != cudaSuccess) break;
        if ((err = cudaMemcpy2DAsync(s.e, dev_pitch, errors_host + j0, host_pitch, width, W, cudaMemcpyHostToDevice, ctx->s_h2d)) != cudaSuccess) break;
        if (mom_host && (err = cudaMemcpy2DAsync(s.m, dev_pitch, mom_host + j0, host_pitch, width, W, cudaMemcpyHostToDevice, ctx->s_h2d)) != cudaSuccess) break;
        if ((err = cudaEventRecord(s.loaded, ctx->s_h2d)) != cudaSuccess) break;

        if ((err = cudaStreamWaitEvent(ctx->s_run, s.loaded, 0)) != cudaSuccess) break;
        rc = enqueue_columns(ctx, c0 + j0, n, chunk, s.x, s.g, s.e, mom_host ? s.m : nullptr, step, seed, ctx->s_run);
        if (rc != DEF_OK) break;
        if ((err = cudaEventRecord(s.computed, ctx->s_run)) != cudaSuccess) break;

        if ((err = cudaStreamWaitEvent(ctx->s_d2h, s.computed, 0)) != cudaSuccess) break;
        if ((err = cudaMemcpyAsync(params_host + j0, s.x, width, cudaMemcpyDeviceToHost, ctx->s_d2h)) != cudaSuccess) break;
        if ((err = cudaMemcpy2DAsync(errors_host + j0, host_pitch, s.e, dev_pitch, width, W, cudaMemcpyDeviceToHost, ctx->s_d2h)) != cudaSuccess) break;
        if (mom_host && (err = cudaMemcpy2DAsync(mom_host + j0, host_pitch, s.m, dev_pitch, width, W, cudaMemcpyDeviceToHost, ctx->s_d2h)) != cudaSuccess) break;
        if ((err = cudaEventRecord(s.drained, ctx->s_d2h)) != cudaSuccess) break;
        s.used = true;
    }
    // drain everything that was enqueued, also after a failure
    cudaError_t e1 = cudaStreamSynchronize(ctx->s_h2d);
    cudaError_t e2 = cudaStreamSynchronize(ctx->s_run);
    cudaError_t e3 = cudaStreamSynchronize(ctx->s_d2h);
    if (rc != DEF_OK) return rc;
    if (err != cudaSuccess) return cuda_fail(err, "def_step_host");
    if (e1 != cudaSuccess) return cuda_fail(e1, "def_step_host (host->device stream)");
    if (e2 != cudaSuccess) return cuda_fail(e2, "def_step_host (compute stream)");
    if (e3 != cudaSuccess) return cuda_fail(e3, "def_step_host (device->host stream)");
    return DEF_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// def_stats_static: the distances of def_stats for callers that must not allocate.
//
// The per-CTA partial sums go to this file-scope device array instead of a buffer obtained
// with cudaMalloc.  Every GPU that loads the library carries its 32 KB until the process
// exits.  The name below is only a host-side stand-in in host code: the address a kernel can
// use comes from cudaGetSymbolAddress, asked for once per device with that device current.
// ---------------------------------------------------------------------------
static __device__ __align__(256) double g_stats_static_scratch[2 * DEF_STATS_STATIC_SLOTS];

namespace {

constexpr int kMaxKnownDevices = 64;
std::mutex g_static_mutex;
double *g_static_scratch_ptr[kMaxKnownDevices] = {};
int g_static_sm_count[kMaxKnownDevices] = {};

// Device address of the static scratch on the current device (looked up on first use).
int static_scratch_address(double **ptr_out, int *sm_count_out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return fail(DEF_ERR_DEVICE, "no usable CUDA device: %s", cudaGetErrorString(err));
    }
    if (dev < 0 || dev >= kMaxKnownDevices) return fail(DEF_ERR_DEVICE, "device ordinal %d is not supported", dev);
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_ptr[dev]) {
        cudaDeviceProp prop;
        err = cudaGetDeviceProperties(&prop, dev);
        if (err != cudaSuccess) { cudaGetLastError(); return fail(DEF_ERR_DEVICE, "cannot query device %d: %s", dev, cudaGetErrorString(err)); }
        if (prop.major != 10)
            return fail(DEF_ERR_DEVICE, "device %d is compute capability %d.%d; this library is built for 10.x (sm_100a)", dev, prop.major, prop.minor);
        void *p = nullptr;
        err = cudaGetSymbolAddress(&p, g_stats_static_scratch);
        if (err != cudaSuccess || !p) { cudaGetLastError(); return cuda_fail(err, "cudaGetSymbolAddress(static scratch)"); }
        g_static_scratch_ptr[dev] = static_cast<double *>(p);
        g_static_sm_count[dev] = prop.multiProcessorCount;
    }
    *ptr_out = g_static_scratch_ptr[dev];
    *sm_count_out = g_static_sm_count[dev];
    return DEF_OK;
}

}  // namespace

extern "C" int def_stats_static(const float *errors, int64_t n, int64_t ld, int32_t W, float lambda,
                                double *stats_out, void *cuda_stream) {
    if (!errors || !stats_out) return fail(DEF_ERR_NULL, "errors and stats_out must not be NULL");
    if (((uintptr_t)errors & 3u) || ((uintptr_t)stats_out & 7u))
        return fail(DEF_ERR_ALIGN, "errors must be 4-byte and stats_out 8-byte aligned");
    if (W < 1 || W > DEF_MAX_WORKERS) return fail(DEF_ERR_ARG, "W must be in 1..%d (got %d)", DEF_MAX_WORKERS, W);
    if (n < 0 || n > DEF_STATS_STATIC_MAX_N)
        return fail(DEF_ERR_ARG, "def_stats_static handles at most %lld coordinates per call (got n=%lld); "
                                 "split the columns and add the results, or use def_stats",
                    (long long)DEF_STATS_STATIC_MAX_N, (long long)n);
    if (ld < n) return fail(DEF_ERR_ARG, "row stride ld=%lld is smaller than n=%lld", (long long)ld, (long long)n);
    if (!(lambda >= 0.f && lambda <= 1.f)) return fail(DEF_ERR_ARG, "lambda must be in [0, 1]");
    double *scratch = nullptr;
    int sm_count = 0;
    int rc = static_scratch_address(&scratch, &sm_count);
    if (rc != DEF_OK) return rc;
    const int V = width_of(ld, errors, nullptr, nullptr);
    const int64_t groups = (n + V - 1) / V;
    const int64_t ctas = stats_grid(groups, sm_count);
    if ((size_t)ctas * 2 * sizeof(double) > sizeof(double) * 2 * DEF_STATS_STATIC_SLOTS)
        return fail(DEF_ERR_ARG, "the static scratch cannot hold %lld partial sums", (long long)ctas);
    // Every slot the second kernel reads ([0, ctas)) is written by the first in this same call,
    // so nothing left over from an earlier call is ever read and nothing needs clearing.
    return launch_stats(errors, n, ld, W, lambda, V, ctas, scratch, stats_out, (cudaStream_t)cuda_stream);
}
