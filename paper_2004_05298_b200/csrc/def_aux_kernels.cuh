// Device code around the step: the detach point (Algorithm 1's detach step), the returned model
// (Algorithm 1's Output) and the squared distances of Eq. 9.  All three are separate
// per coordinate except for the final sum of the distances.
#pragma once

#include "def_kernels.cuh"

namespace defk {

// ---------------------------------------------------------------------------
// Detach point: z[w, j] = x[j] - lambda * e[w, j], one fused multiply-add per element.
// One thread per V coordinates keeps its x in registers and walks the W rows, U in flight,
// so x is read once.
// ---------------------------------------------------------------------------
template <int V, int U>
__global__ void __launch_bounds__(256)
def_detach_kernel(const float *__restrict__ x, const float *__restrict__ e, float *__restrict__ z,
                  int64_t n, int64_t ld, int W, float lambda) {
    const int64_t col = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= n) return;
    if (col + V <= n) {
        const Vec<V> xv = load_vec<V, kCacheDefault>(x + col);
        for (int w = 0; w < W; w += U) {
            Vec<V> ev[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (w + u < W) ev[u] = load_vec<V, kCacheDefault>(e + (size_t)(w + u) * (size_t)ld + (size_t)col);
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (w + u < W) {
                    Vec<V> zv;
#pragma unroll
                    for (int i = 0; i < V; ++i) zv.v[i] = __fmaf_rn(-lambda, ev[u].v[i], xv.v[i]);
                    store_vec<V, kCacheDefault>(z + (size_t)(w + u) * (size_t)ld + (size_t)col, zv);
                }
        }
    } else {                                   // the n % V coordinates at the end of a row
        for (int64_t c = col; c < n; ++c)
            for (int w = 0; w < W; ++w)
                z[(size_t)w * (size_t)ld + (size_t)c] = __fmaf_rn(-lambda, e[(size_t)w * (size_t)ld + (size_t)c], x[c]);
    }
}

// ---------------------------------------------------------------------------
// DEF's returned model: y[j] = x[j] - (sum_w e[w, j]) / W, workers added in order
// w = 0..W-1 in fp32, IEEE division.  One thread per V coordinates, U rows in flight.
// ---------------------------------------------------------------------------
template <int V, int U>
__global__ void __launch_bounds__(256)
def_output_kernel(const float *__restrict__ x, const float *__restrict__ e, float *__restrict__ y,
                  int64_t n, int64_t ld, int W, float W_float) {
    const int64_t col = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * V;
    if (col >= n) return;
    if (col + V <= n) {
        float sum[V];
        for (int w = 0; w < W; w += U) {
            Vec<V> ev[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (w + u < W) ev[u] = load_vec<V, kCacheStreaming>(e + (size_t)(w + u) * (size_t)ld + (size_t)col);
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (w + u < W) {
#pragma unroll
                    for (int i = 0; i < V; ++i) sum[i] = (w + u == 0) ? ev[u].v[i] : __fadd_rn(sum[i], ev[u].v[i]);
                }
        }
        const Vec<V> xv = load_vec<V, kCacheStreaming>(x + col);
        Vec<V> yv;
#pragma unroll
        for (int i = 0; i < V; ++i) yv.v[i] = __fsub_rn(xv.v[i], __fdiv_rn(sum[i], W_float));
        store_vec<V, kCacheStreaming>(y + col, yv);
    } else {
        for (int64_t c = col; c < n; ++c) {
            float sum = e[c];
            for (int w = 1; w < W; ++w) sum = __fadd_rn(sum, e[(size_t)w * (size_t)ld + (size_t)c]);
            y[c] = __fsub_rn(x[c], __fdiv_rn(sum, W_float));
        }
    }
}

// ---------------------------------------------------------------------------
// Distances of Eq. 9 over the current errors, accumulated in fp64:
//   A = (1/W) sum_w |e_w|^2,  B = |e_bar|^2 with e_bar = (1/W) sum_w e_w,
//   C = (1/W) sum_w |e_bar - lambda e_w|^2 = (1 - 2 lambda) B + lambda^2 A   (expand the square).
// Pass 1: a fixed grid of at most kStatsMaxCtas CTAs; every thread walks the W rows of its
// coordinate groups (tile-stride loop), keeps sum e^2 and sum e_bar^2, and each CTA writes
// its two partial sums to scratch[2 * blockIdx.x ..].  Pass 2: one CTA adds the partials in
// a fixed order and writes {A, B, C}.  Same grid, same order => same bits every run.
// ---------------------------------------------------------------------------
constexpr int kStatsThreads = 256;
constexpr int kStatsMaxCtas = 2048;

__device__ __forceinline__ double cta_sum(double v, double *smem) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0)
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) total += smem[i];
    __syncthreads();
    return total;                               // valid on thread 0
}

template <int V, int U>
__global__ void __launch_bounds__(kStatsThreads)
def_stats_partial_kernel(const float *__restrict__ e, int64_t n, int64_t ld, int W,
                         double *__restrict__ scratch) {
    __shared__ double smem[kStatsThreads / 32];
    // the one-CTA kernel that adds the partial sums may be set up while this grid runs (it waits
    // for this grid before it reads anything); a no-op when it was launched the ordinary way
    release_dependent_grids();
    double sq = 0.0, mean_sq = 0.0;
    const double inv_W = 1.0 / (double)W;
    const int64_t groups = (n + V - 1) / V;
    for (int64_t grp = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < groups;
         grp += (int64_t)gridDim.x * blockDim.x) {
        const int64_t col = grp * V;
        double s1[V];
#pragma unroll
        for (int i = 0; i < V; ++i) s1[i] = 0.0;
        if (col + V <= n) {
            for (int w = 0; w < W; w += U) {
                Vec<V> ev[U];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (w + u < W) ev[u] = load_vec<V, kCacheStreaming>(e + (size_t)(w + u) * (size_t)ld + (size_t)col);
#pragma unroll
                for (int u = 0; u < U; ++u)
                    if (w + u < W) {
#pragma unroll
                        for (int i = 0; i < V; ++i) {
                            const double v = (double)ev[u].v[i];
                            s1[i] += v;
                            sq = fma(v, v, sq);
                        }
                    }
            }
        } else {                                // the n % V coordinates at the end
#pragma unroll
            for (int i = 0; i < V; ++i) {       // (i is a compile-time index: s1 stays in registers)
                if (col + i >= n) continue;
                for (int w = 0; w < W; ++w) {
                    const double v = (double)e[(size_t)w * (size_t)ld + (size_t)(col + i)];
                    s1[i] += v;
                    sq = fma(v, v, sq);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const double mean = s1[i] * inv_W;
            mean_sq = fma(mean, mean, mean_sq);
        }
    }
    const double sq_cta = cta_sum(sq, smem);
    const double mean_cta = cta_sum(mean_sq, smem);
    if (threadIdx.x == 0) {
        scratch[2 * blockIdx.x] = sq_cta;
        scratch[2 * blockIdx.x + 1] = mean_cta;
    }
}

__global__ void __launch_bounds__(kStatsThreads)
def_stats_final_kernel(const double *scratch, int ctas, int W, float lambda, double *out) {
    __shared__ double smem[kStatsThreads / 32];
    grid_dependency_wait();                     // the partial sums are complete and visible from here on
    double sq = 0.0, mean_sq = 0.0;
    for (int i = threadIdx.x; i < ctas; i += blockDim.x) {
        sq += __ldcg(scratch + 2 * i);          // from the L2, where the other grid's stores are
        mean_sq += __ldcg(scratch + 2 * i + 1);
    }
    const double sq_all = cta_sum(sq, smem);
    const double mean_all = cta_sum(mean_sq, smem);
    if (threadIdx.x == 0) {
        const double A = sq_all / (double)W, B = mean_all, l = (double)lambda;
        out[0] = A;
        out[1] = B;
        out[2] = (1.0 - 2.0 * l) * B + l * l * A;
    }
}

}  // namespace defk
