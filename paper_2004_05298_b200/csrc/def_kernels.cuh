// Device code of the DEF / DEF-A / EF step for sm_100a.
//
// The step (Algorithm 1 lines 7-10 with the momentum form of Eq. 10) is separate
// per model coordinate: a coordinate j needs g, m, e of its W workers and, if j is
// one of the k block coordinates, x[j].  The kernel therefore gives each thread a
// short vector of consecutive coordinates and walks the W rows in order, so that
//   * g, m, e are read once and m', e' written once (20 bytes per gradient element,
//     the least the method can move), with 128-bit coalesced accesses;
//   * p never goes to memory;
//   * the sum over workers that stands in for the ring-allreduce of line 9 is a
//     register accumulation in the fixed order w = 0..W-1: deterministic, and with
//     no shuffle, shared memory or atomics;
//   * x is touched on the block only (line 10).
// The block is a predicate on j, never a slice: nothing is gathered or scattered.
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

// g, m and e are read once per step and the new m and e are not read again before
// the next step, by which time W*d*20 bytes have passed through the L2: mark the
// traffic as streaming so that it does not push x (which is reused) out.
template <int V> __device__ __forceinline__ Vec<V> load_stream(const float *p);
template <> __device__ __forceinline__ Vec<1> load_stream<1>(const float *p) {
    Vec<1> r; r.v[0] = __ldcs(p); return r;
}
template <> __device__ __forceinline__ Vec<2> load_stream<2>(const float *p) {
    const float2 t = __ldcs(reinterpret_cast<const float2 *>(p));
    Vec<2> r; r.v[0] = t.x; r.v[1] = t.y; return r;
}
template <> __device__ __forceinline__ Vec<4> load_stream<4>(const float *p) {
    const float4 t = __ldcs(reinterpret_cast<const float4 *>(p));
    Vec<4> r; r.v[0] = t.x; r.v[1] = t.y; r.v[2] = t.z; r.v[3] = t.w; return r;
}
template <int V> __device__ __forceinline__ void store_stream(float *p, const Vec<V> &a);
template <> __device__ __forceinline__ void store_stream<1>(float *p, const Vec<1> &a) {
    __stcs(p, a.v[0]);
}
template <> __device__ __forceinline__ void store_stream<2>(float *p, const Vec<2> &a) {
    __stcs(reinterpret_cast<float2 *>(p), make_float2(a.v[0], a.v[1]));
}
template <> __device__ __forceinline__ void store_stream<4>(float *p, const Vec<4> &a) {
    __stcs(reinterpret_cast<float4 *>(p), make_float4(a.v[0], a.v[1], a.v[2], a.v[3]));
}

struct StepArgs {
    float *x;            // [n]      local coordinates of the model
    const float *g;      // [W, ld]
    float *e;            // [W, ld]
    float *m;            // [W, ld] or nullptr
    int64_t n;           // local coordinates
    int64_t ld;          // row stride in floats
    int64_t d;           // model size the block is drawn over
    int64_t j0;          // model coordinate of local coordinate 0
    int64_t k;           // block length
    int32_t W;           // workers
    float eta;           // learning rate
    float mu;            // momentum constant
    float W_float;       // (float)W, the divisor of line 9
    uint64_t seed, step; // the block start is drawn from these
};

// One worker's row for V coordinates: Eq. 10 / line 7, then line 8.
// `sent` accumulates C(p) over the workers in call order.
template <int V, bool MOM, bool FIRST>
__device__ __forceinline__ void worker_row(const Vec<V> &g, const Vec<V> &m, const Vec<V> &e,
                                           const bool (&in)[V], float eta, float mu,
                                           Vec<V> &m_new, Vec<V> &e_new, float (&sent)[V]) {
#pragma unroll
    for (int i = 0; i < V; ++i) {
        float p;
        if (MOM) {
            m_new.v[i] = __fmaf_rn(mu, m.v[i], g.v[i]);      // m' = mu m + g
            p = __fmaf_rn(eta, m_new.v[i], e.v[i]);          // p = eta m' + e
        } else {
            p = __fmaf_rn(eta, g.v[i], e.v[i]);              // p = eta g + e
        }
        const float c = in[i] ? p : 0.0f;                    // C(p)
        e_new.v[i] = __fsub_rn(p, c);                        // e' = p - C(p)
        sent[i] = FIRST ? c : __fadd_rn(sent[i], c);         // running sum of line 9
    }
}

// The step over local coordinates [0, n), V per thread, U rows in flight per thread.
//   grid-stride over groups of V coordinates; rows must be aligned for V-wide access:
//   x, g, e, m aligned to 4V bytes and ld % V == 0.  The n % V tail coordinates are
//   handled by the V = 1 instantiation launched on the tail (see the host code).
template <int V, bool MOM, int U>
__global__ void __launch_bounds__(256)
def_step_kernel(const StepArgs a) {
    const int64_t s = block_start(a.seed, a.step, a.d);
    const int64_t groups = a.n / V;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const size_t ld = (size_t)a.ld;
    for (int64_t grp = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < groups; grp += stride) {
        const int64_t col = grp * V;
        // offset of each coordinate from the block start, mod d; in the block iff < k
        int64_t off = a.j0 + col - s;
        if (off < 0) off += a.d;
        bool in[V];
        bool any = false;
#pragma unroll
        for (int i = 0; i < V; ++i) {
            int64_t o = off + i;
            if (o >= a.d) o -= a.d;
            in[i] = o < a.k;
            any |= in[i];
        }

        float sent[V];
        const float *gp = a.g + col;
        float *ep = a.e + col;
        float *mp = MOM ? a.m + col : nullptr;
        int w = 0;
        // worker 0 starts the sum
        {
            const Vec<V> g = load_stream<V>(gp);
            const Vec<V> e = load_stream<V>(ep);
            Vec<V> m, m_new, e_new;
            if (MOM) m = load_stream<V>(mp);
            worker_row<V, MOM, true>(g, m, e, in, a.eta, a.mu, m_new, e_new, sent);
            if (MOM) store_stream<V>(mp, m_new);
            store_stream<V>(ep, e_new);
            w = 1;
        }
        // U workers at a time: issue all loads, then compute and store in order
        for (; w + U <= a.W; w += U) {
            Vec<V> g[U], e[U], m[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t row = (size_t)(w + u) * ld;
                g[u] = load_stream<V>(gp + row);
                e[u] = load_stream<V>(ep + row);
                if (MOM) m[u] = load_stream<V>(mp + row);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const size_t row = (size_t)(w + u) * ld;
                Vec<V> m_new, e_new;
                worker_row<V, MOM, false>(g[u], m[u], e[u], in, a.eta, a.mu, m_new, e_new, sent);
                if (MOM) store_stream<V>(mp + row, m_new);
                store_stream<V>(ep + row, e_new);
            }
        }
        for (; w < a.W; ++w) {
            const size_t row = (size_t)w * ld;
            const Vec<V> g = load_stream<V>(gp + row);
            const Vec<V> e = load_stream<V>(ep + row);
            Vec<V> m, m_new, e_new;
            if (MOM) m = load_stream<V>(mp + row);
            worker_row<V, MOM, false>(g, m, e, in, a.eta, a.mu, m_new, e_new, sent);
            if (MOM) store_stream<V>(mp + row, m_new);
            store_stream<V>(ep + row, e_new);
        }
        // lines 9-10 on the block coordinates: x -= (sum over workers) / W
        if (any) {
#pragma unroll
            for (int i = 0; i < V; ++i) {
                if (in[i]) {
                    const float C_pt = __fdiv_rn(sent[i], a.W_float);
                    a.x[col + i] = __fsub_rn(a.x[col + i], C_pt);
                }
            }
        }
    }
}

}  // namespace defk
