// Element-wise Beaver product (Section 2.1 "Multiplication", Eq. 1, one element at a time), e.g. the product
// ReLU(gate) * up of a gated FFN:
//   open   : [d]_i = [x]_i - [a]_i,  [e]_i = [y]_i - [b]_i                       (before the exchange)
//   combine: d = [d]_0 + [d]_1, e = [e]_0 + [e]_1,
//            [z]_i = [c]_i + d*[b]_i + e*[a]_i + i*d*e                           (after it)
// HBM-bound; 16-byte accesses when the word count is even and the pointers allow it; blockIdx.y is the party.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace comet {

typedef unsigned long long u64;

struct MulArgs {
    const u64* x[2]; const u64* y[2];
    const u64* a[2]; const u64* b[2]; const u64* c[2];
    u64* d[2]; u64* e[2];        // the messages
    u64* z[2];
    long long pieces;            // 16-byte pairs, or single words
};

__device__ __forceinline__ ulonglong2 mul_sub(ulonglong2 p, ulonglong2 q) { return make_ulonglong2(p.x - q.x, p.y - q.y); }
__device__ __forceinline__ u64 mul_sub(u64 p, u64 q) { return p - q; }
__device__ __forceinline__ u64 mul_eq1(u64 c, u64 d, u64 e, u64 a, u64 b, int party) {
    return c + d * b + e * a + (party ? d * e : 0ull);
}
__device__ __forceinline__ u64 mul_combine(u64 c, u64 d0, u64 d1, u64 e0, u64 e1, u64 a, u64 b, int party) {
    return mul_eq1(c, d0 + d1, e0 + e1, a, b, party);
}
__device__ __forceinline__ ulonglong2 mul_combine(ulonglong2 c, ulonglong2 d0, ulonglong2 d1, ulonglong2 e0,
                                                  ulonglong2 e1, ulonglong2 a, ulonglong2 b, int party) {
    return make_ulonglong2(mul_eq1(c.x, d0.x + d1.x, e0.x + e1.x, a.x, b.x, party),
                           mul_eq1(c.y, d0.y + d1.y, e0.y + e1.y, a.y, b.y, party));
}

template <typename PIECE>
__global__ void __launch_bounds__(256)
beaver_mul_open_kernel(MulArgs g) {
    const int party = blockIdx.y;
    const PIECE* __restrict__ x = reinterpret_cast<const PIECE*>(party ? g.x[1] : g.x[0]);
    const PIECE* __restrict__ y = reinterpret_cast<const PIECE*>(party ? g.y[1] : g.y[0]);
    const PIECE* __restrict__ a = reinterpret_cast<const PIECE*>(party ? g.a[1] : g.a[0]);
    const PIECE* __restrict__ b = reinterpret_cast<const PIECE*>(party ? g.b[1] : g.b[0]);
    PIECE* __restrict__ d = reinterpret_cast<PIECE*>(party ? g.d[1] : g.d[0]);
    PIECE* __restrict__ e = reinterpret_cast<PIECE*>(party ? g.e[1] : g.e[0]);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < g.pieces; t += stride) {
        d[t] = mul_sub(__ldg(x + t), __ldg(a + t));
        e[t] = mul_sub(__ldg(y + t), __ldg(b + t));
    }
}

template <typename PIECE>
__global__ void __launch_bounds__(256)
beaver_mul_combine_kernel(MulArgs g) {
    const int party = blockIdx.y;
    const PIECE* __restrict__ d0 = reinterpret_cast<const PIECE*>(g.d[0]);
    const PIECE* __restrict__ d1 = reinterpret_cast<const PIECE*>(g.d[1]);
    const PIECE* __restrict__ e0 = reinterpret_cast<const PIECE*>(g.e[0]);
    const PIECE* __restrict__ e1 = reinterpret_cast<const PIECE*>(g.e[1]);
    const PIECE* __restrict__ a = reinterpret_cast<const PIECE*>(party ? g.a[1] : g.a[0]);
    const PIECE* __restrict__ b = reinterpret_cast<const PIECE*>(party ? g.b[1] : g.b[0]);
    const PIECE* __restrict__ c = reinterpret_cast<const PIECE*>(party ? g.c[1] : g.c[0]);
    PIECE* __restrict__ z = reinterpret_cast<PIECE*>(party ? g.z[1] : g.z[0]);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < g.pieces; t += stride)
        z[t] = mul_combine(__ldg(c + t), d0[t], d1[t], e0[t], e1[t], __ldg(a + t), __ldg(b + t), party);
}

// Truncation by f bits with a dealer's pair (r, r' = floor(r / 2^f), r read as signed).  Not a protocol of the
// paper; it is Section 2.1's "Reconstruction" of m = z - r followed by its "Addition" of the public value
// floor(m / 2^f):
//   open   : [m]_i = [z]_i - [r]_i                                      (before the exchange)
//   combine: m = [m]_0 + [m]_1,  [z]_i <- [r']_i + i * (m >> f, arithmetic)  (after it)
struct TruncPairArgs {
    u64* z[2];                   // in: shares at scale 2f; out: shares at scale f
    const u64* r[2]; const u64* rp[2];
    u64* m[2];                   // the messages
    long long pieces;
    int f;
};

__device__ __forceinline__ u64 trunc_floor(u64 m, int f) { return (u64)((long long)m >> f); }
__device__ __forceinline__ u64 trunc_pair_out(u64 rp, u64 m0, u64 m1, int f, int party) {
    return party ? rp + trunc_floor(m0 + m1, f) : rp;
}
__device__ __forceinline__ ulonglong2 trunc_pair_out(ulonglong2 rp, ulonglong2 m0, ulonglong2 m1, int f, int party) {
    return make_ulonglong2(trunc_pair_out(rp.x, m0.x, m1.x, f, party), trunc_pair_out(rp.y, m0.y, m1.y, f, party));
}

template <typename PIECE>
__global__ void __launch_bounds__(256)
trunc_pair_open_kernel(TruncPairArgs g) {
    const int party = blockIdx.y;
    const PIECE* __restrict__ z = reinterpret_cast<const PIECE*>(party ? g.z[1] : g.z[0]);
    const PIECE* __restrict__ r = reinterpret_cast<const PIECE*>(party ? g.r[1] : g.r[0]);
    PIECE* __restrict__ m = reinterpret_cast<PIECE*>(party ? g.m[1] : g.m[0]);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < g.pieces; t += stride)
        m[t] = mul_sub(z[t], __ldg(r + t));
}

template <typename PIECE>
__global__ void __launch_bounds__(256)
trunc_pair_combine_kernel(TruncPairArgs g) {
    const int party = blockIdx.y;
    const PIECE* __restrict__ m0 = reinterpret_cast<const PIECE*>(g.m[0]);
    const PIECE* __restrict__ m1 = reinterpret_cast<const PIECE*>(g.m[1]);
    const PIECE* __restrict__ rp = reinterpret_cast<const PIECE*>(party ? g.rp[1] : g.rp[0]);
    PIECE* __restrict__ z = reinterpret_cast<PIECE*>(party ? g.z[1] : g.z[0]);
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < g.pieces; t += stride)
        z[t] = trunc_pair_out(__ldg(rp + t), m0[t], m1[t], g.f, party);
}

// Section 2.1 "Addition": a shared bias [cols] added to every row of a shared matrix, in place; purely local.
struct BiasArgs {
    u64* z[2];
    const u64* bias[2];
    long long rows;
    int cols;
};

__global__ void __launch_bounds__(256)
add_bias_kernel(BiasArgs g) {
    const int party = blockIdx.y;
    u64* __restrict__ z = party ? g.z[1] : g.z[0];
    const u64* __restrict__ b = party ? g.bias[1] : g.bias[0];
    const long long total = g.rows * g.cols, stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride)
        z[t] += __ldg(b + (int)(t % g.cols));
}

}  // namespace comet
