// K4, CUDA-core variant: the gathered ring matmul fused with the Beaver combine,
//   Z_i = C_i + E*B_i + A_i*F + i*E*F   (Eq. 1 in matrix form, party i),
// evaluated as two products per party, E*(B_i + i*F) + A_i*F, in 64-bit integer
// multiply-adds on the ALUs.  The exchange sums E = E_0 + E_1, F = F_0 + F_1 are
// formed while the tiles are staged into shared memory, so no operand is read
// from HBM more than the algorithm requires.
//
// Operand layout: left operands [M, K] row-major; right operands [N, K]
// row-major (output-feature-major), so both are contiguous along K.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace comet {

typedef unsigned long long u64;

struct CombineArgs {
    const u64* E[2];   // messages of party 0 and 1, [M, K]
    const u64* F[2];   // messages of party 0 and 1, [N, K]
    const u64* A[2];   // triple shares, [M, K]
    const u64* B[2];   // triple shares, [N, K]
    const u64* C[2];   // triple shares, [M, N]
    u64* Z[2];         // result shares, [M, N]
    int M, N, K;       // K multiple of 8, N multiple of 4
    // Protocol 3 with per-column row sets: per-token mask over the active blocks of the contraction index,
    // [M, tmask_ld] bytes, or null; where it is zero A_i is no part of the triple and counts as zero.
    const uint8_t* tmask;
    int tmask_ld, bs;
};

namespace simt {
constexpr int BM = 128, BN = 64, BK = 8, TM = 8, TN = 4, THREADS = 256, PAD = 2;
}

__device__ __forceinline__ ulonglong2 ldg2(const u64* p) {
    return __ldg(reinterpret_cast<const ulonglong2*>(p));
}

__global__ void __launch_bounds__(simt::THREADS, 1)
combine_simt_kernel(CombineArgs a) {
    using namespace simt;
    __shared__ __align__(16) u64 sE[BK][BM + PAD];
    __shared__ __align__(16) u64 sA[BK][BM + PAD];
    __shared__ __align__(16) u64 sU[BK][BN + PAD];
    __shared__ __align__(16) u64 sF[BK][BN + PAD];

    const int party = blockIdx.z;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;

    // staging roles: left tile 128 rows x 8 k -> thread = (row, 4-k half);
    // right tile 64 rows x 8 k -> thread = (row, 2-k quarter)
    const int lrow = tid >> 1, lk = (tid & 1) * 4;
    const int rrow = tid >> 2, rk = (tid & 3) * 2;
    const bool lok = (m0 + lrow) < a.M, rok = (n0 + rrow) < a.N;
    const size_t loff = (size_t)(m0 + lrow) * a.K + lk;
    const size_t roff = (size_t)(n0 + rrow) * a.K + rk;
    const u64* __restrict__ E0 = a.E[0];
    const u64* __restrict__ E1 = a.E[1];
    const u64* __restrict__ Ai = (party ? a.A[1] : a.A[0]);
    const u64* __restrict__ F0 = a.F[0];
    const u64* __restrict__ F1 = a.F[1];
    const u64* __restrict__ Bi = (party ? a.B[1] : a.B[0]);

    const ulonglong2 zero2 = make_ulonglong2(0ull, 0ull);
    ulonglong2 ge0[2], ge1[2], ga[2], gf0, gf1, gb;

    auto fetch = [&](int k0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            ge0[h] = lok ? ldg2(E0 + loff + k0 + 2 * h) : zero2;
            ge1[h] = lok ? ldg2(E1 + loff + k0 + 2 * h) : zero2;
            ga[h] = (lok && (!a.tmask || a.tmask[(size_t)(m0 + lrow) * a.tmask_ld + (k0 + lk + 2 * h) / a.bs] != 0))
                        ? ldg2(Ai + loff + k0 + 2 * h) : zero2;
        }
        gf0 = rok ? ldg2(F0 + roff + k0) : zero2;
        gf1 = rok ? ldg2(F1 + roff + k0) : zero2;
        gb = rok ? ldg2(Bi + roff + k0) : zero2;
    };
    auto stage = [&]() {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            sE[lk + 2 * h][lrow] = ge0[h].x + ge1[h].x;          // the exchange: E = E_0 + E_1
            sE[lk + 2 * h + 1][lrow] = ge0[h].y + ge1[h].y;
            sA[lk + 2 * h][lrow] = ga[h].x;
            sA[lk + 2 * h + 1][lrow] = ga[h].y;
        }
        const u64 fx = gf0.x + gf1.x, fy = gf0.y + gf1.y;        // F = F_0 + F_1
        sF[rk][rrow] = fx;
        sF[rk + 1][rrow] = fy;
        sU[rk][rrow] = gb.x + (party ? fx : 0ull);               // U_i = B_i + i*F
        sU[rk + 1][rrow] = gb.y + (party ? fy : 0ull);
    };

    u64 acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0ull;

    fetch(0);
    for (int k0 = 0; k0 < a.K; k0 += BK) {
        stage();
        __syncthreads();
        if (k0 + BK < a.K) fetch(k0 + BK);
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            u64 e[TM], v[TM], u[TN], f[TN];
#pragma unroll
            for (int i = 0; i < TM; i += 2) {
                const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(&sE[k][ty * TM + i]);
                e[i] = t.x, e[i + 1] = t.y;
                const ulonglong2 s = *reinterpret_cast<const ulonglong2*>(&sA[k][ty * TM + i]);
                v[i] = s.x, v[i + 1] = s.y;
            }
#pragma unroll
            for (int j = 0; j < TN; j += 2) {
                const ulonglong2 t = *reinterpret_cast<const ulonglong2*>(&sU[k][tx * TN + j]);
                u[j] = t.x, u[j + 1] = t.y;
                const ulonglong2 s = *reinterpret_cast<const ulonglong2*>(&sF[k][tx * TN + j]);
                f[j] = s.x, f[j + 1] = s.y;
            }
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] += e[i] * u[j] + v[i] * f[j];
        }
        __syncthreads();
    }

    const u64* __restrict__ Ci = (party ? a.C[1] : a.C[0]);
    u64* __restrict__ Zi = (party ? a.Z[1] : a.Z[0]);
    const int col = n0 + tx * TN;
    if (col < a.N) {
#pragma unroll
        for (int i = 0; i < TM; ++i) {
            const int row = m0 + ty * TM + i;
            if (row < a.M) {
                const size_t o = (size_t)row * a.N + col;
#pragma unroll
                for (int j = 0; j < TN; j += 2) {
                    const ulonglong2 c = ldg2(Ci + o + j);
                    *reinterpret_cast<ulonglong2*>(Zi + o + j) =
                        make_ulonglong2(c.x + acc[i][j], c.y + acc[i][j + 1]);
                }
            }
        }
    }
}

}  // namespace comet
