// Memory-bound kernels of the path: mask compaction, the two "open" (masking)
// steps before the exchange, and local truncation.  Written for sm_100a with
// 128-bit coalesced accesses; blockIdx.y is the party.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace comet {

typedef unsigned long long u64;

struct PartyPtrs {          // one pointer per party
    const u64* p[2];
};
struct PartyOut {
    u64* p[2];
};

// ---------------------------------------------------------------------------
// K1: block mask -> ascending list of active block ids and their count.
// The index-set steps of Protocol 2 (I_x, I_y) and Protocol 3 (the non-zero columns) for a token-shared block mask.
// One CTA of 1024 threads walks the mask 1024 blocks at a time: a warp ballot
// ranks each active block inside its warp, a shuffle scan over the 32 warp
// totals gives each warp's base, and a running base carries across chunks.
// `count` points at two words {count, error flag}; both are also written to
// `host_report` (mapped host memory, or null when the host needs no report) so
// that the host needs no copy, followed by `ticket` in host_report[2]: the host
// may watch that word instead of waiting for the stream.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void compact_mask_body(const uint8_t* __restrict__ mask, int nb, int32_t* __restrict__ ids,
                                                  int32_t* __restrict__ count, int32_t* __restrict__ host_report,
                                                  int32_t ticket) {
    __shared__ int warp_excl[32];
    __shared__ int chunk_total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int running = 0;                       // same value in every thread
    for (int start = 0; start < nb; start += 1024) {
        const int b = start + threadIdx.x;
        const bool on = (b < nb) && (mask[b] != 0);
        const unsigned bal = __ballot_sync(0xffffffffu, on);
        const int rank = __popc(bal & ((1u << lane) - 1u));
        if (lane == 0) warp_excl[warp] = __popc(bal);
        __syncthreads();
        if (warp == 0) {
            const int v = warp_excl[lane];
            int incl = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += up;
            }
            warp_excl[lane] = incl - v;
            if (lane == 31) chunk_total = incl;
        }
        __syncthreads();
        if (on) ids[running + warp_excl[warp] + rank] = b;
        running += chunk_total;
        __syncthreads();                   // warp_excl / chunk_total are rewritten next round
    }
    if (threadIdx.x == 0) {
        *count = running;
        if (host_report == nullptr) return;    // the host counted the mask itself and does not wait for this report
        // {count, error flag raised by an earlier kernel's bounded wait} for the host, in mapped pinned memory
        host_report[0] = running;
        host_report[1] = count[1];
        __threadfence_system();
        *reinterpret_cast<volatile int32_t*>(host_report + 2) = ticket;
        __threadfence_system();
    }
}

__global__ void __launch_bounds__(1024)
compact_mask_kernel(const uint8_t* __restrict__ mask, int nb, int32_t* __restrict__ ids, int32_t* __restrict__ count,
                    int32_t* __restrict__ host_report, int32_t ticket) {
    pdl_wait();
    pdl_launch_dependents();
    compact_mask_body(mask, nb, ids, count, host_report, ticket);
}

// The same with the mask bytes passed in the kernel's parameter block: a mask the host holds (the public sparsity
// distribution, one byte per block) needs no copy to the device at all while it fits there.
struct MaskBytes {
    static constexpr int CAPACITY = 3584;
    uint8_t bytes[CAPACITY];
};

__global__ void __launch_bounds__(1024)
compact_mask_arg_kernel(const __grid_constant__ MaskBytes mask, int nb, int32_t* __restrict__ ids,
                        int32_t* __restrict__ count, int32_t* __restrict__ host_report, int32_t ticket) {
    pdl_wait();
    pdl_launch_dependents();
    compact_mask_body(mask.bytes, nb, ids, count, host_report, ticket);
}

// ---------------------------------------------------------------------------
// K2: E_i = X_i - A_i  (Section 2.1 "Multiplication": [d]_i = [x]_i - [a]_i).
// `pairs` = number of 16-byte word pairs per party.
// ---------------------------------------------------------------------------
// With `tmask` (per-token mask over the active blocks, [rows, tmask_ld] bytes; Protocol 3 with per-column row
// sets) an entry whose mask byte is zero is no non-zero of X: it is not opened and E_i is zero there.
__global__ void __launch_bounds__(256)
open_activation_kernel(PartyPtrs X, PartyPtrs A, PartyOut E, int64_t pairs, const uint8_t* __restrict__ tmask,
                       int tmask_ld, int K, int bs, const int32_t* __restrict__ row_label = nullptr) {
    const int party = blockIdx.y;
    const ulonglong2* __restrict__ x = reinterpret_cast<const ulonglong2*>((party ? X.p[1] : X.p[0]));
    const ulonglong2* __restrict__ a = reinterpret_cast<const ulonglong2*>((party ? A.p[1] : A.p[0]));
    ulonglong2* __restrict__ e = reinterpret_cast<ulonglong2*>((party ? E.p[1] : E.p[0]));
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < pairs; t += stride) {
        if (tmask) {
            const unsigned word = (unsigned)(2 * t), row = word / (unsigned)K, col = word - row * (unsigned)K;
            if (tmask[(size_t)row * tmask_ld + col / (unsigned)bs] == 0) {
                e[t] = make_ulonglong2(0ull, 0ull);
                continue;
            }
        }
        if (row_label && row_label[(unsigned)(2 * t) / (unsigned)K] < 0) {   // a row outside every component is not opened
            e[t] = make_ulonglong2(0ull, 0ull);
            continue;
        }
        const ulonglong2 xv = __ldg(x + t), av = __ldg(a + t);
        e[t] = make_ulonglong2(xv.x - av.x, xv.y - av.y);
    }
}

// The Merge step of Protocol 2 on the compact result [T, cols]: an entry whose token and block are not in the same
// component is no part of any result block and is zero in both shares.  Compact column c belongs to active block
// (c mod n) / bs.  `pairs` = 16-byte word pairs per party.
__global__ void __launch_bounds__(256)
somm_merge_kernel(PartyOut Z, int64_t pairs, int cols, int n, int bs, const int32_t* __restrict__ row_label,
                  const int32_t* __restrict__ blk_label) {
    pdl_wait();
    pdl_launch_dependents();
    const int party = blockIdx.y;
    ulonglong2* __restrict__ z = reinterpret_cast<ulonglong2*>((party ? Z.p[1] : Z.p[0]));
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < pairs; t += stride) {
        const unsigned word = (unsigned)(2 * t), row = word / (unsigned)cols, col = word - row * (unsigned)cols;
        const int rl = row_label[row];
        if (rl < 0 || rl != blk_label[(col % (unsigned)n) / (unsigned)bs]) z[t] = make_ulonglong2(0ull, 0ull);
    }
}

// ---------------------------------------------------------------------------
// K3 (up): F_i[c, :] = W_i[neuron(c), :] - B_i[c, :].  The paper's IndexCols
// (Protocol 2) followed by [e]_i = [y]_i - [b]_i; with weights stored
// output-feature-major the column gather is a gather of whole rows of d words.
// Compact row c in [0, g*n): group = c / n selects the weight matrix (WG, W1,
// W3 in that order when there are several), j = c mod n, neuron = ids[j / bs] * bs + j mod bs.
// One CTA per compact row (grid-strided); threads sweep the row 16 bytes each.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
open_weight_rows_kernel(PartyPtrs Wg0, PartyPtrs Wg1, PartyPtrs Wg2, PartyPtrs B, PartyOut F, const int32_t* __restrict__ ids,
                        int n, int groups, int bs, int d, const int32_t* __restrict__ blk_label = nullptr) {
    const int party = blockIdx.y;
    const int pairs = d >> 1;
    for (int c = blockIdx.x; c < groups * n; c += gridDim.x) {
        const int grp = c / n, j = c - grp * n;
        const int neuron = ids[j / bs] * bs + (j % bs);
        if (blk_label && blk_label[j / bs] < 0) {        // a column outside every component is not opened
            ulonglong2* f0 = reinterpret_cast<ulonglong2*>((party ? F.p[1] : F.p[0]) + (size_t)c * d);
            for (int t = threadIdx.x; t < pairs; t += blockDim.x) f0[t] = make_ulonglong2(0ull, 0ull);
            continue;
        }
        const u64* W = (grp == 0 ? (party ? Wg0.p[1] : Wg0.p[0])
                                 : grp == 1 ? (party ? Wg1.p[1] : Wg1.p[0]) : (party ? Wg2.p[1] : Wg2.p[0]));
        const ulonglong2* __restrict__ w = reinterpret_cast<const ulonglong2*>(W + (size_t)neuron * d);
        const ulonglong2* __restrict__ b = reinterpret_cast<const ulonglong2*>((party ? B.p[1] : B.p[0]) + (size_t)c * d);
        ulonglong2* __restrict__ f = reinterpret_cast<ulonglong2*>((party ? F.p[1] : F.p[0]) + (size_t)c * d);
        for (int t = threadIdx.x; t < pairs; t += blockDim.x) {
            const ulonglong2 wv = __ldg(w + t), bv = __ldg(b + t);
            f[t] = make_ulonglong2(wv.x - bv.x, wv.y - bv.y);
        }
    }
}

// ---------------------------------------------------------------------------
// K3 (down): F'_i[q, c] = W2_i[q, neuron(c)] - B'_i[q, c].  The paper's
// IndexRow (Protocol 3) on the stored transpose [d, D] is a gather of
// bs-word strips (256 or 512 contiguous bytes) out of every row q.
// Flat index over (q, c/2); consecutive threads walk consecutive pairs of a row.
// With blk_label (Protocol 3 under a per-token mask): a block no token uses (label < 0) holds no non-zero column
// of X, so its rows of Y are not masked and not sent: their message words are zero.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
open_weight_strips_kernel(PartyPtrs W2, PartyPtrs B, PartyOut F, const int32_t* __restrict__ ids,
                          int n, int bs, int d, int D, const int32_t* __restrict__ blk_label) {
    const int party = blockIdx.y;
    const int half_n = n >> 1;
    const int64_t total = (int64_t)d * half_n;
    const u64* __restrict__ W = (party ? W2.p[1] : W2.p[0]);
    const ulonglong2* __restrict__ b = reinterpret_cast<const ulonglong2*>((party ? B.p[1] : B.p[0]));
    ulonglong2* __restrict__ f = reinterpret_cast<ulonglong2*>((party ? F.p[1] : F.p[0]));
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const int q = (int)(t / half_n);
        const int c = (int)(t - (int64_t)q * half_n) << 1;
        if (blk_label && blk_label[c / bs] < 0) {
            f[t] = make_ulonglong2(0ull, 0ull);
            continue;
        }
        const int neuron = ids[c / bs] * bs + (c % bs);
        const ulonglong2 wv = __ldg(reinterpret_cast<const ulonglong2*>(W + (size_t)q * D + neuron));
        const ulonglong2 bv = __ldg(b + t);
        f[t] = make_ulonglong2(wv.x - bv.x, wv.y - bv.y);
    }
}

// ---------------------------------------------------------------------------
// K5: local truncation by f bits, in place.  Party 0: s >> f; party 1:
// -((-s) >> f), all on unsigned words.
// ---------------------------------------------------------------------------
__device__ __forceinline__ u64 trunc_word(u64 s, int f, int party) {
    return party == 0 ? (s >> f) : (0ull - ((0ull - s) >> f));
}

__global__ void __launch_bounds__(256)
truncate_kernel(PartyOut Z, int64_t pairs, int f) {
    pdl_wait();
    pdl_launch_dependents();
    const int party = blockIdx.y;
    ulonglong2* __restrict__ z = reinterpret_cast<ulonglong2*>((party ? Z.p[1] : Z.p[0]));
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < pairs; t += stride) {
        ulonglong2 v = z[t];
        v.x = trunc_word(v.x, f, party);
        v.y = trunc_word(v.y, f, party);
        z[t] = v;
    }
}

}  // namespace comet
