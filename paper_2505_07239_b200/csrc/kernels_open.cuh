// Memory-bound kernels of the path: mask compaction, the two "open" (masking)
// steps before the exchange, and local truncation.  Written for sm_100a with
// 128-bit coalesced accesses; blockIdx.y is the party.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

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
// `host_report` (mapped host memory) so that the host needs no copy, followed
// by `ticket` in host_report[2]: the host may watch that word instead of
// waiting for the stream.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
compact_mask_kernel(const uint8_t* __restrict__ mask, int nb, int32_t* __restrict__ ids, int32_t* __restrict__ count,
                    int32_t* __restrict__ host_report, int32_t ticket) {
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
        // {count, error flag raised by an earlier kernel's bounded wait} for the host, in mapped pinned memory
        host_report[0] = running;
        host_report[1] = count[1];
        __threadfence_system();
        *reinterpret_cast<volatile int32_t*>(host_report + 2) = ticket;
        __threadfence_system();
    }
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

// ---------------------------------------------------------------------------
// The first step of Protocol 2 on the GPU: connected components of the bipartite graph
// (token rows) x (active blocks) whose edges are the non-zero bytes of the
// per-token mask S [T, nab].  The paper uses depth-first search; here one CTA
// propagates minimum labels back and forth (block <- min over its tokens,
// token <- min over its blocks) until nothing changes, at most T + nab + 1
// rounds.  Every node of a component ends up with the component's smallest
// token index as its label; nodes without an edge get -1.
// report[0] = number of components, [1] = tokens with an edge, [2] = blocks with
// an edge (mapped host memory).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
token_components_kernel(const uint8_t* __restrict__ S, int T, int nab, int32_t* row_label, int32_t* blk_label,
                        long long* report) {
    __shared__ int changed;
    __shared__ int counts[3];
    const int tid = threadIdx.x;
    const int INF = 0x7fffffff;
    for (int r = tid; r < T; r += 1024) {
        bool edge = false;
        for (int b = 0; b < nab && !edge; ++b) edge = S[(size_t)r * nab + b] != 0;
        row_label[r] = edge ? r : INF;
    }
    for (int b = tid; b < nab; b += 1024) blk_label[b] = INF;
    if (tid == 0) counts[0] = counts[1] = counts[2] = 0;
    __syncthreads();
    for (int round = 0; round <= T + nab; ++round) {
        if (tid == 0) changed = 0;
        __syncthreads();
        for (int b = tid; b < nab; b += 1024) {
            int best = blk_label[b];
            for (int r = 0; r < T; ++r)
                if (S[(size_t)r * nab + b] != 0) best = min(best, row_label[r]);
            if (best < blk_label[b]) { blk_label[b] = best; changed = 1; }
        }
        __syncthreads();
        for (int r = tid; r < T; r += 1024) {
            int best = row_label[r];
            if (best != INF) {
                for (int b = 0; b < nab; ++b)
                    if (S[(size_t)r * nab + b] != 0) best = min(best, blk_label[b]);
                if (best < row_label[r]) { row_label[r] = best; changed = 1; }
            }
        }
        __syncthreads();
        if (!changed) break;
        __syncthreads();
    }
    for (int r = tid; r < T; r += 1024) {
        const int l = row_label[r];
        if (l == INF) row_label[r] = -1;
        else {
            atomicAdd(&counts[1], 1);
            if (l == r) atomicAdd(&counts[0], 1);
        }
    }
    for (int b = tid; b < nab; b += 1024) {
        if (blk_label[b] == INF) blk_label[b] = -1;
        else atomicAdd(&counts[2], 1);
    }
    __syncthreads();
    if (tid == 0) {
        report[0] = counts[0];
        report[1] = counts[1];
        report[2] = counts[2];
        __threadfence_system();
    }
}

// ---------------------------------------------------------------------------
// Protocol 2 asks for one multiplication per connected component, over that component's rows and columns only
// (Theorem 1's multiplication count).  On the tensor-core path this is ONE launch over component-sorted operands:
// rows and column blocks are ordered by component label (ties by index), so every component is a contiguous
// rectangle and an output tile has work only if the label ranges of its rows and of its columns intersect.
//   row_map [T]           sorted row position -> token row; rows of no component come last
//   col_map [groups*nab]  sorted block position -> compact block (group * nab + active block); within a
//                         component the order is (group, block); blocks of no component come last
//   tiles   [..]          (m-tile << 16) | n-tile of every tile with work, m-tiles of TM rows, n-tiles of TN columns
//   report[0] = number of listed tiles, report[1] = sum over components of rows x blocks (mapped host memory)
// One CTA of 1024 threads; needs ceil(live rows / TM) <= 1024.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
group_plan_kernel(const int32_t* __restrict__ row_label, const int32_t* __restrict__ blk_label, int T, int nab,
                  int groups, int bs, int TM, int TN, int32_t* row_map, int32_t* col_map, int32_t* tiles,
                  long long* report) {
    __shared__ int live_rows, live_blocks;
    __shared__ unsigned long long pairs;
    __shared__ int tn_first[1024], tn_count[1024], tile_off[1024];
    const int tid = threadIdx.x;
    if (tid == 0) { live_rows = 0; live_blocks = 0; pairs = 0ull; }
    __syncthreads();
    {
        int lr = 0, lb = 0;
        for (int r = tid; r < T; r += 1024) lr += row_label[r] >= 0;
        for (int b = tid; b < nab; b += 1024) lb += blk_label[b] >= 0;
        if (lr) atomicAdd(&live_rows, lr);
        if (lb) atomicAdd(&live_blocks, lb);
    }
    __syncthreads();
    const int M = live_rows, NB = live_blocks;
    unsigned long long my_pairs = 0;
    for (int r = tid; r < T; r += 1024) {
        const int l = row_label[r];
        int rank = 0;
        if (l >= 0) {
            for (int q = 0; q < T; ++q) {
                const int lq = row_label[q];
                rank += lq >= 0 && (lq < l || (lq == l && q < r));
            }
            for (int b = 0; b < nab; ++b) my_pairs += blk_label[b] == l;
        } else {
            rank = M;
            for (int q = 0; q < r; ++q) rank += row_label[q] < 0;
        }
        row_map[rank] = r;
    }
    if (my_pairs) atomicAdd(&pairs, my_pairs);
    for (int b = tid; b < nab; b += 1024) {
        const int l = blk_label[b];
        if (l >= 0) {
            int less = 0, same = 0, before = 0;
            for (int q = 0; q < nab; ++q) {
                const int lq = blk_label[q];
                less += lq >= 0 && lq < l;
                same += lq == l;
                before += lq == l && q < b;
            }
            for (int g = 0; g < groups; ++g) col_map[groups * less + g * same + before] = g * nab + b;
        } else {
            int before = 0;
            for (int q = 0; q < b; ++q) before += blk_label[q] < 0;
            for (int g = 0; g < groups; ++g) col_map[groups * NB + g * (nab - NB) + before] = g * nab + b;
        }
    }
    __syncthreads();
    const int N = groups * NB * bs;
    const int mt = (M + TM - 1) / TM, nt = (N + TN - 1) / TN;
    if (tid < mt) {
        const int lo_m = row_label[row_map[tid * TM]];
        const int hi_m = row_label[row_map[min(tid * TM + TM, M) - 1]];
        int first = 0, count = 0;
        for (int tn = 0; tn < nt; ++tn) {
            const int lo_n = blk_label[col_map[(tn * TN) / bs] % nab];
            const int hi_n = blk_label[col_map[(min(tn * TN + TN, N) - 1) / bs] % nab];
            if (hi_n >= lo_m && lo_n <= hi_m) {
                if (count == 0) first = tn;
                ++count;
            }
        }
        tn_first[tid] = first;
        tn_count[tid] = count;
    }
    __syncthreads();
    if (tid == 0) {
        int off = 0;
        for (int tm = 0; tm < mt; ++tm) { tile_off[tm] = off; off += tn_count[tm]; }
        report[0] = off;
        report[1] = (long long)pairs;
        __threadfence_system();
    }
    __syncthreads();
    if (tid < mt)
        for (int j = 0; j < tn_count[tid]; ++j) tiles[tile_off[tid] + j] = (tid << 16) | (tn_first[tid] + j);
}

// The Merge step of Protocol 2 on the compact result [T, cols]: an entry whose token and block are not in the same
// component is no part of any result block and is zero in both shares.  Compact column c belongs to active block
// (c mod n) / bs.  `pairs` = 16-byte word pairs per party.
__global__ void __launch_bounds__(256)
somm_merge_kernel(PartyOut Z, int64_t pairs, int cols, int n, int bs, const int32_t* __restrict__ row_label,
                  const int32_t* __restrict__ blk_label) {
    const int party = blockIdx.y;
    ulonglong2* __restrict__ z = reinterpret_cast<ulonglong2*>((party ? Z.p[1] : Z.p[0]));
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < pairs; t += stride) {
        const unsigned word = (unsigned)(2 * t), row = word / (unsigned)cols, col = word - row * (unsigned)cols;
        const int rl = row_label[row];
        if (rl < 0 || rl != blk_label[(col % (unsigned)n) / (unsigned)bs]) z[t] = make_ulonglong2(0ull, 0ull);
    }
}

// Number of non-zero bytes of a mask, written to `out` (mapped host memory) as a 64-bit count.
__global__ void __launch_bounds__(1024)
count_mask_kernel(const uint8_t* __restrict__ mask, long long count, long long* out) {
    __shared__ long long partial[32];
    long long mine = 0;
    for (long long t = threadIdx.x; t < count; t += 1024) mine += mask[t] != 0;
    for (int off = 16; off > 0; off >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, off);
    if ((threadIdx.x & 31) == 0) partial[threadIdx.x >> 5] = mine;
    __syncthreads();
    if (threadIdx.x < 32) {
        long long v = partial[threadIdx.x];
        for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
        if (threadIdx.x == 0) {
            *out = v;
            __threadfence_system();
        }
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
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
open_weight_strips_kernel(PartyPtrs W2, PartyPtrs B, PartyOut F, const int32_t* __restrict__ ids,
                          int n, int bs, int d, int D) {
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
