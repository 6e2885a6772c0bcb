// Oblivious shuffle, online stage (Section 4.2, Protocol 1): a row gather through a
// party's sub-permutation plus or minus a one-time mask,
//   mask step  : [y]_i = tau_i([x]_i) + a_i
//   finish step: [z]_i = rho_i([y]_other) - b_i
// with (p(x))[j] = x[p[j]] acting on the rows of a [rows, cols] matrix of ring
// words.  Pure HBM work: 16-byte accesses, consecutive threads on consecutive
// pieces of a row; blockIdx.y is the party.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace comet {

typedef unsigned long long u64;

struct ShuffleArgs {
    const u64* in[2];          // source matrix read by party 0 / party 1 (already swapped for the finish step)
    const int32_t* perm[2];    // the party's sub-permutation, `rows` entries
    const u64* mask[2];        // a_i or b_i, [rows, cols]
    u64* out[2];
    long long rows;
    int pieces;                // pieces per row: cols / 2 (16-byte pieces) or cols (8-byte pieces)
    int subtract;              // 0: out = gathered + mask, 1: out = gathered - mask
    long long stride_rows;     // (gridDim.x * blockDim.x) / pieces
    int stride_pieces;         // (gridDim.x * blockDim.x) % pieces
    int* bad_index;            // optional: set to 1 when a permutation entry is outside [0, rows)
};

// PIECE = ulonglong2 (even cols, 16-byte aligned pointers) or u64.
template <typename PIECE>
__device__ __forceinline__ PIECE shuffle_combine(PIECE g, PIECE m, int subtract);
template <>
__device__ __forceinline__ ulonglong2 shuffle_combine<ulonglong2>(ulonglong2 g, ulonglong2 m, int subtract) {
    return subtract ? make_ulonglong2(g.x - m.x, g.y - m.y) : make_ulonglong2(g.x + m.x, g.y + m.y);
}
template <>
__device__ __forceinline__ u64 shuffle_combine<u64>(u64 g, u64 m, int subtract) {
    return subtract ? g - m : g + m;
}
template <typename PIECE>
__device__ __forceinline__ PIECE shuffle_zero();
template <>
__device__ __forceinline__ ulonglong2 shuffle_zero<ulonglong2>() { return make_ulonglong2(0ull, 0ull); }
template <>
__device__ __forceinline__ u64 shuffle_zero<u64>() { return 0ull; }

template <typename PIECE>
__global__ void __launch_bounds__(256)
shuffle_rows_kernel(ShuffleArgs a) {
    const int party = blockIdx.y;
    const PIECE* __restrict__ in = reinterpret_cast<const PIECE*>(party ? a.in[1] : a.in[0]);
    const PIECE* __restrict__ mask = reinterpret_cast<const PIECE*>(party ? a.mask[1] : a.mask[0]);
    const int32_t* __restrict__ perm = party ? a.perm[1] : a.perm[0];
    PIECE* __restrict__ out = reinterpret_cast<PIECE*>(party ? a.out[1] : a.out[0]);
    const long long first = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long row = first / a.pieces;
    int piece = (int)(first - row * a.pieces);
    while (row < a.rows) {
        const long long src = perm[row];
        const long long at = row * a.pieces + piece;
        PIECE g;
        if (src >= 0 && src < a.rows) {
            g = __ldg(in + src * a.pieces + piece);
        } else {
            g = shuffle_zero<PIECE>();              // never read out of bounds; the caller sees the flag
            if (a.bad_index) *a.bad_index = 1;
        }
        out[at] = shuffle_combine<PIECE>(g, __ldg(mask + at), a.subtract);
        row += a.stride_rows;
        piece += a.stride_pieces;
        if (piece >= a.pieces) { piece -= a.pieces; ++row; }
    }
}

// inverse[perm[j]] = j: what a party does locally to obtain the sub-permutations of the unshuffle.
__global__ void __launch_bounds__(256)
invert_permutation_kernel(const int32_t* __restrict__ perm, int32_t* __restrict__ inverse, long long rows,
                          int* bad_index) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < rows; j += stride) {
        const long long p = perm[j];
        if (p >= 0 && p < rows) inverse[p] = (int32_t)j;
        else if (bad_index) *bad_index = 1;
    }
}

}  // namespace comet
