// K4, tensor-core variant: the gathered ring matmul + Beaver combine
//   Z_i = C_i + E*B_i + A_i*F + i*E*F = C_i + E*B_i + V_i*F,   V_i = A_i + i*E   (Eq. 1, party i)
// on the int8 tensor cores of sm_100a (tcgen05.mma kind::i8, accumulators in TMEM).
//
// A 64-bit ring word is eight unsigned 8-bit limbs, x = sum_p x_p 2^(8p).  Mod 2^64 only limb pairs with
// p + q <= 7 matter: x*y = sum_{s=0..7} 2^(8s) D_s, D_s = sum_{p+q=s} x_p y_q (36 of the 64 limb products).
// Each D_s summed over the contraction index is one 32-bit accumulator per output element: 8 accumulators
// of 128 x 64 fill the 512 TMEM columns of an SM exactly.  Only D_s mod 2^(64-8s) is needed, so 32-bit
// wrap-around is harmless for s >= 4, and for s <= 3 the exact sum (s+1)*K*255^2 stays below 2^32 while a
// segment accumulates at most 16384 contraction elements.
//
// Operands are kept as "blocked limb planes": for a tile of R rows (128 left, 64 right) and a block of 32
// contraction elements, 8 planes of R x 32 bytes, each stored as the tensor core's K-major no-swizzle
// canonical layout (8-row x 16-byte core matrices; the two 16-byte K halves of a row group adjacent).  One
// block is one contiguous bulk copy into shared memory.  With the planes of the right operand stacked
// along N, limb plane p of the left operand meets planes 0..7-p of the right operand in ONE instruction
// whose N spans accumulators D_p..D_7 (split in two when N > 256): 12 instructions per 32-deep step.
//
// Work is split stream-K style over a persistent grid: the (party, tile, k-block) space is cut into equal
// contiguous ranges, every segment's partial sums are added to Z with red.global.add.u64 -- exact and
// order-independent in the ring -- and Z is pre-loaded with C_i.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace comet {

typedef unsigned long long u64;

namespace limb {
constexpr int BM = 128, BN = 64, KC = 32, PLANES = 8;
constexpr int A_BLOCK_BYTES = PLANES * BM * KC;   // 32 KiB
constexpr int B_BLOCK_BYTES = PLANES * BN * KC;   // 16 KiB
constexpr int STAGES = 3;
constexpr int MAX_SEGMENT_UNITS = 16384 / KC;     // keeps the limb sums for s <= 3 below 2^32
constexpr int EPI_WARPS = 8;                      // warp w drains TMEM lanes 32*(w%4).., columns 32*(w/4)..
constexpr int THREADS = 32 * (EPI_WARPS + 2);     // warps 0-7 epilogue, warp 8 copy producer, warp 9 MMA issuer
// The opening kernel streams tiles of 32 rows x one k-block of the weight share and of the triple share through a
// two-stage ring in shared memory (asynchronous 16-byte copies, which hold no registers while in flight), several
// consecutive k-blocks per CTA: the copies of the next k-block fly while the current one is turned into the message
// and the planes.
constexpr int OPEN_ROWS = 32, OPEN_THREADS = 128, OPEN_STAGES = 2;
constexpr int OPEN_STRIDE = KC + 2;               // words per staged row: 272 bytes keep every row 16-byte aligned and
                                                  // the 16-byte reads of eight consecutive rows on distinct banks
constexpr int OPEN_TILE_BYTES = OPEN_ROWS * OPEN_STRIDE * 8;
constexpr size_t OPEN_SMEM_BYTES = (size_t)OPEN_STAGES * 2 * OPEN_TILE_BYTES;      // a W and a B tile per stage: 34 KiB
constexpr int OPEN_MAX_KB_PER_CTA = 8;
constexpr int OUT_COLS = 16;                      // words per staged output row (a thread's 32 go in two rounds)
constexpr int OUT_ROW_BYTES = OUT_COLS * 8 + 16;  // padded against bank conflicts
constexpr size_t SMEM_BYTES = (size_t)STAGES * (A_BLOCK_BYTES + B_BLOCK_BYTES) + (size_t)EPI_WARPS * 32 * OUT_ROW_BYTES + 128;
constexpr long long WAIT_CYCLES = 4000000000ll;   // ~2 s at 1.9 GHz: every wait gives up after this
constexpr unsigned LBO_BYTES = 128, SBO_BYTES = 256;

// byte offset of (plane p, row r, contraction index k in [0,32)) inside a block of `rows` rows
__host__ __device__ __forceinline__ int block_offset(int rows, int p, int r, int k) {
    return p * rows * KC + (r >> 3) * 256 + (k >> 4) * 128 + (r & 7) * 16 + (k & 15);
}
}  // namespace limb

// ---------------------------------------------------------------------------
// Blocked limb planes: helpers shared by the two memory-side kernels below.
// A CTA tile is 32 rows x 32 contraction elements; words are staged in shared memory as [row][34], which keeps
// every row 16-byte aligned for the asynchronous copies (16 threads per row) and puts the 16-byte reads of eight
// consecutive rows, as the byte transposition issues them, on distinct banks.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void limb_transpose4(unsigned x0, unsigned x1, unsigned x2, unsigned x3,
                                                unsigned& p0, unsigned& p1, unsigned& p2, unsigned& p3) {
    const unsigned t0 = __byte_perm(x0, x1, 0x5140), t1 = __byte_perm(x2, x3, 0x5140);
    const unsigned t2 = __byte_perm(x0, x1, 0x7362), t3 = __byte_perm(x2, x3, 0x7362);
    p0 = __byte_perm(t0, t1, 0x5410);
    p1 = __byte_perm(t0, t1, 0x7632);
    p2 = __byte_perm(t2, t3, 0x5410);
    p3 = __byte_perm(t2, t3, 0x7632);
}

// Split the 16 words at `src` (16-byte aligned, shared memory) into 8 limb planes of 16 bytes and store them at
// (plane, row `rin`, k = 16*half) of the block `blk`, whose tiles have `tile_rows` rows.
__device__ __forceinline__ void limb_emit_planes16(const u64* src, int half, uint8_t* blk, int tile_rows, int rin) {
    unsigned lo[16], hi[16];
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(src + j);
        lo[j] = (unsigned)v.x;
        hi[j] = (unsigned)(v.x >> 32);
        lo[j + 1] = (unsigned)v.y;
        hi[j + 1] = (unsigned)(v.y >> 32);
    }
    uint4 plane[8];
    limb_transpose4(lo[0], lo[1], lo[2], lo[3], plane[0].x, plane[1].x, plane[2].x, plane[3].x);
    limb_transpose4(lo[4], lo[5], lo[6], lo[7], plane[0].y, plane[1].y, plane[2].y, plane[3].y);
    limb_transpose4(lo[8], lo[9], lo[10], lo[11], plane[0].z, plane[1].z, plane[2].z, plane[3].z);
    limb_transpose4(lo[12], lo[13], lo[14], lo[15], plane[0].w, plane[1].w, plane[2].w, plane[3].w);
    limb_transpose4(hi[0], hi[1], hi[2], hi[3], plane[4].x, plane[5].x, plane[6].x, plane[7].x);
    limb_transpose4(hi[4], hi[5], hi[6], hi[7], plane[4].y, plane[5].y, plane[6].y, plane[7].y);
    limb_transpose4(hi[8], hi[9], hi[10], hi[11], plane[4].z, plane[5].z, plane[6].z, plane[7].z);
    limb_transpose4(hi[12], hi[13], hi[14], hi[15], plane[4].w, plane[5].w, plane[6].w, plane[7].w);
#pragma unroll
    for (int p = 0; p < 8; ++p)
        *reinterpret_cast<uint4*>(blk + limb::block_offset(tile_rows, p, rin, half * 16)) = plane[p];
}

// 16-byte asynchronous copy global -> shared that bypasses L1; with `bytes` = 0 nothing is read and the 16 bytes
// are filled with zeros.  (The form that also carries an L2 cache-policy operand raised an illegal-instruction
// error on this part when combined with the byte count, so no eviction hint is given here.)
__device__ __forceinline__ void limb_copy16_async(uint32_t dst_smem, const void* src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void limb_copy_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void limb_copy_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

__device__ __forceinline__ uint8_t* limb_block_ptr(uint8_t* base, int tile_rows, int row, int kblocks, int kb,
                                                   int* rin) {
    const int tile = row >> (31 - __clz(tile_rows));          // tile_rows is 32, 64 or 128
    *rin = row - tile * tile_rows;
    return base + ((size_t)tile * kblocks + kb) * (size_t)(limb::PLANES * tile_rows * limb::KC);
}

// ---------------------------------------------------------------------------
// Before the exchange (Section 2.1 "Multiplication"; IndexCols of Protocol 2, IndexRow of Protocol 3), one launch:
//   left  blocks: E_i = X_i - A_i, elementwise;
//   right tiles : F_i = gather(W_i) - B_i written as the message, and the blocked limb planes of the party's
//                 own B_i (it is in registers anyway, so it is not read a second time later).
// gather: up   (down = 0): row c of the right operand is row neuron(c) of W (whole rows of `ldw` words);
//         down (down = 1): contraction index c is column neuron(c) of W (strips of `bs` words in every row).
// grid = 2 * (left_blocks + row_tiles * kchunks), 128 threads, the party being the lowest bit of the block index
// (both parties' messages are then written in the same order, which the next kernel reads backwards).  A right CTA
// owns 32 rows and kb_per_cta consecutive k-blocks: while it turns one k-block into the message and the planes, the
// loads of the next one are in flight (the kernel is bound by memory latency, not by bandwidth, when a CTA loads,
// waits and works in turn).  Dynamic shared memory: OPEN_SMEM_BYTES when there are right tiles.
// ---------------------------------------------------------------------------
struct LimbOpenArgs {
    const u64* X[2];
    const u64* A[2];
    u64* E[2];
    long long left_pairs;
    int left_blocks;
    const u64* W0[2];        // weights of group 0 (gate when gated, else the only matrix)
    const u64* W1[2];        // weights of group 1 (up-projection of a gated FFN)
    const u64* W2g[2];       // weights of group 2 (third stacked matrix, e.g. the value projection)
    const u64* B[2];
    u64* F[2];
    uint8_t* Bpl[2];
    const int32_t* ids;      // ascending active block ids
    int n, bs;               // active neurons, neurons per block
    int rows, K;             // logical size of the right operand [rows, K]
    int ldw;                 // words per row of W
    int kblocks, down;
    int kb_per_cta, kchunks; // k-blocks per right CTA and CTAs per row tile: kchunks = ceil(kblocks / kb_per_cta)
    int right_tile_rows;     // rows per plane tile of the right operand: 64, or 128 for the few-token kernel
    // Protocol 3 with per-column row sets: per-token mask over the active blocks, [rows of X, tmask_ld] bytes, or
    // null.  Where it is zero the entry of X is no non-zero: it is not opened and E_i is zero there.
    const uint8_t* tmask;
    int tmask_ld;
    // Protocol 2 over connected components: component label per row of X and per active block (-1 = in no
    // component), or null.  A row / column outside every component is not opened: its message words are zero.
    // Protocol 3 (down) uses blk_label alone: a block no token uses holds no non-zero column of X, and the rows of
    // the right operand that belong to it are not opened either.
    const int32_t* row_label;
    const int32_t* blk_label;
    // With col_map (up only; one multiplication per component): row r of the plane tiles is compact row
    // col_map[r / bs] * bs + r % bs of the right operand, i.e. the planes are written in component order while the
    // message F_i keeps the compact order.
    const int32_t* col_map;
    // With kmap (down only): contraction index k of the plane tiles is compact index kmap[k / bs] * bs + k % bs,
    // i.e. the planes run over the active blocks in component order while F_i keeps the compact order.
    const int32_t* kmap;
    // Few-token products: the party's message F_i is written as blocked limb planes (same layout as Bpl) INSTEAD of
    // as words: the product kernel reads both parties' messages in that form, so no plane of their sum has to be
    // built and the words are never needed on the path (limb_planes_to_words_kernel rebuilds them when asked for).
    uint8_t* Fpl[2];
    int emit_f;
};

__global__ void __launch_bounds__(limb::OPEN_THREADS)
limb_open_kernel(LimbOpenArgs a) {
    using namespace limb;
    pdl_wait();
    pdl_launch_dependents();
    const int party = blockIdx.x & 1;
    const int bid = blockIdx.x >> 1;
    const int tid = threadIdx.x;
    if (bid < a.left_blocks) {
        const ulonglong2* __restrict__ x = reinterpret_cast<const ulonglong2*>(party ? a.X[1] : a.X[0]);
        const ulonglong2* __restrict__ m = reinterpret_cast<const ulonglong2*>(party ? a.A[1] : a.A[0]);
        ulonglong2* __restrict__ e = reinterpret_cast<ulonglong2*>(party ? a.E[1] : a.E[0]);
        const long long stride = (long long)a.left_blocks * OPEN_THREADS;
        for (long long t = (long long)bid * OPEN_THREADS + tid; t < a.left_pairs; t += stride) {
            if (a.tmask) {
                const unsigned word = (unsigned)(2 * t), row = word / (unsigned)a.K, col = word - row * (unsigned)a.K;
                if (a.tmask[(size_t)row * a.tmask_ld + col / (unsigned)a.bs] == 0) {
                    e[t] = make_ulonglong2(0ull, 0ull);
                    continue;
                }
            }
            if (a.row_label && a.row_label[(unsigned)(2 * t) / (unsigned)a.K] < 0) {
                e[t] = make_ulonglong2(0ull, 0ull);
                continue;
            }
            const ulonglong2 xv = __ldcs(x + t), av = __ldcs(m + t);      // read once: leave L2 to what is written
            e[t] = make_ulonglong2(xv.x - av.x, xv.y - av.y);
        }
        return;
    }
    extern __shared__ __align__(16) uint8_t open_smem[];      // [stage][W tile | B tile], rows of OPEN_STRIDE words
    const int tile_id = bid - a.left_blocks;
    const int chunk = tile_id % a.kchunks;
    const int row0 = (tile_id / a.kchunks) * OPEN_ROWS;
    const int kb0 = chunk * a.kb_per_cta;
    const int kb1 = min(kb0 + a.kb_per_cta, a.kblocks);
    const u64* __restrict__ Bi = party ? a.B[1] : a.B[0];
    u64* __restrict__ Fi = party ? a.F[1] : a.F[0];
    // What depends on the row alone (which row of which weight matrix is gathered, where the row lies in B_i / F_i,
    // whether its block is in use) is worked out once per row and shared.
    __shared__ const u64* s_wrow[OPEN_ROWS];          // first word of the gathered row of W_i; null: no such row
    __shared__ long long s_orow[OPEN_ROWS];           // offset of the row in B_i and F_i
    __shared__ unsigned char s_dead[OPEN_ROWS];
    if (tid < OPEN_ROWS) {
        int row = row0 + tid;
        const u64* wp = nullptr;
        long long o = 0;
        bool dead = false;
        if (row < a.rows) {
            if (a.col_map) {
                const int sb = row / a.bs;
                row = __ldg(a.col_map + sb) * a.bs + (row - sb * a.bs);
            }
            if (a.down) {
                wp = (party ? a.W0[1] : a.W0[0]) + (size_t)row * a.ldw;
            } else {
                const int grp = (row >= a.n) + (row >= 2 * a.n), j = row - grp * a.n;
                const int blk = j / a.bs;
                const int neuron = __ldg(a.ids + blk) * a.bs + (j - blk * a.bs);
                dead = a.blk_label && a.blk_label[blk] < 0;
                wp = (grp == 0 ? (party ? a.W0[1] : a.W0[0])
                               : grp == 1 ? (party ? a.W1[1] : a.W1[0]) : (party ? a.W2g[1] : a.W2g[0])) +
                     (size_t)neuron * a.ldw;
            }
            o = (long long)row * a.K;
        }
        s_wrow[tid] = wp;
        s_orow[tid] = o;
        s_dead[tid] = dead ? 1 : 0;
    }
    __syncthreads();

    // This thread's part of every tile: the 16-byte column c16 (contraction indices 2 c16, 2 c16 + 1 of the k-block)
    // of the rows rbase, rbase + 8, rbase + 16, rbase + 24.
    const int c16 = tid & 15, rbase = tid >> 4;

    // contraction index of this thread's column in k-block kb: plane position k, compact index ks, column kcol of the
    // gathered row of W_i, and whether the block it belongs to is in use (down only)
    auto column = [&](int kb, int& k, int& ks, int& kcol, bool& dead_k) {
        k = kb * KC + 2 * c16;
        ks = k;
        if (a.kmap && k < a.K) {
            const int sb = k / a.bs;
            ks = __ldg(a.kmap + sb) * a.bs + (k - sb * a.bs);
        }
        kcol = k;
        dead_k = false;
        if (a.down && k < a.K) {
            const int blk = ks / a.bs;
            kcol = __ldg(a.ids + blk) * a.bs + (ks - blk * a.bs);
            dead_k = a.blk_label && a.blk_label[blk] < 0;     // a block without a non-zero column of X
        }
    };
    // asynchronous 16-byte copies of this thread's part of k-block kb into a stage; what lies outside the operand
    // is filled with zeros
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(open_smem);
    auto issue = [&](int kb, int stage) {
        int k, ks, kcol;
        bool dead_k;
        column(kb, k, ks, kcol, dead_k);
        const uint32_t w_tile = smem0 + (uint32_t)stage * 2u * OPEN_TILE_BYTES, b_tile = w_tile + OPEN_TILE_BYTES;
#pragma unroll
        for (int i = 0; i < OPEN_ROWS / 8; ++i) {
            const int r = rbase + 8 * i;
            const u64* wp = s_wrow[r];
            const bool live = wp != nullptr && k < a.K;
            const uint32_t at = (uint32_t)(r * OPEN_STRIDE * 8 + c16 * 16);
            limb_copy16_async(w_tile + at, live ? (const void*)(wp + kcol) : (const void*)Bi, live ? 16u : 0u);
            limb_copy16_async(b_tile + at, live ? (const void*)(Bi + s_orow[r] + ks) : (const void*)Bi, live ? 16u : 0u);
        }
        limb_copy_commit();
    };

    issue(kb0, 0);
    for (int kb = kb0; kb < kb1; ++kb) {
        const int stage = (kb - kb0) & 1;
        if (kb + 1 < kb1) {
            issue(kb + 1, stage ^ 1);        // that stage was released by the barrier that ended the last round
            limb_copy_wait<1>();
        } else {
            limb_copy_wait<0>();
        }
        __syncthreads();                     // every thread's copies of this stage have landed
        u64* w_tile = reinterpret_cast<u64*>(open_smem + (size_t)stage * 2 * OPEN_TILE_BYTES);
        u64* b_tile = w_tile + OPEN_ROWS * OPEN_STRIDE;
        int k, ks, kcol;
        bool dead_k;
        column(kb, k, ks, kcol, dead_k);
        // the message F_i = gather(W_i) - B_i: written as words, or left in place of the W tile for the planes
#pragma unroll
        for (int i = 0; i < OPEN_ROWS / 8; ++i) {
            const int r = rbase + 8 * i;
            const bool live = s_wrow[r] != nullptr && k < a.K;
            const bool dead = dead_k || s_dead[r] != 0;
            ulonglong2* wv = reinterpret_cast<ulonglong2*>(w_tile + r * OPEN_STRIDE + 2 * c16);
            const ulonglong2 w = *wv;
            const ulonglong2 b = *reinterpret_cast<const ulonglong2*>(b_tile + r * OPEN_STRIDE + 2 * c16);
            const ulonglong2 f = dead ? make_ulonglong2(0ull, 0ull) : make_ulonglong2(w.x - b.x, w.y - b.y);
            if (a.emit_f) *wv = f;
            else if (live) *reinterpret_cast<ulonglong2*>(Fi + s_orow[r] + ks) = f;
        }
        if (a.emit_f) __syncthreads();       // the planes of F_i are built from words other threads wrote
        // planes of B_i (threads 0-63) and, with emit_f, of F_i (threads 64-127): 16 words of one row each
        const int which = tid >> 6, half = (tid >> 5) & 1, r = tid & 31;
        if (which == 0 || a.emit_f) {
            int rin;
            uint8_t* blk = limb_block_ptr(which ? (party ? a.Fpl[1] : a.Fpl[0]) : (party ? a.Bpl[1] : a.Bpl[0]),
                                          a.right_tile_rows, row0 + r, a.kblocks, kb, &rin);
            limb_emit_planes16((which ? w_tile : b_tile) + r * OPEN_STRIDE + half * 16, half, blk, a.right_tile_rows, rin);
        }
        __syncthreads();                     // the stage may be overwritten by the copies issued next round
    }
}

// Blocked limb planes back to words: out[row, k] for a [rows, K] operand whose plane tiles have `tile_rows` rows.
// Only used off the path, when a message that was written as planes is read back as words.
__global__ void __launch_bounds__(256)
limb_planes_to_words_kernel(const uint8_t* __restrict__ planes, u64* __restrict__ out, int rows, int K, int kblocks,
                            int tile_rows) {
    const long long total = (long long)rows * K, stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const int row = (int)(t / K), k = (int)(t - (long long)row * K);
        const int tile = row / tile_rows, rin = row - tile * tile_rows, kb = k / limb::KC, kin = k - kb * limb::KC;
        const uint8_t* blk = planes + ((size_t)tile * kblocks + kb) * (size_t)(limb::PLANES * tile_rows * limb::KC);
        u64 v = 0;
#pragma unroll
        for (int p = 0; p < limb::PLANES; ++p) v |= (u64)blk[limb::block_offset(tile_rows, p, rin, kin)] << (8 * p);
        out[t] = v;
    }
}

// ---------------------------------------------------------------------------
// After the exchange, one launch: everything the tensor-core kernel needs, per party.
//   left tiles : E = E_0 + E_1 -> planes(E);  V_i = A_i + i*E -> planes(V_i)      [M, K], 128-row blocks
//   right tiles: F = F_0 + F_1 -> planes(F)                                      [N, K],  64-row blocks
//   copy blocks: Z_i <- C_i (the accumulation target starts from the triple's C share)
// grid = 2 * (left_tiles + right_tiles + copy_blocks), 128 threads; a tile CTA owns 32 rows x kb_per_cta k-blocks.
// Any part may be empty.  Dynamic shared memory: 2 stages x (3 tiles with a left part, else 2) x OPEN_TILE_BYTES.
// The party is the lowest bit of the block index: the two parties' CTAs of one tile read the same two messages and
// run side by side, so the second read comes from L2.  Tiles are taken from the last to the first: the kernel before
// this one wrote the messages in ascending order, and its last tiles are the ones most likely still in L2.
// ---------------------------------------------------------------------------
struct LimbPrepArgs {
    const u64* E0; const u64* E1;
    const u64* A[2];
    uint8_t* Epl[2];
    uint8_t* Vpl[2];
    int M, left_tiles;       // left_tiles = (32-row tiles of whole plane tiles) * kchunks, or 0
    int kb_per_cta, kchunks; // k-blocks per tile CTA and CTAs per row tile: kchunks = ceil(kblocks / kb_per_cta)
    const u64* F0; const u64* F1;
    uint8_t* Fpl[2];
    int N, right_tiles;      // likewise for the right operand
    int K, kblocks;
    int left_tile_rows, right_tile_rows;   // rows per plane tile: 128 / 64, or 32 / 128 for the few-token kernel
    const uint8_t* tmask;    // per-token mask over the active blocks (see LimbOpenArgs), or null: where it is zero
    int tmask_ld, bs;        // the party's A_i is no part of the triple and counts as zero
    const u64* C[2];
    u64* Z[2];
    long long copy_pairs;
    int copy_blocks;
    // One multiplication per component (up only): plane row r of the left operand is row row_map[r] of E and A_i,
    // plane row r of the right operand is compact row col_map[r / bs] * bs + r % bs of F; M and N then count the
    // rows and columns that lie in a component.  Null: identity.
    const int32_t* row_map;
    const int32_t* col_map;
    // Down only: contraction index k of the planes is compact index kmap[k / bs] * bs + k % bs (both operands).
    const int32_t* kmap;
};

__global__ void __launch_bounds__(limb::OPEN_THREADS)
limb_prep_kernel(LimbPrepArgs a) {
    using namespace limb;
    pdl_wait();
    pdl_launch_dependents();
    const int party = blockIdx.x & 1;
    const int tid = threadIdx.x;
    int id = blockIdx.x >> 1;
    if (id < a.left_tiles + a.right_tiles) {
        id = a.left_tiles + a.right_tiles - 1 - id;
    } else {
        id -= a.left_tiles + a.right_tiles;
        const ulonglong2* __restrict__ s = reinterpret_cast<const ulonglong2*>(party ? a.C[1] : a.C[0]);
        ulonglong2* __restrict__ d = reinterpret_cast<ulonglong2*>(party ? a.Z[1] : a.Z[0]);
        const long long stride = (long long)a.copy_blocks * OPEN_THREADS;
        for (long long t = (long long)id * OPEN_THREADS + tid; t < a.copy_pairs; t += stride) d[t] = __ldcs(s + t);
        return;
    }
    // A tile CTA owns 32 rows and kb_per_cta consecutive k-blocks and streams them through a two-stage ring of
    // asynchronous copies, as the opening kernel does: per stage the two messages and, on the left, the party's A_i.
    extern __shared__ __align__(16) uint8_t prep_smem[];     // [stage][message 0 | message 1 | (left) A_i]
    const bool left = id < a.left_tiles;
    if (!left) id -= a.left_tiles;
    const int chunk = id % a.kchunks;
    const int row0 = (id / a.kchunks) * OPEN_ROWS;
    const int kb0 = chunk * a.kb_per_cta;
    const int kb1 = min(kb0 + a.kb_per_cta, a.kblocks);
    const int rows = left ? a.M : a.N;
    const int tiles_per_stage = left ? 3 : 2;
    const u64* __restrict__ in0 = left ? a.E0 : a.F0;
    const u64* __restrict__ in1 = left ? a.E1 : a.F1;
    const u64* __restrict__ own = party ? a.A[1] : a.A[0];
    __shared__ int s_row[OPEN_ROWS];                  // the row of the operands a tile row stands for; -1: none
    if (tid < OPEN_ROWS) {
        int row = row0 + tid;
        if (row >= rows) {
            row = -1;
        } else if (left) {
            if (a.row_map) row = __ldg(a.row_map + row);
        } else if (a.col_map) {
            const int sb = row / a.bs;
            row = __ldg(a.col_map + sb) * a.bs + (row - sb * a.bs);
        }
        s_row[tid] = row;
    }
    __syncthreads();

    const int c16 = tid & 15, rbase = tid >> 4;
    const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(prep_smem);
    const uint32_t stage_bytes = (uint32_t)tiles_per_stage * OPEN_TILE_BYTES;
    // plane position k of this thread's column in k-block kb and its compact contraction index ks
    auto column = [&](int kb, int& k, int& ks) {
        k = kb * KC + 2 * c16;
        ks = k;
        if (a.kmap && k < a.K) {
            const int sb = k / a.bs;
            ks = __ldg(a.kmap + sb) * a.bs + (k - sb * a.bs);
        }
    };
    auto issue = [&](int kb, int stage) {
        int k, ks;
        column(kb, k, ks);
        const uint32_t t0 = smem0 + (uint32_t)stage * stage_bytes;
#pragma unroll
        for (int i = 0; i < OPEN_ROWS / 8; ++i) {
            const int r = rbase + 8 * i;
            const int row = s_row[r];
            const bool live = row >= 0 && k < a.K;
            const size_t o = live ? (size_t)row * a.K + ks : 0;
            const uint32_t at = (uint32_t)(r * OPEN_STRIDE * 8 + c16 * 16);
            limb_copy16_async(t0 + at, in0 + o, live ? 16u : 0u);
            limb_copy16_async(t0 + OPEN_TILE_BYTES + at, in1 + o, live ? 16u : 0u);
            if (left) limb_copy16_async(t0 + 2 * OPEN_TILE_BYTES + at, own + o, live ? 16u : 0u);
        }
        limb_copy_commit();
    };

    issue(kb0, 0);
    for (int kb = kb0; kb < kb1; ++kb) {
        const int stage = (kb - kb0) & 1;
        if (kb + 1 < kb1) {
            issue(kb + 1, stage ^ 1);        // that stage was released by the barrier that ended the last round
            limb_copy_wait<1>();
        } else {
            limb_copy_wait<0>();
        }
        __syncthreads();                     // every thread's copies of this stage have landed
        u64* t_sum = reinterpret_cast<u64*>(prep_smem + (size_t)stage * stage_bytes);      // message 0, then the sum
        u64* t_in1 = t_sum + OPEN_ROWS * OPEN_STRIDE;
        u64* t_own = t_in1 + OPEN_ROWS * OPEN_STRIDE;                                       // A_i, then V_i (left)
        int k, ks;
        column(kb, k, ks);
#pragma unroll
        for (int i = 0; i < OPEN_ROWS / 8; ++i) {
            const int r = rbase + 8 * i;
            const int at = r * OPEN_STRIDE + 2 * c16;
            ulonglong2* sv = reinterpret_cast<ulonglong2*>(t_sum + at);
            const ulonglong2 x = *sv, y = *reinterpret_cast<const ulonglong2*>(t_in1 + at);
            const ulonglong2 sum = make_ulonglong2(x.x + y.x, x.y + y.y);       // the exchange: both messages summed
            *sv = sum;
            if (left) {
                // where the per-token mask is zero the party's A_i is no part of the triple and counts as zero
                const int row = s_row[r];
                const bool own_part = row >= 0 && k < a.K &&
                                      (!a.tmask || a.tmask[(size_t)row * a.tmask_ld + ks / a.bs] != 0);
                ulonglong2* ov = reinterpret_cast<ulonglong2*>(t_own + at);
                const ulonglong2 z = *ov;
                *ov = own_part ? make_ulonglong2(z.x + (party ? sum.x : 0ull), z.y + (party ? sum.y : 0ull))   // V_i = A_i + i*E
                               : make_ulonglong2(0ull, 0ull);
            }
        }
        __syncthreads();                     // the planes are built from words other threads wrote
        // threads 0-63: planes of the summed message; threads 64-127 (left only): planes of V_i; 16 words of a row each
        const int which = tid >> 6, half = (tid >> 5) & 1, r = tid & 31;
        if (which == 0 || left) {
            const int tile_rows = left ? a.left_tile_rows : a.right_tile_rows;
            uint8_t* base = left ? (which ? (party ? a.Vpl[1] : a.Vpl[0]) : (party ? a.Epl[1] : a.Epl[0]))
                                 : (party ? a.Fpl[1] : a.Fpl[0]);
            int rin;
            uint8_t* blk = limb_block_ptr(base, tile_rows, row0 + r, a.kblocks, kb, &rin);
            limb_emit_planes16((which ? t_own : t_sum) + r * OPEN_STRIDE + half * 16, half, blk, tile_rows, rin);
        }
        __syncthreads();                     // the stage may be overwritten by the copies issued next round
    }
}

// ---------------------------------------------------------------------------
// PTX wrappers (sm_100a)
// ---------------------------------------------------------------------------
namespace ptx {
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// shared -> global bulk reduction: 64-bit integer add of `bytes` (multiple of 16) contiguous bytes
__device__ __forceinline__ void bulk_reduce_add_u64(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.u64 [%0], [%1], %2;"
                 ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_group0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem desc] * B[smem desc], u8 x u8 -> s32.  The descriptors are passed as (low, high) words: only
// the low word (the shared-memory address field) changes between instructions.
#define COMET_MMA_I8(NAME, QUAL)                                                                                   \
    __device__ __forceinline__ void NAME(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,            \
                                         uint32_t b_hi, uint32_t idesc, uint32_t acc) {                           \
        asm volatile(                                                                                              \
            "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"                                                           \
            "setp.ne.b32 p, %6, 0;\n\t"                                                                            \
            "mov.b64 da, {%1, %2};\n\t"                                                                            \
            "mov.b64 db, {%3, %4};\n\t"                                                                            \
            "tcgen05.mma.cta_group::1.kind::i8" QUAL " [%0], da, db, %5, p;\n\t}"                                  \
            ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(acc) : "memory");          \
    }
COMET_MMA_I8(mma_i8, "")                               // A operand fetched for this instruction only
COMET_MMA_I8(mma_i8_keep_a, ".collector::a::fill")     // A operand kept in the collector for the next instruction
COMET_MMA_I8(mma_i8_reuse_a, ".collector::a::lastuse") // A operand taken from the collector, then dropped
#undef COMET_MMA_I8
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* d) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
}  // namespace ptx

// ---------------------------------------------------------------------------
// What a per-token mask S [T, nab] (non-zero byte = token t uses active block b) implies, in one launch of one CTA.
//
// 1. The first step of Protocol 2: the connected components of the bipartite graph (token rows) x (active
//    blocks) with the non-zero bytes as edges.  The paper uses depth-first search; here S becomes a bit matrix
//    and minimum labels are propagated without atomics: every block takes the minimum over its rows (one warp per
//    block), then every row the minimum over its blocks (one thread per row), until nothing changes (at most
//    T + nab + 1 sweeps).  Every node of a component ends up with the component's smallest token index as its
//    label; nodes without an edge get -1.
//
// 2. (plan != 0) Protocols 2 and 3 ask for one multiplication per component / per non-zero column entry, over the
//    rows and columns that take part only (the multiplication counts of Theorems 1 and 2).  On the tensor cores
//    this becomes ONE launch over component-sorted operands: token rows and active blocks are ordered by
//    component label (ties by index), so every component is a contiguous rectangle, and
//      up   (Protocol 2): an output tile has work only if the label ranges of its rows and of its columns
//                         intersect; per row tile these column tiles form an interval;
//      down (Protocol 3): a row tile's contraction runs only over the blocks of the components its rows belong
//                         to, an interval of k-blocks in the sorted order of the contraction index.
//    row_map [T]           sorted row position -> token row; rows of no component come last
//    col_map [groups*nab]  sorted block position -> compact block (group * nab + active block) of the
//                          up-projection's columns; inside a component the order is (group, block); blocks of no
//                          component last
//    kmap    [nab]         sorted block position -> active block, for the down-projection's contraction index
//    up, dn  [row tiles]   the work of every tile of 128 sorted rows (LimbGroupRow); needs at most 32768 tokens
//
// report (mapped host memory): [0] edges, [1] components, [2] rows with an edge, [3] blocks with an edge,
// [4] k-block units of the up-projection per party, [5] sum over components of rows x blocks, [6] units of the
// down-projection per party ([4..6] only with plan).
// Working storage: bit matrix [T, wpr] words, labels, and the labels of the sorted column blocks, in dynamic
// shared memory when `in_smem` (T*wpr + T + nab + groups*nab words), else in `scratch` (global, same size) with
// the labels kept in the output arrays.
// ---------------------------------------------------------------------------
struct LimbGroupRow {
    int unit0;       // units (k-blocks, both operand pairs) of the row tiles before this one, per party
    int tn0, ntn;    // interval of column tiles with work
    int klo, kcnt;   // interval of k-blocks with work; a tile runs over 2 * kcnt units
};

struct TokenPlanArgs {
    const uint8_t* S;
    int T, nab, wpr;             // wpr = ceil(nab / 32)
    int32_t* row_label;          // out [T]
    int32_t* blk_label;          // out [nab]
    long long* report;
    int in_smem;
    uint32_t* scratch;
    int plan, groups, bs, kb_up, nt_dn;
    int32_t* row_map;
    int32_t* col_map;
    int32_t* kmap;
    LimbGroupRow* up;
    LimbGroupRow* dn;
};

__global__ void __launch_bounds__(1024, 1)
token_plan_kernel(TokenPlanArgs a) {
    constexpr int TM = limb::BM, TN = limb::BN, KC = limb::KC;
    extern __shared__ uint32_t plan_smem[];
    __shared__ int counts[3];
    __shared__ unsigned long long edges, pairs;
    __shared__ int units_up[1024], units_dn[1024];
    const int tid = threadIdx.x;
    const int T = a.T, nab = a.nab, wpr = a.wpr;
    const int INF = 0x7fffffff;
    uint32_t* bits = a.in_smem ? plan_smem : a.scratch;
    int* rl = a.in_smem ? reinterpret_cast<int*>(plan_smem + (size_t)T * wpr) : a.row_label;
    int* bl = a.in_smem ? rl + T : a.blk_label;
    int* sorted_bl = a.in_smem ? bl + nab : reinterpret_cast<int*>(a.scratch + (size_t)T * wpr);

    const int warp = tid >> 5, lane = tid & 31;
    for (int w = tid; w < T * wpr; w += 1024) bits[w] = 0u;
    for (int b = tid; b < nab; b += 1024) bl[b] = INF;
    if (tid == 0) { counts[0] = counts[1] = counts[2] = 0; edges = 0ull; pairs = 0ull; }
    __syncthreads();
    {
        // S is read four bytes at a time (its buffer is 256-byte aligned); the last 0-3 bytes singly
        const int total = T * nab, words = total >> 2;
        const uint32_t* S4 = reinterpret_cast<const uint32_t*>(a.S);
        for (int q = tid; q < words; q += 1024) {
            uint32_t v = __ldg(S4 + q);
            if (v == 0u) continue;
#pragma unroll
            for (int k = 0; k < 4; ++k, v >>= 8)
                if (v & 0xffu) {
                    const int t = 4 * q + k, r = t / nab, b = t - r * nab;
                    atomicOr(&bits[r * wpr + (b >> 5)], 1u << (b & 31));
                }
        }
        for (int t = 4 * words + tid; t < total; t += 1024)
            if (a.S[t] != 0) {
                const int r = t / nab, b = t - r * nab;
                atomicOr(&bits[r * wpr + (b >> 5)], 1u << (b & 31));
            }
    }
    __syncthreads();
    {
        int mine = 0;
        for (int r = tid; r < T; r += 1024) {
            int deg = 0;
            for (int w = 0; w < wpr; ++w) deg += __popc(bits[r * wpr + w]);
            rl[r] = deg ? r : INF;               // a row with an edge starts from its own index
            mine += deg;
        }
        mine = __reduce_add_sync(0xffffffffu, mine);
        if (lane == 0 && mine) atomicAdd(&edges, (unsigned long long)mine);
    }
    __syncthreads();
    for (int sweep = 0; sweep <= T + nab; ++sweep) {
        int changed = 0;
        // blocks take the minimum over their rows: one warp per block, no atomics
        for (int b = warp; b < nab; b += 32) {
            const int w = b >> 5;
            const uint32_t bit = 1u << (b & 31);
            int m = INF;
            for (int r = lane; r < T; r += 32)
                if (bits[r * wpr + w] & bit) m = min(m, rl[r]);
            m = __reduce_min_sync(0xffffffffu, m);
            if (lane == 0 && m < bl[b]) { bl[b] = m; changed = 1; }
        }
        __syncthreads();
        // rows take the minimum over their blocks
        for (int r = tid; r < T; r += 1024) {
            const int mine = rl[r];
            if (mine == INF) continue;
            int m = mine;
            for (int w = 0; w < wpr; ++w)
                for (uint32_t v = bits[r * wpr + w]; v; v &= v - 1) m = min(m, bl[w * 32 + __ffs(v) - 1]);
            if (m < mine) { rl[r] = m; changed = 1; }
        }
        if (!__syncthreads_or(changed)) break;
    }
    {
        int comps = 0, live_r = 0, live_b = 0;
        for (int r = tid; r < T; r += 1024) {
            const int l = rl[r];
            if (l == INF) rl[r] = -1;
            else {
                ++live_r;
                comps += l == r;
            }
            a.row_label[r] = l == INF ? -1 : l;
        }
        for (int b = tid; b < nab; b += 1024) {
            const int l = bl[b];
            if (l == INF) bl[b] = -1;
            else ++live_b;
            a.blk_label[b] = l == INF ? -1 : l;
        }
        comps = __reduce_add_sync(0xffffffffu, comps);
        live_r = __reduce_add_sync(0xffffffffu, live_r);
        live_b = __reduce_add_sync(0xffffffffu, live_b);
        if (lane == 0) {
            if (comps) atomicAdd(&counts[0], comps);
            if (live_r) atomicAdd(&counts[1], live_r);
            if (live_b) atomicAdd(&counts[2], live_b);
        }
    }
    __syncthreads();
    if (tid == 0) {
        a.report[0] = (long long)edges;
        a.report[1] = counts[0];
        a.report[2] = counts[1];
        a.report[3] = counts[2];
        if (!a.plan) __threadfence_system();
    }
    if (!a.plan) return;

    // ---- component-sorted order
    const int M = counts[1], NB = counts[2], groups = a.groups, bs = a.bs;
    // rank of a row = number of rows with a smaller key label * T + row; rows of no component take T for the
    // label and so come last, in index order.  T <= 32768 keeps the key within 32 bits.
    unsigned long long my_pairs = 0;
    for (int r = tid; r < T; r += 1024) {
        const int l = rl[r];
        const unsigned key = (l >= 0 ? (unsigned)l : (unsigned)T) * (unsigned)T + (unsigned)r;
        int rank0 = 0, rank1 = 0;
        int q = 0;
        for (; q + 1 < T; q += 2) {
            const int l0 = rl[q], l1 = rl[q + 1];
            rank0 += (l0 >= 0 ? (unsigned)l0 : (unsigned)T) * (unsigned)T + (unsigned)q < key;
            rank1 += (l1 >= 0 ? (unsigned)l1 : (unsigned)T) * (unsigned)T + (unsigned)(q + 1) < key;
        }
        if (q < T) rank0 += (rl[q] >= 0 ? (unsigned)rl[q] : (unsigned)T) * (unsigned)T + (unsigned)q < key;
        a.row_map[rank0 + rank1] = r;
        if (l >= 0)
            for (int b = 0; b < nab; ++b) my_pairs += bl[b] == l;
    }
    my_pairs = __reduce_add_sync(0xffffffffu, (unsigned)my_pairs);
    if (lane == 0 && my_pairs) atomicAdd(&pairs, my_pairs);
    for (int b = tid; b < nab; b += 1024) {
        const int l = bl[b];
        if (l >= 0) {
            int less = 0, same = 0, before = 0;
            for (int q = 0; q < nab; ++q) {
                const int lq = bl[q];
                less += lq >= 0 && lq < l;
                same += lq == l;
                before += lq == l && q < b;
            }
            for (int g = 0; g < groups; ++g) {
                a.col_map[groups * less + g * same + before] = g * nab + b;
                sorted_bl[groups * less + g * same + before] = l;
            }
            a.kmap[less + before] = b;
        } else {
            int before = 0;
            for (int q = 0; q < b; ++q) before += bl[q] < 0;
            for (int g = 0; g < groups; ++g) {
                a.col_map[groups * NB + g * (nab - NB) + before] = g * nab + b;
                sorted_bl[groups * NB + g * (nab - NB) + before] = -1;
            }
            a.kmap[NB + before] = b;
        }
    }
    __syncthreads();

    // ---- the work of every row tile
    const int N = groups * NB * bs;
    const int mt = (M + TM - 1) / TM, nt = (N + TN - 1) / TN;
    if (tid < mt) {
        const int lo_m = rl[a.row_map[tid * TM]];
        const int hi_m = rl[a.row_map[min(tid * TM + TM, M) - 1]];
        int first = 0, count = 0;
        for (int tn = 0; tn < nt; ++tn) {
            const int lo_n = sorted_bl[(tn * TN) / bs];
            const int hi_n = sorted_bl[(min(tn * TN + TN, N) - 1) / bs];
            if (hi_n >= lo_m && lo_n <= hi_m) {
                if (count == 0) first = tn;
                ++count;
            }
        }
        a.up[tid].tn0 = first;
        a.up[tid].ntn = count;
        a.up[tid].klo = 0;
        a.up[tid].kcnt = a.kb_up;
        units_up[tid] = count * 2 * a.kb_up;
        int blk_begin = 0, blk_end = 0;          // sorted block positions of the components lo_m .. hi_m
        for (int q = 0; q < nab; ++q) {
            const int lq = bl[q];
            blk_begin += lq >= 0 && lq < lo_m;
            blk_end += lq >= 0 && lq <= hi_m;
        }
        const int klo = (blk_begin * bs) / KC, khi = (blk_end * bs + KC - 1) / KC;
        a.dn[tid].tn0 = 0;
        a.dn[tid].ntn = a.nt_dn;
        a.dn[tid].klo = klo;
        a.dn[tid].kcnt = khi - klo;
        units_dn[tid] = a.nt_dn * 2 * (khi - klo);
    }
    __syncthreads();
    if (tid == 0) {
        int off_up = 0, off_dn = 0;
        for (int tm = 0; tm < mt; ++tm) {
            a.up[tm].unit0 = off_up;
            a.dn[tm].unit0 = off_dn;
            off_up += units_up[tm];
            off_dn += units_dn[tm];
        }
        a.report[4] = off_up;
        a.report[5] = (long long)pairs;
        a.report[6] = off_dn;
        __threadfence_system();
    }
}

struct LimbArgs {
    const uint8_t* Epl[2];   // left planes of E = E_0 + E_1, per party: [m-tile][k-block][32 KiB]
    const uint8_t* Vpl[2];   // left planes of V_i = A_i + i*E
    const uint8_t* Bpl[2];   // right planes of B_i: [n-tile][k-block][16 KiB]
    const uint8_t* Fpl[2];   // right planes of F = F_0 + F_1
    u64* Z[2];               // [M, N], pre-loaded with C_i; partial sums are added with bulk reductions
    int M, N;                // N a multiple of 16
    int mt, nt, kb;          // tiles and k-blocks per operand pair; one tile runs over 2*kb blocks
    int* error_flag;         // set to 1 if a bounded wait ran out
    int* error_host;         // the same report in mapped host memory, so that the host sees it without a copy
    // Only read by the grouped kernel (one multiplication per connected component): the planes hold the operands
    // in component-sorted order, M counts the rows that lie in a component (and N the columns, when col_map is
    // given), and every row tile runs over the column tiles and k-blocks its LimbGroupRow names.  kb stays the
    // number of k-blocks per plane tile in memory.  A finished row piece goes to row row_map[r] of Z, whose rows are
    // ldz words long, and the 16 columns from sorted column c on to compact columns
    // col_map[c / bs] * bs + c % bs.. (bs is a multiple of 16; col_map null: column c itself).
    int ldz, bs;
    int group_units;             // units per party: sum over row tiles of ntn * 2 * kcnt
    const LimbGroupRow* groups;  // [mt]
    const int32_t* row_map;      // [M] sorted row -> row of Z
    const int32_t* col_map;      // [N / bs] sorted block -> compact block of Z, or null
};

// Slow path of a bounded wait, kept out of line so that the polling loops of the three roles stay short.
__device__ __noinline__ bool limb_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 128; ++i)
            if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limb::WAIT_CYCLES) {
            *abort_flag = 1;
            return false;
        }
    }
}

// Bounded wait: false (and the CTA-wide abort flag raised) if the barrier did not flip in time or another
// role already gave up.
__device__ __forceinline__ bool limb_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    return limb_wait_slow(bar, parity, abort_flag);
}

// The epilogue warps' wait for a finished segment lasts tens of microseconds and involves 256 threads: one lane
// per warp polls, sleeping between polls so that the warp leaves the issue slots to whoever shares the SM (a
// co-resident memory-side CTA), and then every lane acquires the completed phase with one (succeeding) poll.
__device__ __noinline__ bool limb_wait_sleeping(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limb::WAIT_CYCLES) {
            *abort_flag = 1;
            return false;
        }
        __nanosleep(400);
    }
}

__device__ __forceinline__ bool limb_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = limb_wait_sleeping(bar, parity, abort_flag);
    ok = __shfl_sync(0xffffffffu, ok, 0);      // also reconverges the warp for the aligned TMEM loads
    if (ok) ok = limb_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}

// Z = sum_s 2^(8s) D_s mod 2^64 from the eight 32-bit accumulators of one output element: the terms with s <= 3 are
// 32 x 32 -> 64-bit multiply-adds by 2^(8s), the terms with s >= 4 only reach the high word (32-bit shifts and adds).
__device__ __forceinline__ u64 limb_recombine(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t d3, uint32_t d4,
                                              uint32_t d5, uint32_t d6, uint32_t d7) {
    u64 v = (u64)d0;
    v += (u64)d1 * (u64)(1u << 8);
    v += (u64)d2 * (u64)(1u << 16);
    v += (u64)d3 * (u64)(1u << 24);
    const uint32_t hi = (uint32_t)(v >> 32) + d4 + (d5 << 8) + (d6 << 16) + (d7 << 24);
    return ((u64)hi << 32) | (u64)(uint32_t)v;
}

// One contiguous piece of a CTA's share of the (party, tile, k-block) space: a run of k-blocks of one tile.
struct LimbSegment {
    int party, tm, tn;
    int kpos;        // first k-block, in [0, 2*kb): blocks [0,kb) pair E with B_i, [kb,2kb) pair V_i with F
    int count;       // k-blocks in this segment, <= MAX_SEGMENT_UNITS
    int kb, klo;     // grouped kernel only: k-blocks per operand pair of this tile and the first of them
};

template <bool GROUPED = false>
__device__ __forceinline__ LimbSegment limb_segment(const LimbArgs& a, long long u, long long u_end) {
    LimbSegment s;
    long long seg_end;
    if (GROUPED) {
        s.party = (int)(u / a.group_units);
        const int ul = (int)(u - (long long)s.party * a.group_units);
        int tm = 0;
        while (tm + 1 < a.mt && __ldg(&a.groups[tm + 1].unit0) <= ul) ++tm;     // row tiles without work are passed over
        const int unit0 = __ldg(&a.groups[tm].unit0);
        s.kb = __ldg(&a.groups[tm].kcnt);
        s.klo = __ldg(&a.groups[tm].klo);
        const int tile_units = 2 * s.kb, r = ul - unit0, ti = r / tile_units;
        s.tm = tm;
        s.tn = __ldg(&a.groups[tm].tn0) + ti;
        s.kpos = r - ti * tile_units;
        seg_end = u - s.kpos + tile_units;
    } else {
        const long long tile_units = 2ll * a.kb;
        const long long tile = u / tile_units;
        seg_end = (tile + 1) * tile_units;
        const int per_party = a.mt * a.nt;
        s.party = (int)(tile / per_party);
        const int t2 = (int)(tile - (long long)s.party * per_party);
        s.tm = t2 / a.nt;
        s.tn = t2 - s.tm * a.nt;
        s.kpos = (int)(u - tile * tile_units);
        s.kb = a.kb;
        s.klo = 0;
    }
    if (seg_end > u_end) seg_end = u_end;
    if (seg_end > u + limb::MAX_SEGMENT_UNITS) seg_end = u + limb::MAX_SEGMENT_UNITS;
    s.count = (int)(seg_end - u);
    return s;
}

// Low / high word of a shared-memory matrix descriptor, K-major, no swizzle: bits 0-13 address>>4, 16-29 leading
// byte offset>>4 (between the two 16-byte K halves), 32-45 stride byte offset>>4 (between 8-row groups), 46-47
// descriptor version 1.
__device__ __forceinline__ uint32_t limb_desc_lo(uint32_t addr) {
    return ((addr & 0x3FFFFu) >> 4) | ((uint32_t)(limb::LBO_BYTES >> 4) << 16);
}
constexpr uint32_t LIMB_DESC_HI = (uint32_t)(limb::SBO_BYTES >> 4) | (1u << 14);

template <bool GROUPED>
__device__ __forceinline__ void combine_limb_body(const LimbArgs a) {
    using namespace limb;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES];
    __shared__ __align__(8) uint64_t empty_bar[STAGES];
    __shared__ __align__(8) uint64_t accum_full_bar, accum_empty_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    uint8_t* sA = smem;
    uint8_t* sB = smem + (size_t)STAGES * A_BLOCK_BYTES;
    uint8_t* sOut = sB + (size_t)STAGES * B_BLOCK_BYTES;      // EPI_WARPS x 32 rows x OUT_ROW_BYTES

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total_units = GROUPED ? 2ll * a.group_units : 2ll * a.mt * a.nt * 2ll * a.kb;
    const long long u_begin = total_units * blockIdx.x / gridDim.x;
    const long long u_end = total_units * (blockIdx.x + 1) / gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&accum_full_bar), 1);
        ptx::mbar_init(ptx::smem_u32(&accum_empty_bar), 32 * EPI_WARPS);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_before_sync();
    __syncthreads();
    ptx::fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    // barriers and tensor memory are set up; from here on the kernel touches what its predecessors wrote
    pdl_wait();

    if (warp == EPI_WARPS) {
        // ---------------- producer: one bulk copy per operand block ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            const uint32_t full0 = ptx::smem_u32(&full_bar[0]), empty0 = ptx::smem_u32(&empty_bar[0]);
            const uint32_t sA0 = ptx::smem_u32(sA), sB0 = ptx::smem_u32(sB);
            for (long long u = u_begin; u < u_end && ok;) {
                const LimbSegment sg = limb_segment<GROUPED>(a, u, u_end);
                u += sg.count;
                int kpos = sg.kpos;
                const int kbe = GROUPED ? sg.kb : a.kb;       // k-blocks per operand pair of this tile
                const int klo = GROUPED ? sg.klo : 0;         // and where they start in the plane tile
                bool second = kpos >= kbe;
                if (second) kpos -= kbe;
                const uint8_t* left = (second ? (sg.party ? a.Vpl[1] : a.Vpl[0]) : (sg.party ? a.Epl[1] : a.Epl[0])) +
                                      ((size_t)sg.tm * a.kb + klo + kpos) * A_BLOCK_BYTES;
                const uint8_t* right = (second ? (sg.party ? a.Fpl[1] : a.Fpl[0]) : (sg.party ? a.Bpl[1] : a.Bpl[0])) +
                                       ((size_t)sg.tn * a.kb + klo + kpos) * B_BLOCK_BYTES;
                for (int it = 0; it < sg.count; ++it) {
                    ok = limb_wait(empty0 + 8 * stage, phase ^ 1u, &abort_flag);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * stage;
                    ptx::mbar_expect_tx(bar, A_BLOCK_BYTES + B_BLOCK_BYTES);
                    ptx::bulk_g2s(sA0 + stage * A_BLOCK_BYTES, left, A_BLOCK_BYTES, bar);
                    ptx::bulk_g2s(sB0 + stage * B_BLOCK_BYTES, right, B_BLOCK_BYTES, bar);
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    left += A_BLOCK_BYTES;
                    right += B_BLOCK_BYTES;
                    if (++kpos == kbe && !second) {
                        // the tile's first product (E with B_i) is done: go on with the second (V_i with F)
                        second = true;
                        kpos = 0;
                        left = (sg.party ? a.Vpl[1] : a.Vpl[0]) + ((size_t)sg.tm * a.kb + klo) * A_BLOCK_BYTES;
                        right = (sg.party ? a.Fpl[1] : a.Fpl[0]) + ((size_t)sg.tn * a.kb + klo) * B_BLOCK_BYTES;
                    }
                }
            }
            if (!ok) {
                // gave up: let the copies already in flight land before the CTA leaves
                const int back = issued < STAGES ? issued : STAGES;
                for (int j = 1; j <= back; ++j) {
                    int s = stage - j;
                    uint32_t ph = phase;
                    if (s < 0) { s += STAGES; ph ^= 1u; }
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&full_bar[s]), ph) && clock64() - t0 < 20000000ll) {}
                }
            }
        }
    } else if (warp == EPI_WARPS + 1) {
        // ---------------- MMA issuer: 12 instructions per k-block, as little else as possible ----------------
        if (lane == 0) {
            // instruction descriptor: s32 accumulate, u8 x u8, both K-major, M = 128, N filled in per instruction
            constexpr uint32_t IDESC = (2u << 4) | ((uint32_t)(BM >> 4) << 24);
            const uint32_t full0 = ptx::smem_u32(&full_bar[0]), empty0 = ptx::smem_u32(&empty_bar[0]);
            const uint32_t accum_full = ptx::smem_u32(&accum_full_bar), accum_empty = ptx::smem_u32(&accum_empty_bar);
            const uint32_t a_lo0 = limb_desc_lo(ptx::smem_u32(sA)), b_lo0 = limb_desc_lo(ptx::smem_u32(sB));
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (long long u = u_begin; u < u_end && ok;) {
                const LimbSegment sg = limb_segment<GROUPED>(a, u, u_end);
                u += sg.count;
                ok = limb_wait(accum_empty, acc_phase ^ 1u, &abort_flag);
                if (!ok) break;
                ptx::fence_after_sync();
                uint32_t acc = 0;                         // the segment's first block overwrites the accumulators
                for (int it = 0; it < sg.count; ++it) {
                    ok = limb_wait(full0 + 8 * stage, phase, &abort_flag);
                    if (!ok) break;
                    ptx::fence_after_sync();
                    const uint32_t a_lo = a_lo0 + stage * (A_BLOCK_BYTES >> 4);
                    const uint32_t b_lo = b_lo0 + stage * (B_BLOCK_BYTES >> 4);
                    const uint32_t b_lo_hi = b_lo + ((256 * KC) >> 4);         // right-operand rows 256.. (planes 4..7)
                    // Left plane p meets right planes 0..7-p, whose products land in accumulators D_p..D_7: one
                    // instruction of N = 64*(8-p), cut at 256.  When a plane issues two instructions the second
                    // takes the left operand from the collector instead of shared memory.
#pragma unroll
                    for (int i = 0; i < PLANES; ++i) {
                        // wide and narrow instructions alternate (plane 0, which overwrites every accumulator when a
                        // segment starts, stays first)
                        const int p = (i & 1) ? PLANES - 1 - (i >> 1) : (i >> 1);
                        const uint32_t ap = a_lo + ((p * BM * KC) >> 4);
                        const int n_total = BN * (PLANES - p);
                        const uint32_t acc_p = p == 0 ? acc : 1u;
                        if (n_total > 256) {
                            ptx::mma_i8_keep_a(tmem_base + BN * p, ap, LIMB_DESC_HI, b_lo, LIMB_DESC_HI,
                                               IDESC | ((uint32_t)(256 >> 3) << 17), acc_p);
                            ptx::mma_i8_reuse_a(tmem_base + BN * p + 256, ap, LIMB_DESC_HI, b_lo_hi, LIMB_DESC_HI,
                                                IDESC | ((uint32_t)((n_total - 256) >> 3) << 17), acc_p);
                        } else {
                            ptx::mma_i8(tmem_base + BN * p, ap, LIMB_DESC_HI, b_lo, LIMB_DESC_HI,
                                        IDESC | ((uint32_t)(n_total >> 3) << 17), acc_p);
                        }
                    }
                    ptx::mma_commit(empty0 + 8 * stage);    // frees the stage once the MMAs have read it
                    acc = 1u;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                ptx::mma_commit(accum_full);
                acc_phase ^= 1u;
            }
            // the main loop is over: the next kernel of the stream may be brought in beside the last drain
            pdl_launch_dependents();
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> recombine mod 2^64 -> release TMEM ->
        //                  stage the rows in shared memory -> one bulk add-reduction per row into Z ----------------
        uint32_t acc_phase = 0;
        bool ok = true;
        const int quarter = warp & 3, chalf = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + chalf * 32;
        uint8_t* my_row = sOut + ((size_t)warp * 32 + lane) * OUT_ROW_BYTES;
        const uint32_t my_row_s = ptx::smem_u32(my_row);
        for (long long u = u_begin; u < u_end && ok;) {
            const LimbSegment sg = limb_segment<GROUPED>(a, u, u_end);
            u += sg.count;
            ok = limb_wait_warp(ptx::smem_u32(&accum_full_bar), acc_phase, &abort_flag);
            if (!ok) break;
            ptx::fence_after_sync();
            const int row = sg.tm * BM + quarter * 32 + lane;
            const int col0 = sg.tn * BN + chalf * 32;
            u64* zrow;
            if (GROUPED)
                zrow = (sg.party ? a.Z[1] : a.Z[0]) + (size_t)(row < a.M ? __ldg(a.row_map + row) : 0) * a.ldz;
            else
                zrow = (sg.party ? a.Z[1] : a.Z[0]) + (size_t)row * a.N + col0;
#pragma unroll
            for (int h = 0; h < 32 / OUT_COLS; ++h) {          // this thread's 32 columns, OUT_COLS at a time
                u64 v[OUT_COLS];
#pragma unroll
                for (int c = 0; c < OUT_COLS / 8; ++c) {
                    uint32_t d[PLANES][8];
#pragma unroll
                    for (int s = 0; s < PLANES; ++s) ptx::tmem_ld8(lane_base + BN * s + h * OUT_COLS + c * 8, d[s]);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        v[c * 8 + j] = limb_recombine(d[0][j], d[1][j], d[2][j], d[3][j], d[4][j], d[5][j], d[6][j],
                                                      d[7][j]);
                }
                if (h == 32 / OUT_COLS - 1) {
                    // every accumulator has been read: hand TMEM back before anything that waits on the copy engine
                    ptx::fence_before_sync();
                    ptx::mbar_arrive(ptx::smem_u32(&accum_empty_bar));
                }
                ptx::bulk_wait_group_read0();                  // the previous reduction has read this thread's staging row
#pragma unroll
                for (int j = 0; j < OUT_COLS; j += 2)
                    *reinterpret_cast<ulonglong2*>(my_row + j * 8) = make_ulonglong2(v[j], v[j + 1]);
                int cols = a.N - col0 - h * OUT_COLS;
                if (cols > OUT_COLS) cols = OUT_COLS;
                if (row < a.M && cols > 0) {
                    ptx::fence_proxy_async_smem();     // this thread's row, written above, is read by the copy engine
                    u64* dst;
                    if (GROUPED) {
                        const int c = col0 + h * OUT_COLS, blk = c / a.bs;
                        dst = a.col_map ? zrow + (size_t)__ldg(a.col_map + blk) * a.bs + (c - blk * a.bs) : zrow + c;
                    } else {
                        dst = zrow + h * OUT_COLS;
                    }
                    ptx::bulk_reduce_add_u64(dst, my_row_s, (uint32_t)cols * 8u);
                }
                ptx::bulk_commit_group();
            }
            acc_phase ^= 1u;
        }
        ptx::bulk_wait_group0();                       // every reduction of this thread has completed
    }

    ptx::fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) {
        *a.error_flag = 1;
        *reinterpret_cast<volatile int*>(a.error_host) = 1;
        __threadfence_system();
    }
    if (warp == 0) {
        ptx::fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

__global__ void __launch_bounds__(limb::THREADS, 1)
combine_limb_kernel(LimbArgs a) {
    combine_limb_body<false>(a);
}

// One multiplication per connected component (Protocols 2 and 3 under a per-token mask): the same kernel over the
// tiles and k-blocks of the component-sorted operands that have work, scattering the result rows back to Z.
__global__ void __launch_bounds__(limb::THREADS, 1)
combine_limb_grouped_kernel(LimbArgs a) {
    combine_limb_body<true>(a);
}

// ---------------------------------------------------------------------------
// Few tokens (M <= 32, the decode step): the roles of the two operands are exchanged.  The weight-side operand
// (B_i, then F) supplies the 128 rows of the MMA, one limb plane per instruction, and the token-side operand
// (E, then V_i) is the one whose planes are stacked along N: 32 token rows per plane, so right plane q meets
// left planes 0..7-q in one instruction of N = 32*(8-q) <= 256, 8 instructions per 32-deep step, and the eight
// accumulators D_s (128 neurons x 32 tokens) take 256 TMEM columns.  A 128-row tile of the ordinary kernel would
// spend three quarters of its tensor work on padding rows here.  Every weight plane is used by exactly one tile,
// so the kernel streams them once; it is bound by that traffic, not by the tensor pipe.  That leaves tensor time
// to spare, which buys a pass over memory: the second product is taken as V_i*F_0 + V_i*F_1 over the planes of the
// two messages as the parties wrote them, so no kernel has to read both messages back, add them and write planes
// of the sum.  A tile thus runs over three operand pairs: (E, B_i), (V_i, F_0), (V_i, F_1).
// Plane layouts: token side [k-block][8 planes x 32 rows x 32 B] (8 KiB blocks), weight side
// [n-tile of 128][k-block][32 KiB].  The output tile Z^T (neurons x tokens) is transposed through shared memory
// so that each bulk reduction adds 32 consecutive neurons of one token row.
// ---------------------------------------------------------------------------
namespace limb_few {
constexpr int BW = 128, BT = 32, KC = limb::KC, PLANES = limb::PLANES;
constexpr int W_BLOCK_BYTES = PLANES * BW * KC;   // 32 KiB
constexpr int T_BLOCK_BYTES = PLANES * BT * KC;   // 8 KiB
constexpr int STAGES = 4;
constexpr int EPI_WARPS = 8;                      // warp w: neurons 32*(w%4).., tokens 16*(w/4)..
constexpr int THREADS = 32 * (EPI_WARPS + 2);
constexpr int OUT_BYTES_PER_WARP = 16 * 32 * 8;   // 16 token rows x 32 neurons
constexpr int TMEM_COLS = PLANES * BT;            // 256
constexpr size_t SMEM_BYTES = (size_t)STAGES * (W_BLOCK_BYTES + T_BLOCK_BYTES) + (size_t)EPI_WARPS * OUT_BYTES_PER_WARP + 128;
}  // namespace limb_few

// LimbArgs as for combine_limb_kernel with Epl/Vpl = token-side planes, Bpl = weight-side planes of the party's
// B_i, Fpl[0] / Fpl[1] = weight-side planes of the messages F_0 / F_1 (read by both parties), mt = 1,
// nt = ceil(N / 128), M <= 32.
constexpr int LIMB_FEW_PAIRS = 3;

// One contiguous piece of a CTA's share: a run of k-blocks of one tile, kpos in [0, 3*kb).
__device__ __forceinline__ LimbSegment limb_few_segment(const LimbArgs& a, long long u, long long u_end) {
    const long long tile_units = (long long)LIMB_FEW_PAIRS * a.kb;
    const long long tile = u / tile_units;
    long long seg_end = (tile + 1) * tile_units;
    if (seg_end > u_end) seg_end = u_end;
    if (seg_end > u + limb::MAX_SEGMENT_UNITS) seg_end = u + limb::MAX_SEGMENT_UNITS;
    const int per_party = a.mt * a.nt;
    LimbSegment s;
    s.party = (int)(tile / per_party);
    const int t2 = (int)(tile - (long long)s.party * per_party);
    s.tm = t2 / a.nt;
    s.tn = t2 - s.tm * a.nt;
    s.kpos = (int)(u - tile * tile_units);
    s.count = (int)(seg_end - u);
    s.kb = a.kb;
    s.klo = 0;
    return s;
}

__global__ void __launch_bounds__(limb_few::THREADS, 1)
combine_limb_few_kernel(LimbArgs a) {
    using namespace limb_few;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[STAGES];
    __shared__ __align__(8) uint64_t empty_bar[STAGES];
    __shared__ __align__(8) uint64_t accum_full_bar, accum_empty_bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    uint8_t* sW = smem;
    uint8_t* sT = smem + (size_t)STAGES * W_BLOCK_BYTES;
    uint8_t* sOut = sT + (size_t)STAGES * T_BLOCK_BYTES;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total_units = 2ll * a.mt * a.nt * LIMB_FEW_PAIRS * a.kb;
    const long long u_begin = total_units * blockIdx.x / gridDim.x;
    const long long u_end = total_units * (blockIdx.x + 1) / gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&full_bar[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&empty_bar[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&accum_full_bar), 1);
        ptx::mbar_init(ptx::smem_u32(&accum_empty_bar), 32 * EPI_WARPS);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_slot), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::fence_before_sync();
    __syncthreads();
    ptx::fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    // barriers and tensor memory are set up; from here on the kernel touches what its predecessors wrote
    pdl_wait();

    if (warp == EPI_WARPS) {
        // ---------------- producer: one bulk copy per operand block ----------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            bool ok = true;
            const uint32_t full0 = ptx::smem_u32(&full_bar[0]), empty0 = ptx::smem_u32(&empty_bar[0]);
            const uint32_t sW0 = ptx::smem_u32(sW), sT0 = ptx::smem_u32(sT);
            for (long long u = u_begin; u < u_end && ok;) {
                const LimbSegment sg = limb_few_segment(a, u, u_end);
                u += sg.count;
                int pair = sg.kpos / a.kb;                    // 0: (E, B_i), 1: (V_i, F_0), 2: (V_i, F_1)
                int kpos = sg.kpos - pair * a.kb;
                const uint8_t* tok_e = sg.party ? a.Epl[1] : a.Epl[0];
                const uint8_t* tok_v = sg.party ? a.Vpl[1] : a.Vpl[0];
                const size_t tile_off = (size_t)sg.tn * a.kb * W_BLOCK_BYTES;
                const uint8_t* wgt_b = (sg.party ? a.Bpl[1] : a.Bpl[0]) + tile_off;
                const uint8_t* tok = (pair == 0 ? tok_e : tok_v) + (size_t)kpos * T_BLOCK_BYTES;
                const uint8_t* wgt = (pair == 0 ? wgt_b : (pair == 1 ? a.Fpl[0] : a.Fpl[1]) + tile_off) +
                                     (size_t)kpos * W_BLOCK_BYTES;
                for (int it = 0; it < sg.count; ++it) {
                    ok = limb_wait(empty0 + 8 * stage, phase ^ 1u, &abort_flag);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * stage;
                    ptx::mbar_expect_tx(bar, W_BLOCK_BYTES + T_BLOCK_BYTES);
                    ptx::bulk_g2s(sW0 + stage * W_BLOCK_BYTES, wgt, W_BLOCK_BYTES, bar);
                    ptx::bulk_g2s(sT0 + stage * T_BLOCK_BYTES, tok, T_BLOCK_BYTES, bar);
                    ++issued;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    tok += T_BLOCK_BYTES;
                    wgt += W_BLOCK_BYTES;
                    if (++kpos == a.kb && pair < LIMB_FEW_PAIRS - 1) {
                        ++pair;                               // on to V_i with the next message
                        kpos = 0;
                        tok = tok_v;
                        wgt = (pair == 1 ? a.Fpl[0] : a.Fpl[1]) + tile_off;
                    }
                }
            }
            if (!ok) {
                const int back = issued < STAGES ? issued : STAGES;
                for (int j = 1; j <= back; ++j) {
                    int s = stage - j;
                    uint32_t ph = phase;
                    if (s < 0) { s += STAGES; ph ^= 1u; }
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&full_bar[s]), ph) && clock64() - t0 < 20000000ll) {}
                }
            }
        }
    } else if (warp == EPI_WARPS + 1) {
        // ---------------- MMA issuer: weight plane q against token planes 0..7-q ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC = (2u << 4) | ((uint32_t)(BW >> 4) << 24);
            const uint32_t full0 = ptx::smem_u32(&full_bar[0]), empty0 = ptx::smem_u32(&empty_bar[0]);
            const uint32_t accum_full = ptx::smem_u32(&accum_full_bar), accum_empty = ptx::smem_u32(&accum_empty_bar);
            const uint32_t w_lo0 = limb_desc_lo(ptx::smem_u32(sW)), t_lo0 = limb_desc_lo(ptx::smem_u32(sT));
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (long long u = u_begin; u < u_end && ok;) {
                const LimbSegment sg = limb_few_segment(a, u, u_end);
                u += sg.count;
                ok = limb_wait(accum_empty, acc_phase ^ 1u, &abort_flag);
                if (!ok) break;
                ptx::fence_after_sync();
                uint32_t acc = 0;
                for (int it = 0; it < sg.count; ++it) {
                    ok = limb_wait(full0 + 8 * stage, phase, &abort_flag);
                    if (!ok) break;
                    ptx::fence_after_sync();
                    const uint32_t w_lo = w_lo0 + stage * (W_BLOCK_BYTES >> 4);
                    const uint32_t t_lo = t_lo0 + stage * (T_BLOCK_BYTES >> 4);
#pragma unroll
                    for (int q = 0; q < PLANES; ++q)
                        ptx::mma_i8(tmem_base + BT * q, w_lo + ((q * BW * KC) >> 4), LIMB_DESC_HI, t_lo, LIMB_DESC_HI,
                                    IDESC | ((uint32_t)((BT * (PLANES - q)) >> 3) << 17), q == 0 ? acc : 1u);
                    ptx::mma_commit(empty0 + 8 * stage);
                    acc = 1u;
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                ptx::mma_commit(accum_full);
                acc_phase ^= 1u;
            }
            // the main loop is over: the next kernel of the stream may be brought in beside the last drain
            pdl_launch_dependents();
        }
    } else {
        // ---------------- epilogue: lane = neuron, registers = tokens; transpose through shared memory ----------------
        uint32_t acc_phase = 0;
        bool ok = true;
        const int quarter = warp & 3, thalf = warp >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + thalf * 16;
        u64* stage_out = reinterpret_cast<u64*>(sOut + (size_t)warp * OUT_BYTES_PER_WARP);   // [16 tokens][32 neurons]
        for (long long u = u_begin; u < u_end && ok;) {
            const LimbSegment sg = limb_few_segment(a, u, u_end);
            u += sg.count;
            ok = limb_wait_warp(ptx::smem_u32(&accum_full_bar), acc_phase, &abort_flag);
            if (!ok) break;
            ptx::fence_after_sync();
            u64 z[16];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t d[PLANES][8];
#pragma unroll
                for (int s = 0; s < PLANES; ++s) ptx::tmem_ld8(lane_base + BT * s + c * 8, d[s]);
                ptx::tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    z[c * 8 + j] = limb_recombine(d[0][j], d[1][j], d[2][j], d[3][j], d[4][j], d[5][j], d[6][j], d[7][j]);
            }
            ptx::fence_before_sync();
            ptx::mbar_arrive(ptx::smem_u32(&accum_empty_bar));
            if (lane < 16) ptx::bulk_wait_group_read0();       // this lane's previous reduction has read its row
            __syncwarp();
#pragma unroll
            for (int t = 0; t < 16; ++t) stage_out[t * 32 + lane] = z[t];
            ptx::fence_proxy_async_smem();
            __syncwarp();
            const int token = thalf * 16 + lane;               // lanes 0..15 each own one token row of the piece
            const int col0 = sg.tn * BW + quarter * 32;
            int cols = a.N - col0;
            if (cols > 32) cols = 32;
            if (lane < 16) {
                if (token < a.M && cols > 0)
                    ptx::bulk_reduce_add_u64((sg.party ? a.Z[1] : a.Z[0]) + (size_t)token * a.N + col0,
                                             ptx::smem_u32(stage_out + lane * 32), (uint32_t)cols * 8u);
                ptx::bulk_commit_group();
            }
            acc_phase ^= 1u;
        }
        if (lane < 16) ptx::bulk_wait_group0();
    }

    ptx::fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) {
        *a.error_flag = 1;
        *reinterpret_cast<volatile int*>(a.error_host) = 1;
        __threadfence_system();
    }
    if (warp == 0) {
        ptx::fence_after_sync();
        ptx::tmem_dealloc(tmem_base, limb_few::TMEM_COLS);
    }
}

}  // namespace comet
