// C ABI of the library: context, host-side validation and kernel launches.
// Every argument is checked on the host before anything is enqueued; device
// code never traps.  See include/comet.h for the contract of each call.
#include "../../include/comet.h"

#include <chrono>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include <cuda_runtime.h>

#include "kernels_limb.cuh"
#include "kernels_mul.cuh"
#include "kernels_open.cuh"
#include "kernels_peak.cuh"
#include "kernels_shuffle.cuh"
#include "kernels_simt.cuh"

using comet::u64;

struct comet_ctx {
    comet_config cfg;
    cudaStream_t stream;
    int groups;                   // 1, 2 or 3 weight matrices stacked in the up-projection
    int64_t cap_T, cap_n;         // capacities
    int sm_count;
    u64* buf[2][COMET_NUM_TENSORS];   // where each tensor is read / written: the library's own buffer, or a bound one
    u64* own[2][COMET_NUM_TENSORS];   // the library's own buffers (allocated in comet_init, freed in comet_destroy)
    int64_t cap_words[COMET_NUM_TENSORS];
    bool loaded[2][COMET_NUM_TENSORS];
    // limb path: blocked limb planes per party (left: E and V_i; right: B_i and F), and the device error flag
    int path;                     // COMET_PATH_SIMT or COMET_PATH_LIMB
    uint8_t* planes_left[2][2];       // [party][E, V_i]; shared by the two projections
    uint8_t* planes_right_up[2][2];   // [party][B_i, F] of the up-projection
    uint8_t* planes_right_dn[2][2];   // [party][B'_i, F'] of the down-projection
    size_t planes_left_bytes, planes_right_up_bytes, planes_right_dn_bytes;
    int* d_error;                     // = d_count + 1
    // the weight side of the down-projection is opened on a second stream while the up-projection's
    // tensor-core kernel runs (it only needs the mask, W2 and B'_i)
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;
    bool side_pending;                // ev_join not yet waited for on the main stream
    bool dn_right_ready;              // F'_i and the right planes of the down-projection are current
    bool dn_right_few;                // ... and were laid out for the few-token kernel (128-row tiles)
    bool dn_copy_ready;               // Y_i already holds C'_i (copied beside the up-projection)
    int32_t dn_copy_tokens;           // ... for this many token rows
    bool f_as_planes[2];              // the messages F_i of the last up / down product exist as planes only
    uint8_t* d_mask;
    // a block mask given in host memory is counted on the host and copied from a pinned staging slot of the
    // library's own, so that comet_set_mask need not wait for the device
    uint8_t* h_mask_stage;            // pinned: kMaskSlots x n_blocks bytes
    cudaEvent_t stage_done[4];        // recorded after the copy out of each slot
    bool stage_used[4];
    int stage_next;
    uint8_t* d_tmask;             // per-token mask over the active blocks, [cap_T, d_ff / block] capacity
    bool tmask_set;
    int32_t tmask_tokens;
    int64_t tmask_masked;         // non-zero entries of the hidden state under the token mask (neurons, not blocks)
    long long* h_masked;          // pinned and mapped: token_plan_kernel's report [0..6]
    uint32_t* d_plan_scratch;     // its working storage when that does not fit into shared memory
    long long* h_masked_dev;
    int32_t* d_row_label;         // component label per token row / per active block under the token mask
    int32_t* d_blk_label;
    int32_t n_components, live_rows, live_blocks;
    // one multiplication per component on the tensor-core path: component-sorted order and the tiles with work
    int32_t* d_row_map;
    int32_t* d_col_map;
    int32_t* d_kmap;
    comet::LimbGroupRow* d_group_up;
    comet::LimbGroupRow* d_group_dn;
    bool grouped;                 // the products under the current token mask run over the component rectangles only
    int32_t group_units_up, group_units_dn;   // k-block units per party of the two grouped launches
    int64_t component_pairs;      // sum over components of token rows x active blocks
    int32_t* d_ids;
    int32_t* d_count;             // {count, error flag of the bounded waits}
    int32_t* h_count;             // pinned and mapped: {count, error flag as the compaction kernel saw it, ticket,
                                  // error word written by a kernel whose bounded wait ran out}
    int32_t* h_count_dev;         // device-side address of h_count
    int top_priority;             // the device's highest stream / launch priority (numerically lowest)
    int32_t ticket;               // sequence number of the last compaction launch (echoed in h_count[2])
    bool mask_set;
    int32_t n_active, n_active_blocks;
    int32_t tokens;               // T fixed by the last load of X / A_UP / H
    bool up_done, down_done;
    int32_t up_tokens, down_tokens;
    comet_stats_t stats;
    int last_cuda_error;
    // per-phase timers: pairs of events recorded around each phase while profiling is on
    bool profiling;
    struct Pending { cudaEvent_t start, stop; int phase, launches; };
    std::vector<Pending>* pending;
    std::vector<cudaEvent_t>* free_events;
};

namespace {

#define COMET_CUDA(ctx, call)                                  \
    do {                                                       \
        cudaError_t err__ = (call);                            \
        if (err__ != cudaSuccess) {                            \
            (ctx)->last_cuda_error = (int)err__;               \
            return COMET_ERR_CUDA;                             \
        }                                                      \
    } while (0)

// Brackets the launches of one phase with two events when profiling is on.
struct PhaseTimer {
    comet_ctx* c;
    comet_ctx::Pending p;
    bool on;
    static cudaEvent_t take(comet_ctx* c) {
        if (!c->free_events->empty()) {
            cudaEvent_t e = c->free_events->back();
            c->free_events->pop_back();
            return e;
        }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    PhaseTimer(comet_ctx* ctx, int phase, int launches) : c(ctx), on(ctx->profiling) {
        if (!on) return;
        p.phase = phase;
        p.launches = launches;
        p.start = take(c);
        p.stop = take(c);
        cudaEventRecord(p.start, c->stream);
    }
    ~PhaseTimer() {
        if (!on) return;
        cudaEventRecord(p.stop, c->stream);
        c->pending->push_back(p);
    }
};

inline int is_input(int id) { return (id >= COMET_X && id <= COMET_C_DN) || id == COMET_W3; }

// current shape of a tensor as stored; rows = cols = 0 when not defined yet
void tensor_shape(const comet_ctx* c, int id, int64_t T, int64_t* rows, int64_t* cols) {
    const int64_t d = c->cfg.d_model, D = c->cfg.d_ff, n = c->n_active, gn = (int64_t)c->groups * n;
    switch (id) {
        case COMET_X: case COMET_A_UP: case COMET_E_UP: case COMET_C_DN: case COMET_Y: *rows = T; *cols = d; break;
        case COMET_W1: case COMET_WG: case COMET_W3: *rows = D; *cols = d; break;
        case COMET_W2: *rows = d; *cols = D; break;
        case COMET_B_UP: case COMET_F_UP: *rows = gn; *cols = d; break;
        case COMET_C_UP: case COMET_Z_UP: *rows = T; *cols = gn; break;
        case COMET_H: case COMET_A_DN: case COMET_E_DN: *rows = T; *cols = n; break;
        case COMET_B_DN: case COMET_F_DN: *rows = d; *cols = n; break;
        default: *rows = 0; *cols = 0;
    }
}

int64_t tensor_capacity(const comet_ctx* c, int id) {
    const int64_t d = c->cfg.d_model, D = c->cfg.d_ff, T = c->cap_T, n = c->cap_n, gn = c->groups * n;
    switch (id) {
        case COMET_X: case COMET_A_UP: case COMET_E_UP: case COMET_C_DN: case COMET_Y: return T * d;
        case COMET_W1: return D * d;
        case COMET_WG: return c->groups >= 2 ? D * d : 0;
        case COMET_W3: return c->groups == 3 ? D * d : 0;
        case COMET_W2: return d * D;
        case COMET_B_UP: case COMET_F_UP: return gn * d;
        case COMET_C_UP: case COMET_Z_UP: return T * gn;
        case COMET_H: case COMET_A_DN: case COMET_E_DN: return T * n;
        case COMET_B_DN: case COMET_F_DN: return d * n;
        default: return 0;
    }
}

inline int ew_grid(const comet_ctx* c, int64_t items, int threads) {
    int64_t want = (items + threads - 1) / threads;
    int64_t cap = (int64_t)c->sm_count * 8;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}

cudaMemcpyKind copy_kind(int location, bool to_library) {
    if (location == COMET_DEVICE) return cudaMemcpyDeviceToDevice;
    return to_library ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Launch of a kernel of the step's chain: programmatic stream serialisation (the kernel may begin while its
// predecessor on the stream is finishing; it calls pdl_wait() before it touches global memory) and, for the
// tensor-core kernels, the device's highest scheduling priority.
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                           const int* priority, Args&&... args) {
    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof(lc));
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.numAttrs = 1;
    if (priority) {
        attr[1].id = cudaLaunchAttributePriority;
        attr[1].val.priority = *priority;
        lc.numAttrs = 2;
    }
    lc.attrs = attr;
    return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}

// True once a kernel of this context gave up on a bounded wait (the word is written by the kernel itself, in
// mapped host memory, and never cleared: the context's results are not to be trusted from then on).
inline bool timed_out(const comet_ctx* c) {
    return *reinterpret_cast<volatile int32_t*>(c->h_count + 3) != 0 ||
           *reinterpret_cast<volatile int32_t*>(c->h_count + 1) != 0;
}

// One Pi_MatMul of the path: sizes and tensor ids.
struct Proj {
    int M, N, K;
    int idX, idA, idE, idB, idF, idC, idZ;
    bool down;
};

Proj proj_up(const comet_ctx* c, int tokens) {
    return Proj{tokens, c->groups * c->n_active, c->cfg.d_model, COMET_X, COMET_A_UP, COMET_E_UP, COMET_B_UP,
                COMET_F_UP, COMET_C_UP, COMET_Z_UP, false};
}
Proj proj_down(const comet_ctx* c, int tokens) {
    return Proj{tokens, c->cfg.d_model, c->n_active, COMET_H, COMET_A_DN, COMET_E_DN, COMET_B_DN, COMET_F_DN,
                COMET_C_DN, COMET_Y, true};
}

// The few-token kernel (operand roles exchanged) serves products with at most 32 token rows.
inline bool limb_few(const Proj& pr) { return pr.M <= comet::limb_few::BT; }

// Makes the main stream wait for the side stream's outstanding work (if any).
int join_side(comet_ctx* c) {
    if (c->side_pending) {
        COMET_CUDA(c, cudaStreamWaitEvent(c->stream, c->ev_join, 0));
        c->side_pending = false;
    }
    return COMET_OK;
}

// Tensor-core path, before the exchange: E_i (left) and/or F_i + planes(B_i) (right), one launch.
int limb_open(comet_ctx* c, const Proj& pr, bool left, bool right, cudaStream_t stream) {
    namespace lb = comet::limb;
    comet::LimbOpenArgs a;
    std::memset(&a, 0, sizeof(a));
    const int kb = ceil_div(pr.K, lb::KC);
    uint8_t* (*planes)[2] = pr.down ? c->planes_right_dn : c->planes_right_up;
    for (int p = 0; p < 2; ++p) {
        a.X[p] = c->buf[p][pr.idX];
        a.A[p] = c->buf[p][pr.idA];
        a.E[p] = c->buf[p][pr.idE];
        a.W0[p] = pr.down ? c->buf[p][COMET_W2] : (c->groups >= 2 ? c->buf[p][COMET_WG] : c->buf[p][COMET_W1]);
        a.W1[p] = c->buf[p][COMET_W1];
        a.W2g[p] = c->buf[p][COMET_W3];
        a.B[p] = c->buf[p][pr.idB];
        a.F[p] = c->buf[p][pr.idF];
        a.Bpl[p] = planes[p][0];
        a.Fpl[p] = planes[p][1];
    }
    a.emit_f = limb_few(pr) ? 1 : 0;       // few-token products read the messages as planes (no plane of their sum)
    a.left_pairs = left ? (long long)pr.M * pr.K / 2 : 0;
    a.left_blocks = left ? ew_grid(c, a.left_pairs, lb::OPEN_THREADS) : 0;
    a.ids = c->d_ids;
    a.n = c->n_active;
    a.bs = c->cfg.block;
    a.rows = pr.N;
    a.K = pr.K;
    a.ldw = pr.down ? c->cfg.d_ff : c->cfg.d_model;
    a.kblocks = kb;
    a.down = pr.down ? 1 : 0;
    a.right_tile_rows = limb_few(pr) ? comet::limb_few::BW : lb::BN;
    a.tmask = (pr.down && c->tmask_set) ? c->d_tmask : nullptr;
    a.tmask_ld = c->n_active_blocks;
    a.row_label = (!pr.down && c->tmask_set) ? c->d_row_label : nullptr;
    a.blk_label = c->tmask_set ? c->d_blk_label : nullptr;
    a.col_map = (!pr.down && c->grouped) ? c->d_col_map : nullptr;
    a.kmap = (pr.down && c->grouped) ? c->d_kmap : nullptr;
    // right CTAs: 32 rows x kb_per_cta k-blocks each, over whole plane tiles (rows past the operand are zero planes);
    // enough k-blocks per CTA for the copies of one to fly under the work on another, enough CTAs to fill the device
    const int row_tiles = right ? ceil_div(pr.N, a.right_tile_rows) * (a.right_tile_rows / lb::OPEN_ROWS) : 0;
    {
        const long long fill = (long long)c->sm_count * 6;
        long long per = fill > 0 ? 2ll * row_tiles * kb / fill : 1;
        if (per < 1) per = 1;
        if (per > lb::OPEN_MAX_KB_PER_CTA) per = lb::OPEN_MAX_KB_PER_CTA;
        a.kb_per_cta = (int)per;
        a.kchunks = ceil_div(kb, a.kb_per_cta);
    }
    const int right_tiles = row_tiles * a.kchunks;
    if (a.left_blocks + right_tiles == 0) return COMET_OK;
    if (right_tiles) c->f_as_planes[pr.down ? 1 : 0] = a.emit_f != 0;
    const size_t smem = right_tiles ? lb::OPEN_SMEM_BYTES : 0;
    COMET_CUDA(c, launch_chained(comet::limb_open_kernel, dim3(2 * (a.left_blocks + right_tiles)),
                                 dim3(lb::OPEN_THREADS), smem, stream, nullptr, a));
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

// Tensor-core path, after the exchange: planes(E), planes(V_i) (left), planes(F) (right), Z <- C, one launch.
int limb_prep(comet_ctx* c, const Proj& pr, bool left, bool right, bool copy, cudaStream_t stream) {
    namespace lb = comet::limb;
    comet::LimbPrepArgs a;
    std::memset(&a, 0, sizeof(a));
    const int kb = ceil_div(pr.K, lb::KC);
    uint8_t* (*planes)[2] = pr.down ? c->planes_right_dn : c->planes_right_up;
    a.E0 = c->buf[0][pr.idE]; a.E1 = c->buf[1][pr.idE];
    a.F0 = c->buf[0][pr.idF]; a.F1 = c->buf[1][pr.idF];
    for (int p = 0; p < 2; ++p) {
        a.A[p] = c->buf[p][pr.idA];
        a.Epl[p] = c->planes_left[p][0];
        a.Vpl[p] = c->planes_left[p][1];
        a.Fpl[p] = planes[p][1];
        a.C[p] = c->buf[p][pr.idC];
        a.Z[p] = c->buf[p][pr.idZ];
    }
    a.M = pr.M; a.N = pr.N; a.K = pr.K; a.kblocks = kb;
    if (c->grouped) {                       // component-sorted planes of the rows and columns that lie in a component
        a.M = c->live_rows;
        a.row_map = c->d_row_map;
        if (pr.down) {
            a.kmap = c->d_kmap;
        } else {
            a.N = c->groups * c->live_blocks * c->cfg.block;
            a.col_map = c->d_col_map;
        }
    }
    a.left_tile_rows = limb_few(pr) ? comet::limb_few::BT : lb::BM;
    a.right_tile_rows = limb_few(pr) ? comet::limb_few::BW : lb::BN;
    a.tmask = (pr.down && c->tmask_set) ? c->d_tmask : nullptr;
    a.tmask_ld = c->n_active_blocks;
    a.bs = c->cfg.block;
    // tile CTAs: 32 rows x kb_per_cta k-blocks each, over whole plane tiles (rows past the operand are zero planes)
    const int left_rows32 = left ? ceil_div(a.M, a.left_tile_rows) * (a.left_tile_rows / lb::OPEN_ROWS) : 0;
    // few-token products take the planes of the two messages as limb_open_kernel wrote them
    const int right_rows32 = (right && !limb_few(pr))
                                 ? ceil_div(a.N, a.right_tile_rows) * (a.right_tile_rows / lb::OPEN_ROWS) : 0;
    {
        const long long fill = (long long)c->sm_count * 4;
        long long per = fill > 0 ? 2ll * (left_rows32 + right_rows32) * kb / fill : 1;
        if (per < 1) per = 1;
        if (per > lb::OPEN_MAX_KB_PER_CTA) per = lb::OPEN_MAX_KB_PER_CTA;
        a.kb_per_cta = (int)per;
        a.kchunks = ceil_div(kb, a.kb_per_cta);
    }
    a.left_tiles = left_rows32 * a.kchunks;
    a.right_tiles = right_rows32 * a.kchunks;
    a.copy_pairs = copy ? (long long)pr.M * pr.N / 2 : 0;
    a.copy_blocks = copy ? ew_grid(c, a.copy_pairs, lb::OPEN_THREADS) : 0;
    const int blocks = a.left_tiles + a.right_tiles + a.copy_blocks;
    if (blocks == 0) return COMET_OK;
    const size_t smem = (size_t)lb::OPEN_STAGES * (left ? 3 : 2) * lb::OPEN_TILE_BYTES;
    COMET_CUDA(c, launch_chained(comet::limb_prep_kernel, dim3(2 * blocks), dim3(lb::OPEN_THREADS), smem, stream,
                                 nullptr, a));
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

// Tensor-core path: the persistent stream-K kernel over both parties' tiles (the few-token variant when the
// product has at most 32 token rows).
int limb_combine(comet_ctx* c, const Proj& pr) {
    namespace lb = comet::limb;
    namespace lf = comet::limb_few;
    const bool few = limb_few(pr);
    const int kb = ceil_div(pr.K, lb::KC);
    const int mt = few ? 1 : ceil_div(pr.M, lb::BM), nt = few ? ceil_div(pr.N, lf::BW) : ceil_div(pr.N, lb::BN);
    uint8_t* (*planes)[2] = pr.down ? c->planes_right_dn : c->planes_right_up;
    comet::LimbArgs a;
    for (int p = 0; p < 2; ++p) {
        a.Epl[p] = c->planes_left[p][0];
        a.Vpl[p] = c->planes_left[p][1];
        a.Bpl[p] = planes[p][0];
        a.Fpl[p] = planes[p][1];
        a.Z[p] = c->buf[p][pr.idZ];
    }
    a.M = pr.M; a.N = pr.N; a.mt = mt; a.nt = nt; a.kb = kb;
    a.error_flag = c->d_error;
    a.error_host = c->h_count_dev + 3;
    a.ldz = pr.N; a.bs = c->cfg.block; a.group_units = 0;
    a.groups = nullptr; a.row_map = nullptr; a.col_map = nullptr;
    const bool grouped = c->grouped && !few;
    if (grouped) {
        a.M = c->live_rows;
        a.mt = ceil_div(a.M, lb::BM);
        a.row_map = c->d_row_map;
        if (pr.down) {
            a.groups = c->d_group_dn;
            a.group_units = c->group_units_dn;
        } else {
            a.N = c->groups * c->live_blocks * c->cfg.block;
            a.nt = ceil_div(a.N, lb::BN);
            a.col_map = c->d_col_map;
            a.groups = c->d_group_up;
            a.group_units = c->group_units_up;
        }
    }
    const long long total_units = grouped ? 2ll * a.group_units
                                          : 2ll * mt * nt * (few ? comet::LIMB_FEW_PAIRS : 2) * kb;
    c->stats.tensor_tile_macs = total_units * lb::KC * (few ? lf::BW * lf::BT : lb::BM * lb::BN);
    const int grid = (int)(total_units < c->sm_count ? total_units : c->sm_count);
    {
        PhaseTimer timer(c, COMET_PHASE_COMBINE, 1);
        // The persistent kernel needs a slot on every SM.  With the device's highest scheduling priority its CTAs
        // get the slots that free up before the memory-side CTAs of other contexts queued beside it do, so the
        // tensor cores do not wait behind work that could as well run under them.
        const dim3 block(few ? lf::THREADS : lb::THREADS);
        const size_t smem = few ? lf::SMEM_BYTES : lb::SMEM_BYTES;
        auto* kernel = few ? comet::combine_limb_few_kernel
                           : grouped ? comet::combine_limb_grouped_kernel : comet::combine_limb_kernel;
        COMET_CUDA(c, launch_chained(kernel, dim3(grid), block, smem, c->stream, &c->top_priority, a));
    }
    c->stats.kernel_launches += 1;
    c->stats.matmul_path = COMET_PATH_LIMB;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

bool limb_fits(const comet_ctx* c, const Proj& pr) {
    namespace lb = comet::limb;
    // the few-token layout (32-row token tiles, 128-row weight tiles) never needs more than the ordinary one
    // plus one 64-row tile of the right operand, which the allocation includes
    const size_t kb = ceil_div(pr.K, lb::KC), mt = ceil_div(pr.M, lb::BM), nt = ceil_div(pr.N, lb::BN) + 1;
    return mt * kb * lb::A_BLOCK_BYTES <= c->planes_left_bytes &&
           nt * kb * lb::B_BLOCK_BYTES <= (pr.down ? c->planes_right_dn_bytes : c->planes_right_up_bytes);
}

int launch_combine(comet_ctx* c, int M, int N, int K, int idE, int idF, int idA, int idB, int idC, int idZ) {
    comet::CombineArgs a;
    for (int p = 0; p < 2; ++p) {
        a.E[p] = c->buf[p][idE];
        a.F[p] = c->buf[p][idF];
        a.A[p] = c->buf[p][idA];
        a.B[p] = c->buf[p][idB];
        a.C[p] = c->buf[p][idC];
        a.Z[p] = c->buf[p][idZ];
    }
    a.M = M; a.N = N; a.K = K;
    a.tmask = (idZ == COMET_Y && c->tmask_set) ? c->d_tmask : nullptr;
    a.tmask_ld = c->n_active_blocks;
    a.bs = c->cfg.block;
    dim3 grid((N + comet::simt::BN - 1) / comet::simt::BN, (M + comet::simt::BM - 1) / comet::simt::BM, 2);
    PhaseTimer timer(c, COMET_PHASE_COMBINE, 1);
    comet::combine_simt_kernel<<<grid, comet::simt::THREADS, 0, c->stream>>>(a);
    c->stats.kernel_launches += 1;
    c->stats.matmul_path = COMET_PATH_SIMT;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

// The Merge step of Protocol 2 under a token mask: entries of the compact result outside the component blocks become zero.
int somm_merge(comet_ctx* c, int tokens) {
    if (!c->tmask_set) return COMET_OK;
    const int cols = c->groups * c->n_active;
    const int64_t pairs = (int64_t)tokens * cols / 2;
    if (pairs == 0) return COMET_OK;
    comet::PartyOut Z;
    for (int p = 0; p < 2; ++p) Z.p[p] = c->buf[p][COMET_Z_UP];
    COMET_CUDA(c, launch_chained(comet::somm_merge_kernel, dim3(ew_grid(c, pairs, 256), 2), dim3(256), 0, c->stream,
                                 nullptr, Z, pairs, cols, (int)c->n_active, (int)c->cfg.block,
                                 (const int32_t*)c->d_row_label, (const int32_t*)c->d_blk_label));
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

}  // namespace

extern "C" {

const char* comet_strerror(int code) {
    switch (code) {
        case COMET_OK: return "ok";
        case COMET_ERR_INVALID_ARG: return "invalid argument";
        case COMET_ERR_SHAPE: return "shape disagrees with the configuration or the current mask";
        case COMET_ERR_STATE: return "call out of order: a required input has not been loaded";
        case COMET_ERR_OOM: return "device memory allocation failed";
        case COMET_ERR_CUDA: return "a CUDA runtime call failed";
        case COMET_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case COMET_ERR_SCRATCH_LIMIT:
            return "problem exceeds the library's static scratch array (COMET_STATIC_SCRATCH_WORDS)";
        default: return "unknown error code";
    }
}

int comet_last_cuda_error(comet_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

int comet_init(const comet_config* cfg, void* cuda_stream, comet_ctx** out) {
    if (!cfg || !out) return COMET_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->gated < 0 || cfg->gated > 2) return COMET_ERR_INVALID_ARG;
    if (cfg->matmul_path < COMET_PATH_AUTO || cfg->matmul_path > COMET_PATH_LIMB) return COMET_ERR_INVALID_ARG;
    if (cfg->device < 0) return COMET_ERR_INVALID_ARG;
    if (cfg->max_tokens < 1 || cfg->d_model < 16 || cfg->d_ff < 16 || cfg->block < 16) return COMET_ERR_SHAPE;
    if (cfg->d_model % 16 || cfg->block % 16 || cfg->d_ff % cfg->block) return COMET_ERR_SHAPE;
    if (cfg->frac_bits < 1 || cfg->frac_bits > 31) return COMET_ERR_SHAPE;
    if (cfg->max_active < 0 || cfg->max_active > cfg->d_ff || cfg->max_active % cfg->block) return COMET_ERR_SHAPE;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device >= ndev) {
        cudaGetLastError();
        return COMET_ERR_CUDA;
    }
    comet_ctx* c = new (std::nothrow) comet_ctx;
    if (!c) return COMET_ERR_OOM;
    std::memset(c, 0, sizeof(*c));
    c->pending = new (std::nothrow) std::vector<comet_ctx::Pending>();
    c->free_events = new (std::nothrow) std::vector<cudaEvent_t>();
    if (!c->pending || !c->free_events) {
        delete c->pending;
        delete c->free_events;
        delete c;
        return COMET_ERR_OOM;
    }
    c->cfg = *cfg;
    c->stream = (cudaStream_t)cuda_stream;
    c->groups = cfg->gated + 1;
    c->cap_T = cfg->max_tokens;
    c->cap_n = cfg->max_active ? cfg->max_active : cfg->d_ff;
    if (cudaSetDevice(cfg->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) {
        cudaGetLastError();
        delete c->pending;
        delete c->free_events;
        delete c;
        return COMET_ERR_CUDA;
    }
    {
        int least = 0, greatest = 0;
        if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) cudaGetLastError();
        c->top_priority = greatest;
    }
    bool ok = true;
    for (int id = 0; id < COMET_NUM_TENSORS && ok; ++id) {
        c->cap_words[id] = tensor_capacity(c, id);
        for (int p = 0; p < 2 && ok; ++p)
            if (c->cap_words[id] > 0)
            {
                ok = cudaMalloc((void**)&c->own[p][id], (size_t)c->cap_words[id] * sizeof(u64)) == cudaSuccess;
                c->buf[p][id] = c->own[p][id];
            }
    }
    c->path = cfg->matmul_path == COMET_PATH_AUTO ? COMET_PATH_LIMB : cfg->matmul_path;
    if (c->path == COMET_PATH_LIMB) {
        namespace lb = comet::limb;
        const int d = cfg->d_model;
        const int64_t n = c->cap_n, gn = c->groups * n;
        const int64_t kb_up = (d + lb::KC - 1) / lb::KC, kb_dn = (n + lb::KC - 1) / lb::KC;
        const int64_t kb_max = kb_up > kb_dn ? kb_up : kb_dn;
        const int64_t mt = (c->cap_T + lb::BM - 1) / lb::BM;
        c->planes_left_bytes = (size_t)(mt * kb_max) * lb::A_BLOCK_BYTES;
        c->planes_right_up_bytes = (size_t)(((gn + lb::BN - 1) / lb::BN + 1) * kb_up) * lb::B_BLOCK_BYTES;
        c->planes_right_dn_bytes = (size_t)(((d + lb::BN - 1) / lb::BN + 1) * kb_dn) * lb::B_BLOCK_BYTES;
        for (int p = 0; p < 2 && ok; ++p)
            for (int w = 0; w < 2 && ok; ++w) {
                ok = cudaMalloc((void**)&c->planes_left[p][w], c->planes_left_bytes) == cudaSuccess;
                ok = ok && cudaMalloc((void**)&c->planes_right_up[p][w], c->planes_right_up_bytes) == cudaSuccess;
                ok = ok && cudaMalloc((void**)&c->planes_right_dn[p][w], c->planes_right_dn_bytes) == cudaSuccess;
            }
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)lb::SMEM_BYTES) == cudaSuccess;
        // the memory-side kernels may share an SM with a resident tensor-core CTA (which forces the largest
        // shared-memory carve-out), so they ask for the same carve-out
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_few_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)comet::limb_few::SMEM_BYTES) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_few_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_grouped_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)lb::SMEM_BYTES) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::combine_limb_grouped_kernel,
                                        cudaFuncAttributePreferredSharedMemoryCarveout,
                                        (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::limb_open_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::limb_prep_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                        (int)cudaSharedmemCarveoutMaxShared) == cudaSuccess;
        ok = ok && cudaFuncSetAttribute(comet::limb_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(lb::OPEN_STAGES * 3 * lb::OPEN_TILE_BYTES)) == cudaSuccess;
        ok = ok && cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
    }
    const int nb = cfg->d_ff / cfg->block;
    ok = ok && cudaMalloc((void**)&c->d_mask, (size_t)nb) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_tmask, (size_t)nb * (size_t)c->cap_T) == cudaSuccess;
    ok = ok && cudaHostAlloc((void**)&c->h_mask_stage, (size_t)nb * 4, cudaHostAllocDefault) == cudaSuccess;
    for (int k = 0; k < 4 && ok; ++k)
        ok = cudaEventCreateWithFlags(&c->stage_done[k], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc((void**)&c->h_masked, 7 * sizeof(long long), cudaHostAllocMapped) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_row_map, (size_t)c->cap_T * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_col_map, (size_t)c->groups * nb * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_kmap, (size_t)nb * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_plan_scratch,
                          ((size_t)c->cap_T * ceil_div(nb, 32) + (size_t)c->groups * nb) * sizeof(uint32_t)) == cudaSuccess;
    {
        const size_t mt = ceil_div((int)c->cap_T, comet::limb::BM);
        ok = ok && cudaMalloc((void**)&c->d_group_up, mt * sizeof(comet::LimbGroupRow)) == cudaSuccess;
        ok = ok && cudaMalloc((void**)&c->d_group_dn, mt * sizeof(comet::LimbGroupRow)) == cudaSuccess;
    }
    ok = ok && cudaMalloc((void**)&c->d_row_label, (size_t)c->cap_T * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_blk_label, (size_t)nb * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaHostGetDevicePointer((void**)&c->h_masked_dev, c->h_masked, 0) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_ids, (size_t)nb * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->d_count, 2 * sizeof(int32_t)) == cudaSuccess;   // {count, error flag}
    ok = ok && cudaMemset(c->d_count, 0, 2 * sizeof(int32_t)) == cudaSuccess;
    if (ok) c->d_error = c->d_count + 1;
    ok = ok && cudaHostAlloc((void**)&c->h_count, 4 * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess;
    if (ok) c->h_count[0] = c->h_count[1] = c->h_count[2] = c->h_count[3] = 0;     // pinned memory is not zeroed
    ok = ok && cudaHostGetDevicePointer((void**)&c->h_count_dev, c->h_count, 0) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        comet_destroy(c);
        return COMET_ERR_OOM;
    }
    *out = c;
    return COMET_OK;
}

void comet_destroy(comet_ctx* c) {
    if (!c) return;
    cudaSetDevice(c->cfg.device);
    cudaStreamSynchronize(c->stream);
    for (int id = 0; id < COMET_NUM_TENSORS; ++id)
        for (int p = 0; p < 2; ++p)
            if (c->own[p][id]) cudaFree(c->own[p][id]);
    if (c->side) cudaStreamSynchronize(c->side);
    for (int p = 0; p < 2; ++p)
        for (int w = 0; w < 2; ++w) {
            if (c->planes_left[p][w]) cudaFree(c->planes_left[p][w]);
            if (c->planes_right_up[p][w]) cudaFree(c->planes_right_up[p][w]);
            if (c->planes_right_dn[p][w]) cudaFree(c->planes_right_dn[p][w]);
        }
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->side) cudaStreamDestroy(c->side);
    if (c->d_mask) cudaFree(c->d_mask);
    if (c->d_tmask) cudaFree(c->d_tmask);
    if (c->h_mask_stage) cudaFreeHost(c->h_mask_stage);
    for (int k = 0; k < 4; ++k)
        if (c->stage_done[k]) cudaEventDestroy(c->stage_done[k]);
    if (c->h_masked) cudaFreeHost(c->h_masked);
    if (c->d_row_label) cudaFree(c->d_row_label);
    if (c->d_row_map) cudaFree(c->d_row_map);
    if (c->d_col_map) cudaFree(c->d_col_map);
    if (c->d_kmap) cudaFree(c->d_kmap);
    if (c->d_plan_scratch) cudaFree(c->d_plan_scratch);
    if (c->d_group_up) cudaFree(c->d_group_up);
    if (c->d_group_dn) cudaFree(c->d_group_dn);
    if (c->d_blk_label) cudaFree(c->d_blk_label);
    if (c->d_ids) cudaFree(c->d_ids);
    if (c->d_count) cudaFree(c->d_count);
    if (c->h_count) cudaFreeHost(c->h_count);
    for (auto& p : *c->pending) {
        cudaEventDestroy(p.start);
        cudaEventDestroy(p.stop);
    }
    for (auto e : *c->free_events) cudaEventDestroy(e);
    delete c->pending;
    delete c->free_events;
    cudaGetLastError();
    delete c;
}

// Shared by comet_load_shares (copy) and comet_bind_shares (use in place).
static int set_shares(comet_ctx* c, int party, int tensor_id, const uint64_t* ptr, int location, int64_t rows,
                      int64_t cols, bool bind) {
    if (!c || (party != 0 && party != 1) || !is_input(tensor_id)) return COMET_ERR_INVALID_ARG;
    if (!ptr && rows * cols != 0) return COMET_ERR_INVALID_ARG;      // an empty tensor may come with a null pointer
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (bind && (location != COMET_DEVICE || (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0)) return COMET_ERR_INVALID_ARG;
    if (tensor_id == COMET_WG && c->groups < 2) return COMET_ERR_INVALID_ARG;
    if (tensor_id == COMET_W3 && c->groups != 3) return COMET_ERR_INVALID_ARG;
    const bool needs_mask = tensor_id == COMET_B_UP || tensor_id == COMET_C_UP || tensor_id == COMET_H ||
                            tensor_id == COMET_A_DN || tensor_id == COMET_B_DN;
    if (needs_mask && !c->mask_set) return COMET_ERR_STATE;
    const bool token_rows = tensor_id == COMET_X || tensor_id == COMET_A_UP || tensor_id == COMET_C_UP ||
                            tensor_id == COMET_H || tensor_id == COMET_A_DN || tensor_id == COMET_C_DN;
    if (token_rows && (rows < 1 || rows > c->cap_T)) return COMET_ERR_SHAPE;
    int64_t er, ec;
    tensor_shape(c, tensor_id, rows, &er, &ec);
    if (rows != er || cols != ec) return COMET_ERR_SHAPE;
    if (rows * cols > c->cap_words[tensor_id]) return COMET_ERR_SHAPE;
    if (tensor_id == COMET_W2 || tensor_id == COMET_B_DN || tensor_id == COMET_C_DN) {
        const int rc = join_side(c);       // the side stream may still be reading the old contents
        if (rc != COMET_OK) return rc;
        if (tensor_id == COMET_C_DN) c->dn_copy_ready = false;
        else c->dn_right_ready = false;
    }
    if (bind && rows * cols > 0) {
        c->buf[party][tensor_id] = const_cast<u64*>(reinterpret_cast<const u64*>(ptr));   // only ever read
    } else {
        c->buf[party][tensor_id] = c->own[party][tensor_id];
        if (rows * cols > 0)
            COMET_CUDA(c, cudaMemcpyAsync(c->buf[party][tensor_id], ptr, (size_t)(rows * cols) * sizeof(u64),
                                          copy_kind(location, true), c->stream));
    }
    c->loaded[party][tensor_id] = true;
    if (token_rows) c->tokens = (int32_t)rows;
    return COMET_OK;
}

int comet_load_shares(comet_ctx* c, int party, int tensor_id, const uint64_t* ptr, int location, int64_t rows,
                      int64_t cols) {
    return set_shares(c, party, tensor_id, ptr, location, rows, cols, false);
}

int comet_bind_shares(comet_ctx* c, int party, int tensor_id, const uint64_t* dev_ptr, int64_t rows, int64_t cols) {
    return set_shares(c, party, tensor_id, dev_ptr, COMET_DEVICE, rows, cols, true);
}

int comet_set_mask(comet_ctx* c, const uint8_t* block_mask, int location, int32_t n_blocks, int32_t* n_active_out) {
    if (!c || !block_mask || !n_active_out) return COMET_ERR_INVALID_ARG;
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (n_blocks != c->cfg.d_ff / c->cfg.block) return COMET_ERR_SHAPE;
    {
        const int rc = join_side(c);           // the side stream reads the index list
        if (rc != COMET_OK) return rc;
    }
    c->dn_right_ready = false;
    const uint8_t* dmask = block_mask;         // a device mask is read in place
    int32_t host_count = -1;                   // number of active blocks when the host could count them itself
    bool launched = false;
    if (location == COMET_HOST) {
        // The count is public (Section 3.2) and the mask is in host memory: count here and do not wait for the
        // device.  A mask that fits into a kernel's parameter block travels with the launch; a larger one is handed
        // to the copy engine from a pinned slot of our own (the caller's buffer is free again on return either way).
        host_count = 0;
        for (int32_t b = 0; b < n_blocks; ++b) host_count += block_mask[b] != 0;
        if (n_blocks <= comet::MaskBytes::CAPACITY) {
            comet::MaskBytes arg;
            std::memcpy(arg.bytes, block_mask, (size_t)n_blocks);
            PhaseTimer timer(c, COMET_PHASE_COMPACT, 1);
            c->ticket += 1;
            COMET_CUDA(c, launch_chained(comet::compact_mask_arg_kernel, dim3(1), dim3(1024), 0, c->stream, nullptr, arg,
                                         (int)n_blocks, c->d_ids, c->d_count, (int32_t*)nullptr, c->ticket));
            launched = true;
        } else {
            const int slot = c->stage_next;
            c->stage_next = (slot + 1) % 4;
            if (c->stage_used[slot]) COMET_CUDA(c, cudaEventSynchronize(c->stage_done[slot]));
            uint8_t* stage = c->h_mask_stage + (size_t)slot * n_blocks;
            std::memcpy(stage, block_mask, (size_t)n_blocks);
            COMET_CUDA(c, cudaMemcpyAsync(c->d_mask, stage, (size_t)n_blocks, cudaMemcpyHostToDevice, c->stream));
            COMET_CUDA(c, cudaEventRecord(c->stage_done[slot], c->stream));
            c->stage_used[slot] = true;
            dmask = c->d_mask;
        }
    }
    if (!launched) {
        PhaseTimer timer(c, COMET_PHASE_COMPACT, 1);
        // the kernel reports {count, error flag} straight into mapped host memory: no copy to enqueue
        c->ticket += 1;
        COMET_CUDA(c, launch_chained(comet::compact_mask_kernel, dim3(1), dim3(1024), 0, c->stream, nullptr, dmask,
                                     (int)n_blocks, c->d_ids, c->d_count, host_count < 0 ? c->h_count_dev : (int32_t*)nullptr,
                                     c->ticket));
    }
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    if (host_count < 0) {
        // The kernel is the last thing on the stream and reports through mapped memory: watching its ticket for
        // a short while is quicker than a stream synchronise; after that, synchronise as usual.
        volatile int32_t* seen = c->h_count + 2;
        const auto t0 = std::chrono::steady_clock::now();
        bool arrived = false;
        while (!(arrived = (*seen == c->ticket))) {
            if (std::chrono::steady_clock::now() - t0 > std::chrono::microseconds(300)) break;
        }
        if (!arrived) COMET_CUDA(c, cudaStreamSynchronize(c->stream));
        std::atomic_thread_fence(std::memory_order_acquire);
    }
    if (timed_out(c)) return COMET_ERR_TIMEOUT;           // an earlier kernel gave up on a bounded wait
    const int32_t blocks = host_count >= 0 ? host_count : *c->h_count;
    const int64_t n = (int64_t)blocks * c->cfg.block;
    if (n > c->cap_n) {            // more active neurons than the context was sized for
        c->mask_set = false;
        return COMET_ERR_SHAPE;
    }
    c->n_active_blocks = blocks;
    c->n_active = (int32_t)n;
    c->mask_set = true;
    c->tmask_set = false;             // a token mask refines one block mask
    c->grouped = false;
    c->up_done = c->down_done = false;
    for (int p = 0; p < 2; ++p)
        for (int id = COMET_A_UP; id <= COMET_C_DN; ++id) {
            c->loaded[p][id] = false;
            c->buf[p][id] = c->own[p][id];          // a binding ends with the mask it was made under
        }
    c->stats.n_active = c->n_active;
    c->stats.n_active_blocks = blocks;
    *n_active_out = c->n_active;
    return COMET_OK;
}

int comet_set_token_mask(comet_ctx* c, const uint8_t* token_mask, int location, int32_t tokens,
                         int32_t n_active_blocks, int64_t* masked_out) {
    if (!c) return COMET_ERR_INVALID_ARG;
    if (!c->mask_set) return COMET_ERR_STATE;
    if (!token_mask) {                         // back to "every token uses every active neuron"
        if (tokens != 0 || n_active_blocks != 0) return COMET_ERR_INVALID_ARG;
        // the weight side of the down-projection may have been opened early under the mask that is going away
        // (its unused blocks zeroed, its contraction index in component order): it is opened again
        if (c->tmask_set) c->dn_right_ready = false;
        c->tmask_set = false;
        c->grouped = false;
        if (masked_out) *masked_out = 0;
        return COMET_OK;
    }
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (tokens < 1 || tokens > c->cap_T || n_active_blocks != c->n_active_blocks || n_active_blocks < 1)
        return COMET_ERR_SHAPE;
    if ((int64_t)tokens * c->n_active < 0 || (int64_t)tokens * c->n_active > 0x7fffffffll) return COMET_ERR_SHAPE;
    const size_t bytes = (size_t)tokens * (size_t)n_active_blocks;
    COMET_CUDA(c, cudaMemcpyAsync(c->d_tmask, token_mask, bytes, copy_kind(location, true), c->stream));
    // Protocol 2, first step: the connected components the up-projection is partitioned into, the number of
    // non-zero entries (Theorem 2's count) and, for the tensor-core path, the component-sorted order and the work
    // of every row tile, in one launch
    const bool plan = c->path == COMET_PATH_LIMB && tokens > comet::limb_few::BT && tokens <= 32768;
    {
        comet::TokenPlanArgs a;
        std::memset(&a, 0, sizeof(a));
        a.S = c->d_tmask;
        a.T = tokens; a.nab = n_active_blocks; a.wpr = ceil_div(n_active_blocks, 32);
        a.row_label = c->d_row_label; a.blk_label = c->d_blk_label;
        a.report = c->h_masked_dev;
        a.scratch = c->d_plan_scratch;
        a.plan = plan ? 1 : 0;
        a.groups = c->groups; a.bs = c->cfg.block;
        a.kb_up = ceil_div(c->cfg.d_model, comet::limb::KC);
        a.nt_dn = ceil_div(c->cfg.d_model, comet::limb::BN);
        a.row_map = c->d_row_map; a.col_map = c->d_col_map; a.kmap = c->d_kmap;
        a.up = c->d_group_up; a.dn = c->d_group_dn;
        const size_t words = (size_t)tokens * a.wpr + tokens + (size_t)n_active_blocks * (1 + c->groups);
        a.in_smem = words * sizeof(uint32_t) <= 36 * 1024 ? 1 : 0;
        comet::token_plan_kernel<<<1, 1024, a.in_smem ? words * sizeof(uint32_t) : 0, c->stream>>>(a);
    }
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    COMET_CUDA(c, cudaStreamSynchronize(c->stream));
    c->tmask_masked = (int64_t)c->h_masked[0] * c->cfg.block;
    c->n_components = (int32_t)c->h_masked[1];
    c->live_rows = (int32_t)c->h_masked[2];
    c->live_blocks = (int32_t)c->h_masked[3];
    c->group_units_up = plan ? (int32_t)c->h_masked[4] : 0;
    c->component_pairs = plan ? (int64_t)c->h_masked[5] : -1;
    c->group_units_dn = plan ? (int32_t)c->h_masked[6] : 0;
    // several components, or rows / blocks in none: compute the component rectangles only
    c->grouped = plan && c->group_units_up > 0 && c->group_units_dn > 0 &&
                 (c->n_components > 1 || c->live_rows < tokens || c->live_blocks < n_active_blocks);
    c->dn_right_ready = false;    // the order of the contraction index in the down-projection's planes may change
    c->stats.n_components = c->n_components;
    c->tmask_tokens = tokens;
    c->tmask_set = true;
    if (masked_out) *masked_out = c->tmask_masked;
    return COMET_OK;
}

int comet_ffn_up(comet_ctx* c, int32_t tokens) {
    if (!c) return COMET_ERR_INVALID_ARG;
    if (tokens < 1 || tokens > c->cap_T) return COMET_ERR_SHAPE;
    if (!c->mask_set) return COMET_ERR_STATE;
    const int need[] = {COMET_X, COMET_W1, COMET_A_UP, COMET_B_UP, COMET_C_UP};
    for (int p = 0; p < 2; ++p) {
        for (int id : need)
            if (!c->loaded[p][id]) return COMET_ERR_STATE;
        if (c->groups >= 2 && !c->loaded[p][COMET_WG]) return COMET_ERR_STATE;
        if (c->groups == 3 && !c->loaded[p][COMET_W3]) return COMET_ERR_STATE;
    }
    const int d = c->cfg.d_model, n = c->n_active, g = c->groups, bs = c->cfg.block;
    if (c->tmask_set && c->tmask_tokens != tokens) return COMET_ERR_SHAPE;   // the token mask was given for another T
    c->stats.tokens = tokens;
    // under a token mask only the rows and columns of the connected components are opened (Theorem 1)
    c->stats.message_bytes = c->tmask_set
        ? 2ll * 8 * ((int64_t)c->live_rows * d + (int64_t)d * g * c->live_blocks * bs)
        : 2ll * 8 * ((int64_t)tokens * d + (int64_t)d * g * n);
    // Theorem 1's multiplication count when the components are known (one product per component), else the
    // product over the union of the supports
    c->stats.ring_macs = (c->tmask_set && c->component_pairs >= 0)
        ? 2ll * 2 * d * g * bs * c->component_pairs : 2ll * 2 * tokens * (int64_t)d * g * n;
    c->stats.tensor_tile_macs = 0;
    c->up_tokens = tokens;
    c->up_done = true;
    if (n == 0) return COMET_OK;

    if (c->path == COMET_PATH_LIMB) {
        const Proj up = proj_up(c, tokens), dn = proj_down(c, tokens);
        if (!limb_fits(c, up)) return COMET_ERR_SHAPE;
        int rc = join_side(c);
        if (rc != COMET_OK) return rc;
        {
            PhaseTimer timer(c, COMET_PHASE_OPEN, 1);
            rc = limb_open(c, up, true, true, c->stream);
        }
        if (rc != COMET_OK) return rc;
        // The weight side of the down-projection depends only on the mask, W2 and B'_i: if those are loaded
        // already, open it now on the side stream, beside the preparation and the tensor-core kernel that follow.
        // (The fork sits before the preparation kernel so that nothing separates that kernel from the tensor-core
        // kernel on the main stream: the latter is launched as the former's programmatic dependent.)
        const bool early = !c->dn_right_ready && limb_fits(c, dn) && c->loaded[0][COMET_W2] &&
                           c->loaded[1][COMET_W2] && c->loaded[0][COMET_B_DN] && c->loaded[1][COMET_B_DN];
        if (early) {
            COMET_CUDA(c, cudaEventRecord(c->ev_fork, c->stream));
            COMET_CUDA(c, cudaStreamWaitEvent(c->side, c->ev_fork, 0));
            // ... and if the triple's C' share is there too, Y_i <- C'_i, the value the down-projection's sums are
            // added to, is copied in the same launch
            const bool copy = c->loaded[0][COMET_C_DN] && c->loaded[1][COMET_C_DN];
            rc = limb_open(c, dn, false, true, c->side);
            if (rc == COMET_OK) rc = limb_prep(c, dn, false, true, copy, c->side);
            if (rc != COMET_OK) return rc;
            COMET_CUDA(c, cudaEventRecord(c->ev_join, c->side));
            c->side_pending = true;
            c->dn_right_ready = true;
            c->dn_right_few = limb_few(dn);
            c->dn_copy_ready = copy;
            c->dn_copy_tokens = tokens;
        }
        {
            PhaseTimer timer(c, COMET_PHASE_PREP, 1);
            rc = limb_prep(c, up, true, true, true, c->stream);
        }
        if (rc != COMET_OK) return rc;
        rc = limb_combine(c, up);
        if (rc != COMET_OK) return rc;
        return somm_merge(c, tokens);
    }

    comet::PartyPtrs X, A, W0, W1, W3, B;
    comet::PartyOut E, F;
    for (int p = 0; p < 2; ++p) {
        X.p[p] = c->buf[p][COMET_X];
        A.p[p] = c->buf[p][COMET_A_UP];
        E.p[p] = c->buf[p][COMET_E_UP];
        W0.p[p] = (g >= 2) ? c->buf[p][COMET_WG] : c->buf[p][COMET_W1];
        W3.p[p] = c->buf[p][COMET_W3];
        W1.p[p] = c->buf[p][COMET_W1];
        B.p[p] = c->buf[p][COMET_B_UP];
        F.p[p] = c->buf[p][COMET_F_UP];
    }
    const int64_t pairs = (int64_t)tokens * d / 2;
    {
        PhaseTimer timer(c, COMET_PHASE_OPEN, 2);
        comet::open_activation_kernel<<<dim3(ew_grid(c, pairs, 256), 2), 256, 0, c->stream>>>(
            X, A, E, pairs, nullptr, 0, d, bs, c->tmask_set ? c->d_row_label : nullptr);
        int rows_grid = g * n < c->sm_count * 8 ? g * n : c->sm_count * 8;
        comet::open_weight_rows_kernel<<<dim3(rows_grid, 2), 256, 0, c->stream>>>(
            W0, W1, W3, B, F, c->d_ids, n, g, bs, d, c->tmask_set ? c->d_blk_label : nullptr);
    }
    c->stats.kernel_launches += 2;
    COMET_CUDA(c, cudaGetLastError());
    const int rc = launch_combine(c, tokens, g * n, d, COMET_E_UP, COMET_F_UP, COMET_A_UP, COMET_B_UP, COMET_C_UP,
                                  COMET_Z_UP);
    if (rc != COMET_OK) return rc;
    return somm_merge(c, tokens);
}

int comet_ffn_down(comet_ctx* c, int32_t tokens) {
    if (!c) return COMET_ERR_INVALID_ARG;
    if (tokens < 1 || tokens > c->cap_T) return COMET_ERR_SHAPE;
    if (!c->mask_set) return COMET_ERR_STATE;
    const int d = c->cfg.d_model, n = c->n_active, bs = c->cfg.block, D = c->cfg.d_ff;
    for (int p = 0; p < 2; ++p) {
        if (!c->loaded[p][COMET_W2] || !c->loaded[p][COMET_C_DN]) return COMET_ERR_STATE;
        if (n > 0 && (!c->loaded[p][COMET_H] || !c->loaded[p][COMET_A_DN] || !c->loaded[p][COMET_B_DN]))
            return COMET_ERR_STATE;
    }
    if (c->tmask_set && c->tmask_tokens != tokens) return COMET_ERR_SHAPE;   // the token mask was given for another T
    c->stats.tokens = tokens;
    // with a token mask only the non-zero entries of the hidden state and the rows of the weight matrix that meet
    // a non-zero column are opened (Theorem 2's communication)
    c->stats.message_bytes = c->tmask_set
        ? 2ll * 8 * (c->tmask_masked + (int64_t)c->live_blocks * bs * d)
        : 2ll * 8 * ((int64_t)tokens * n + (int64_t)n * d);
    // Theorem 2's multiplication count under a token mask (one product row per non-zero entry), else the full product
    c->stats.ring_macs = 2ll * 2 * (c->tmask_set ? c->tmask_masked : (int64_t)tokens * n) * d;
    c->stats.tensor_tile_macs = 0;
    c->down_tokens = tokens;
    c->down_done = true;
    if (n == 0) {
        // no active neuron: the product is empty and both result shares are zero
        for (int p = 0; p < 2; ++p)
            COMET_CUDA(c, cudaMemsetAsync(c->buf[p][COMET_Y], 0, (size_t)tokens * d * sizeof(u64), c->stream));
        return COMET_OK;
    }
    if (c->path == COMET_PATH_LIMB) {
        const Proj dn = proj_down(c, tokens);
        if (!limb_fits(c, dn)) return COMET_ERR_SHAPE;
        // opened early, during the up-projection, and in the plane layout this token count needs
        const bool have_right = c->dn_right_ready && c->dn_right_few == limb_few(dn);
        const bool have_copy = c->dn_right_ready && c->dn_copy_ready && c->dn_copy_tokens == tokens;
        int rc = join_side(c);
        if (rc != COMET_OK) return rc;
        {
            PhaseTimer timer(c, COMET_PHASE_OPEN, 1);
            rc = limb_open(c, dn, true, !have_right, c->stream);
        }
        if (rc != COMET_OK) return rc;
        {
            PhaseTimer timer(c, COMET_PHASE_PREP, 1);
            rc = limb_prep(c, dn, true, !have_right, !have_copy, c->stream);
        }
        if (rc != COMET_OK) return rc;
        c->dn_right_ready = false;                     // a triple serves one product
        c->dn_copy_ready = false;
        return limb_combine(c, dn);
    }

    comet::PartyPtrs H, A, W, B;
    comet::PartyOut E, F;
    for (int p = 0; p < 2; ++p) {
        H.p[p] = c->buf[p][COMET_H];
        A.p[p] = c->buf[p][COMET_A_DN];
        E.p[p] = c->buf[p][COMET_E_DN];
        W.p[p] = c->buf[p][COMET_W2];
        B.p[p] = c->buf[p][COMET_B_DN];
        F.p[p] = c->buf[p][COMET_F_DN];
    }
    const int64_t pairs = (int64_t)tokens * n / 2;
    {
        PhaseTimer timer(c, COMET_PHASE_OPEN, 2);
        comet::open_activation_kernel<<<dim3(ew_grid(c, pairs, 256), 2), 256, 0, c->stream>>>(
            H, A, E, pairs, c->tmask_set ? c->d_tmask : nullptr, c->n_active_blocks, n, bs);
        const int64_t wpairs = (int64_t)d * n / 2;
        comet::open_weight_strips_kernel<<<dim3(ew_grid(c, wpairs, 256), 2), 256, 0, c->stream>>>(
            W, B, F, c->d_ids, n, bs, d, D, c->tmask_set ? c->d_blk_label : nullptr);
    }
    c->stats.kernel_launches += 2;
    COMET_CUDA(c, cudaGetLastError());
    return launch_combine(c, tokens, d, n, COMET_E_DN, COMET_F_DN, COMET_A_DN, COMET_B_DN, COMET_C_DN, COMET_Y);
}

int comet_truncate(comet_ctx* c, int tensor_id) {
    if (!c || (tensor_id != COMET_Z_UP && tensor_id != COMET_Y)) return COMET_ERR_INVALID_ARG;
    const bool up = tensor_id == COMET_Z_UP;
    if (up ? !c->up_done : !c->down_done) return COMET_ERR_STATE;
    int64_t rows, cols;
    tensor_shape(c, tensor_id, up ? c->up_tokens : c->down_tokens, &rows, &cols);
    const int64_t pairs = rows * cols / 2;
    if (pairs == 0) return COMET_OK;
    comet::PartyOut Z;
    for (int p = 0; p < 2; ++p) Z.p[p] = c->buf[p][tensor_id];
    {
        PhaseTimer timer(c, COMET_PHASE_TRUNCATE, 1);
        COMET_CUDA(c, launch_chained(comet::truncate_kernel, dim3(ew_grid(c, pairs, 256), 2), dim3(256), 0, c->stream,
                                     nullptr, Z, pairs, (int)c->cfg.frac_bits));
    }
    c->stats.kernel_launches += 1;
    COMET_CUDA(c, cudaGetLastError());
    return COMET_OK;
}

int comet_get(comet_ctx* c, int party, int tensor_id, uint64_t* out, int location, int64_t capacity,
              int64_t* written) {
    if (!c || !out || (party != 0 && party != 1) || tensor_id < 0 || tensor_id >= COMET_NUM_TENSORS)
        return COMET_ERR_INVALID_ARG;
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (tensor_id == COMET_WG && c->groups < 2) return COMET_ERR_INVALID_ARG;
    if (tensor_id == COMET_W3 && c->groups != 3) return COMET_ERR_INVALID_ARG;
    int64_t T = c->tokens;
    if (tensor_id == COMET_E_UP || tensor_id == COMET_Z_UP) T = c->up_tokens;
    if (tensor_id == COMET_E_DN || tensor_id == COMET_Y) T = c->down_tokens;
    int64_t rows, cols;
    tensor_shape(c, tensor_id, T, &rows, &cols);
    const int64_t words = rows * cols;
    if (is_input(tensor_id) ? !c->loaded[party][tensor_id]
                            : !((tensor_id == COMET_E_UP || tensor_id == COMET_F_UP || tensor_id == COMET_Z_UP)
                                    ? c->up_done : c->down_done))
        return COMET_ERR_STATE;
    if (capacity < words) return COMET_ERR_SHAPE;
    if (words > 0 && (tensor_id == COMET_F_UP || tensor_id == COMET_F_DN) &&
        c->f_as_planes[tensor_id == COMET_F_DN ? 1 : 0] && c->path == COMET_PATH_LIMB) {
        // a few-token product wrote this message as limb planes only: rebuild the words
        uint8_t* (*planes)[2] = tensor_id == COMET_F_DN ? c->planes_right_dn : c->planes_right_up;
        comet::limb_planes_to_words_kernel<<<ew_grid(c, words, 256), 256, 0, c->stream>>>(
            planes[party][1], c->buf[party][tensor_id], (int)rows, (int)cols, ceil_div((int)cols, comet::limb::KC),
            comet::limb_few::BW);
        c->stats.kernel_launches += 1;
        COMET_CUDA(c, cudaGetLastError());
    }
    if (words > 0)
        COMET_CUDA(c, cudaMemcpyAsync(out, c->buf[party][tensor_id], (size_t)words * sizeof(u64),
                                      copy_kind(location, false), c->stream));
    if (written) *written = words;
    if (timed_out(c)) return COMET_ERR_TIMEOUT;    // what has been handed out is not the result
    return COMET_OK;
}

int comet_synchronize(comet_ctx* c) {
    if (!c) return COMET_ERR_INVALID_ARG;
    COMET_CUDA(c, cudaStreamSynchronize(c->stream));
    if (c->side) COMET_CUDA(c, cudaStreamSynchronize(c->side));
    std::atomic_thread_fence(std::memory_order_acquire);
    return timed_out(c) ? COMET_ERR_TIMEOUT : COMET_OK;
}

int comet_inject_timeout(comet_ctx* c) {
    if (!c) return COMET_ERR_INVALID_ARG;
    COMET_CUDA(c, cudaStreamSynchronize(c->stream));
    const int32_t one = 1;
    COMET_CUDA(c, cudaMemcpy(c->d_error, &one, sizeof(one), cudaMemcpyHostToDevice));
    c->h_count[3] = 1;
    return COMET_OK;
}

int comet_device_pointer(comet_ctx* c, int party, int tensor_id, uint64_t** out) {
    if (!c || !out || (party != 0 && party != 1)) return COMET_ERR_INVALID_ARG;
    if (tensor_id != COMET_Z_UP && tensor_id != COMET_Y) return COMET_ERR_INVALID_ARG;
    *out = reinterpret_cast<uint64_t*>(c->own[party][tensor_id]);
    return COMET_OK;
}

int comet_get_index(comet_ctx* c, int32_t* out, int location, int32_t capacity, int32_t* n_active_blocks_out) {
    if (!c || !out || !n_active_blocks_out) return COMET_ERR_INVALID_ARG;
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (!c->mask_set) return COMET_ERR_STATE;
    if (capacity < c->n_active_blocks) return COMET_ERR_SHAPE;
    if (c->n_active_blocks > 0)
        COMET_CUDA(c, cudaMemcpyAsync(out, c->d_ids, (size_t)c->n_active_blocks * sizeof(int32_t),
                                      copy_kind(location, false), c->stream));
    *n_active_blocks_out = c->n_active_blocks;
    return COMET_OK;
}

int comet_get_components(comet_ctx* c, int32_t* row_label, int32_t* blk_label, int location,
                         int32_t* n_components_out) {
    if (!c || !row_label || !blk_label || !n_components_out) return COMET_ERR_INVALID_ARG;
    if (location != COMET_DEVICE && location != COMET_HOST) return COMET_ERR_INVALID_ARG;
    if (!c->mask_set || !c->tmask_set) return COMET_ERR_STATE;
    COMET_CUDA(c, cudaMemcpyAsync(row_label, c->d_row_label, (size_t)c->tmask_tokens * sizeof(int32_t),
                                  copy_kind(location, false), c->stream));
    COMET_CUDA(c, cudaMemcpyAsync(blk_label, c->d_blk_label, (size_t)c->n_active_blocks * sizeof(int32_t),
                                  copy_kind(location, false), c->stream));
    *n_components_out = c->n_components;
    return COMET_OK;
}

int comet_stats(comet_ctx* c, comet_stats_t* out) {
    if (!c || !out) return COMET_ERR_INVALID_ARG;
    if (!c->pending->empty()) {
        COMET_CUDA(c, cudaStreamSynchronize(c->stream));
        for (auto& p : *c->pending) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, p.start, p.stop) == cudaSuccess) {
                c->stats.phase_ms[p.phase] += ms;
                c->stats.phase_launches[p.phase] += p.launches;
            }
            c->free_events->push_back(p.start);
            c->free_events->push_back(p.stop);
        }
        c->pending->clear();
        cudaGetLastError();
    }
    *out = c->stats;
    return COMET_OK;
}

int comet_set_profiling(comet_ctx* c, int on) {
    if (!c) return COMET_ERR_INVALID_ARG;
    comet_stats_t tmp;
    const int rc = comet_stats(c, &tmp);      // drain what is pending
    if (rc != COMET_OK) return rc;
    c->profiling = on != 0;
    if (c->profiling)
        for (int k = 0; k < COMET_NUM_PHASES; ++k) {
            c->stats.phase_ms[k] = 0.0;
            c->stats.phase_launches[k] = 0;
        }
    return COMET_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Allocation-free Pi_MatMul: the message buffers live in the library image.
// ---------------------------------------------------------------------------
namespace {

// Scratch for E_0, E_1, F_0, F_1 of comet_beaver_matmul_static.  In host code
// this name is only a handle for cudaGetSymbolAddress, never an address to hand
// to a kernel; each GPU that loads the library carries its own 8 MiB copy.
static __device__ __align__(256) unsigned long long g_static_scratch[COMET_STATIC_SCRATCH_WORDS];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
u64* g_static_scratch_addr[kMaxDevices] = {};    // device address of the array, per device ordinal

// Device address of the scratch array on the current device (looked up once per device).
cudaError_t static_scratch_on_current_device(u64** out) {
    int dev = -1;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        err = cudaGetSymbolAddress(&p, g_static_scratch);
        if (err != cudaSuccess) return err;
        g_static_scratch_addr[dev] = static_cast<u64*>(p);
    }
    *out = g_static_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int comet_beaver_matmul_static(void* cuda_stream, const uint64_t* const X[2], const uint64_t* const A[2],
                                          const uint64_t* const Y[2], const uint64_t* const B[2],
                                          const uint64_t* const C[2], uint64_t* const Z[2], int32_t T, int32_t K,
                                          int32_t N) {
    if (!X || !A || !Y || !B || !C || !Z) return COMET_ERR_INVALID_ARG;
    for (int p = 0; p < 2; ++p)
        if (!X[p] || !A[p] || !Y[p] || !B[p] || !C[p] || !Z[p]) return COMET_ERR_INVALID_ARG;
    // the kernels below read and write every operand 16 bytes at a time
    for (int p = 0; p < 2; ++p) {
        const void* ptrs[6] = {X[p], A[p], Y[p], B[p], C[p], Z[p]};
        for (const void* q : ptrs)
            if ((reinterpret_cast<uintptr_t>(q) & 15u) != 0) return COMET_ERR_INVALID_ARG;
    }
    if (T < 1 || K < 8 || N < 4 || K % 8 || N % 4) return COMET_ERR_SHAPE;
    const int64_t left = (int64_t)T * K, right = (int64_t)N * K;
    if (2 * (left + right) > (int64_t)COMET_STATIC_SCRATCH_WORDS) return COMET_ERR_SCRATCH_LIMIT;

    u64* scratch = nullptr;
    if (static_scratch_on_current_device(&scratch) != cudaSuccess) {
        cudaGetLastError();
        return COMET_ERR_CUDA;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // carve the array: E_0 | E_1 | F_0 | F_1 (every word used below is written before it is read)
    u64* E[2] = {scratch, scratch + left};
    u64* F[2] = {scratch + 2 * left, scratch + 2 * left + right};

    comet::PartyPtrs x, a, y, b;
    comet::PartyOut e, f;
    comet::CombineArgs args;
    for (int p = 0; p < 2; ++p) {
        x.p[p] = reinterpret_cast<const u64*>(X[p]);
        a.p[p] = reinterpret_cast<const u64*>(A[p]);
        y.p[p] = reinterpret_cast<const u64*>(Y[p]);
        b.p[p] = reinterpret_cast<const u64*>(B[p]);
        e.p[p] = E[p];
        f.p[p] = F[p];
        args.E[p] = E[p];
        args.F[p] = F[p];
        args.A[p] = a.p[p];
        args.B[p] = b.p[p];
        args.C[p] = reinterpret_cast<const u64*>(C[p]);
        args.Z[p] = reinterpret_cast<u64*>(Z[p]);
    }
    args.M = T; args.N = N; args.K = K;
    args.tmask = nullptr; args.tmask_ld = 0; args.bs = 1;
    auto blocks = [](int64_t pairs) { return (unsigned)((pairs + 255) / 256 < 1184 ? (pairs + 255) / 256 : 1184); };
    comet::open_activation_kernel<<<dim3(blocks(left / 2), 2), 256, 0, stream>>>(x, a, e, left / 2, nullptr, 0, K, 1);
    comet::open_activation_kernel<<<dim3(blocks(right / 2), 2), 256, 0, stream>>>(y, b, f, right / 2, nullptr, 0, K, 1);
    dim3 grid((N + comet::simt::BN - 1) / comet::simt::BN, (T + comet::simt::BM - 1) / comet::simt::BM, 2);
    comet::combine_simt_kernel<<<grid, comet::simt::THREADS, 0, stream>>>(args);
    if (cudaGetLastError() != cudaSuccess) return COMET_ERR_CUDA;
    return COMET_OK;
}

// ---------------------------------------------------------------------------
// Oblivious shuffle (Protocol 1), online stage.  Stateless: no context, no
// memory of its own.
// ---------------------------------------------------------------------------
namespace {

int shuffle_grid(long long items) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    long long want = (items + 255) / 256, cap = (long long)sms * 16;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// out_i = in_i[perm_i] +/- mask_i for both parties, one launch
int launch_shuffle_step(cudaStream_t stream, const uint64_t* const in[2], const int32_t* const perm[2],
                        const uint64_t* const mask[2], uint64_t* const out[2], int64_t rows, int64_t cols,
                        int subtract, int32_t* bad) {
    comet::ShuffleArgs a;
    bool vec = (cols % 2) == 0;
    for (int p = 0; p < 2; ++p) {
        a.in[p] = reinterpret_cast<const u64*>(in[p]);
        a.perm[p] = perm[p];
        a.mask[p] = reinterpret_cast<const u64*>(mask[p]);
        a.out[p] = reinterpret_cast<u64*>(out[p]);
        vec = vec && aligned16(in[p]) && aligned16(mask[p]) && aligned16(out[p]);
    }
    a.rows = rows;
    a.pieces = (int)(vec ? cols / 2 : cols);
    a.subtract = subtract;
    a.bad_index = bad;
    const int grid = shuffle_grid(rows * a.pieces);
    const long long stride = (long long)grid * 256;
    a.stride_rows = stride / a.pieces;
    a.stride_pieces = (int)(stride % a.pieces);
    if (vec) comet::shuffle_rows_kernel<ulonglong2><<<dim3(grid, 2), 256, 0, stream>>>(a);
    else comet::shuffle_rows_kernel<u64><<<dim3(grid, 2), 256, 0, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? COMET_OK : COMET_ERR_CUDA;
}

}  // namespace

extern "C" int comet_shuffle(void* cuda_stream, const uint64_t* const X[2], const int32_t* const tau[2],
                             const int32_t* const rho[2], const uint64_t* const a[2], const uint64_t* const b[2],
                             uint64_t* const Y[2], uint64_t* const Z[2], int64_t rows, int64_t cols,
                             int32_t* bad_index_flag) {
    if (!X || !tau || !rho || !a || !b || !Y || !Z) return COMET_ERR_INVALID_ARG;
    for (int p = 0; p < 2; ++p)
        if (!X[p] || !tau[p] || !rho[p] || !a[p] || !b[p] || !Y[p] || !Z[p]) return COMET_ERR_INVALID_ARG;
    if (rows < 1 || cols < 1 || rows > 0x7fffffffll || cols > 0x7fffffffll) return COMET_ERR_SHAPE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // [y]_i = tau_i([x]_i) + a_i
    int rc = launch_shuffle_step(stream, X, tau, a, Y, rows, cols, 0, bad_index_flag);
    if (rc != COMET_OK) return rc;
    // the exchange: party i reads what the other party wrote.  [z]_i = rho_i([y]_other) - b_i
    const uint64_t* const received[2] = {Y[1], Y[0]};
    return launch_shuffle_step(stream, received, rho, b, Z, rows, cols, 1, bad_index_flag);
}

extern "C" int comet_invert_permutation(void* cuda_stream, const int32_t* perm, int32_t* inverse, int64_t rows,
                                        int32_t* bad_index_flag) {
    if (!perm || !inverse) return COMET_ERR_INVALID_ARG;
    if (rows < 1 || rows > 0x7fffffffll) return COMET_ERR_SHAPE;
    comet::invert_permutation_kernel<<<shuffle_grid(rows), 256, 0, (cudaStream_t)cuda_stream>>>(perm, inverse, rows,
                                                                                                  bad_index_flag);
    return cudaGetLastError() == cudaSuccess ? COMET_OK : COMET_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Element-wise Beaver product (Eq. 1 element by element).  Stateless.
// ---------------------------------------------------------------------------
extern "C" int comet_beaver_mul(void* cuda_stream, const uint64_t* const X[2], const uint64_t* const Y[2],
                                const uint64_t* const A[2], const uint64_t* const B[2], const uint64_t* const C[2],
                                uint64_t* const D[2], uint64_t* const E[2], uint64_t* const Z[2], int64_t count) {
    if (!X || !Y || !A || !B || !C || !D || !E || !Z) return COMET_ERR_INVALID_ARG;
    for (int p = 0; p < 2; ++p)
        if (!X[p] || !Y[p] || !A[p] || !B[p] || !C[p] || !D[p] || !E[p] || !Z[p]) return COMET_ERR_INVALID_ARG;
    if (count < 1) return COMET_ERR_SHAPE;
    comet::MulArgs g;
    bool vec = (count % 2) == 0;
    for (int p = 0; p < 2; ++p) {
        g.x[p] = reinterpret_cast<const u64*>(X[p]); g.y[p] = reinterpret_cast<const u64*>(Y[p]);
        g.a[p] = reinterpret_cast<const u64*>(A[p]); g.b[p] = reinterpret_cast<const u64*>(B[p]);
        g.c[p] = reinterpret_cast<const u64*>(C[p]);
        g.d[p] = reinterpret_cast<u64*>(D[p]); g.e[p] = reinterpret_cast<u64*>(E[p]);
        g.z[p] = reinterpret_cast<u64*>(Z[p]);
        vec = vec && aligned16(X[p]) && aligned16(Y[p]) && aligned16(A[p]) && aligned16(B[p]) && aligned16(C[p]) &&
              aligned16(D[p]) && aligned16(E[p]) && aligned16(Z[p]);
    }
    g.pieces = vec ? count / 2 : count;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const dim3 grid(shuffle_grid(g.pieces), 2);
    if (vec) {
        comet::beaver_mul_open_kernel<ulonglong2><<<grid, 256, 0, stream>>>(g);
        comet::beaver_mul_combine_kernel<ulonglong2><<<grid, 256, 0, stream>>>(g);      // after the exchange
    } else {
        comet::beaver_mul_open_kernel<u64><<<grid, 256, 0, stream>>>(g);
        comet::beaver_mul_combine_kernel<u64><<<grid, 256, 0, stream>>>(g);
    }
    return cudaGetLastError() == cudaSuccess ? COMET_OK : COMET_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Truncation with a dealer's pair: Section 2.1's Reconstruction and Addition.
// ---------------------------------------------------------------------------
extern "C" int comet_truncate_pair(void* cuda_stream, uint64_t* const Z[2], const uint64_t* const R[2],
                                   const uint64_t* const RP[2], uint64_t* const M[2], int64_t count,
                                   int32_t frac_bits) {
    if (!Z || !R || !RP || !M) return COMET_ERR_INVALID_ARG;
    for (int p = 0; p < 2; ++p)
        if (!Z[p] || !R[p] || !RP[p] || !M[p]) return COMET_ERR_INVALID_ARG;
    if (count < 1) return COMET_ERR_SHAPE;
    if (frac_bits < 1 || frac_bits > 31) return COMET_ERR_SHAPE;
    comet::TruncPairArgs g;
    bool vec = (count % 2) == 0;
    for (int p = 0; p < 2; ++p) {
        g.z[p] = reinterpret_cast<u64*>(Z[p]); g.m[p] = reinterpret_cast<u64*>(M[p]);
        g.r[p] = reinterpret_cast<const u64*>(R[p]); g.rp[p] = reinterpret_cast<const u64*>(RP[p]);
        vec = vec && aligned16(Z[p]) && aligned16(R[p]) && aligned16(RP[p]) && aligned16(M[p]);
    }
    g.pieces = vec ? count / 2 : count;
    g.f = frac_bits;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const dim3 grid(shuffle_grid(g.pieces), 2);
    if (vec) {
        comet::trunc_pair_open_kernel<ulonglong2><<<grid, 256, 0, stream>>>(g);
        comet::trunc_pair_combine_kernel<ulonglong2><<<grid, 256, 0, stream>>>(g);      // after the exchange
    } else {
        comet::trunc_pair_open_kernel<u64><<<grid, 256, 0, stream>>>(g);
        comet::trunc_pair_combine_kernel<u64><<<grid, 256, 0, stream>>>(g);
    }
    return cudaGetLastError() == cudaSuccess ? COMET_OK : COMET_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// KV-cache manager (Section 6): request merging and the prefetch rule.  Host logic.
// ---------------------------------------------------------------------------
extern "C" int comet_kv_plan(const uint8_t* present, const uint8_t* active, int32_t tokens, int32_t heads, int64_t x,
                             int64_t w, uint8_t* request, uint8_t* prefetch, int32_t* l1_out) {
    if (!present || !active || !request || !prefetch) return COMET_ERR_INVALID_ARG;
    if (tokens < 1 || heads < 1 || x < 1 || w < 1) return COMET_ERR_SHAPE;
    std::vector<int64_t> missing(heads, 0);
    int32_t l1 = 0;
    for (int32_t t = 0; t < tokens; ++t) {
        bool in_batch = false;
        for (int32_t h = 0; h < heads; ++h) {
            const bool miss = present[(size_t)t * heads + h] == 0;
            missing[h] += miss;
            const bool want = miss && active[h] != 0;
            request[(size_t)t * heads + h] = want ? 1 : 0;
            in_batch = in_batch || want;
        }
        l1 += in_batch;
    }
    for (int32_t h = 0; h < heads; ++h) {
        prefetch[h] = 0;
        if (active[h] != 0) continue;
        const int64_t l2 = missing[h], beyond = l2 > l1 ? l2 - l1 : 0;
        // saved 2*L2*x against spent 2*(w + x*max(0, L2 - L1)), in integers: L2 > w/x + max(0, L2 - L1)
        if (l2 * x > w + x * beyond) {
            prefetch[h] = 1;
            for (int32_t t = 0; t < tokens; ++t)
                if (present[(size_t)t * heads + h] == 0) request[(size_t)t * heads + h] = 1;
        }
    }
    if (l1_out) *l1_out = l1;
    return COMET_OK;
}

extern "C" int comet_add_bias(void* cuda_stream, uint64_t* const Z[2], const uint64_t* const bias[2], int64_t rows,
                              int64_t cols) {
    if (!Z || !bias || !Z[0] || !Z[1] || !bias[0] || !bias[1]) return COMET_ERR_INVALID_ARG;
    if (rows < 1 || cols < 1 || cols > 0x7fffffffll) return COMET_ERR_SHAPE;
    comet::BiasArgs g;
    for (int p = 0; p < 2; ++p) {
        g.z[p] = reinterpret_cast<u64*>(Z[p]);
        g.bias[p] = reinterpret_cast<const u64*>(bias[p]);
    }
    g.rows = rows;
    g.cols = (int)cols;
    comet::add_bias_kernel<<<dim3(shuffle_grid(rows * cols), 2), 256, 0, (cudaStream_t)cuda_stream>>>(g);
    return cudaGetLastError() == cudaSuccess ? COMET_OK : COMET_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Measured peak of a multiply pipe (support for the roofline; not a step of the path).
// ---------------------------------------------------------------------------
extern "C" int comet_pipe_probe(void* cuda_stream, int pipe, int32_t launches, int32_t work, float* ms_out,
                                double* macs_per_launch_out) {
    namespace pk = comet::peak;
    if (!ms_out || !macs_per_launch_out) return COMET_ERR_INVALID_ARG;
    if (pipe != COMET_PIPE_TENSOR_I8 && pipe != COMET_PIPE_ALU_U64) return COMET_ERR_INVALID_ARG;
    if (launches < 1 || launches > 4096 || work < 1 || work > (1 << 24)) return COMET_ERR_SHAPE;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return COMET_ERR_CUDA;
    }
    const int alu_blocks = sms * 2;
    const size_t sink_bytes = pipe == COMET_PIPE_TENSOR_I8 ? (size_t)sms * 32 * sizeof(unsigned) + sizeof(int)
                                                           : (size_t)alu_blocks * pk::ALU_THREADS * sizeof(u64);
    void* sink = nullptr;
    if (cudaMalloc(&sink, sink_bytes) != cudaSuccess) {
        cudaGetLastError();
        return COMET_ERR_OOM;
    }
    std::vector<cudaEvent_t> ev((size_t)launches + 1, nullptr);
    int rc = COMET_OK;
    for (auto& e : ev)
        if (cudaEventCreate(&e) != cudaSuccess) rc = COMET_ERR_CUDA;
    int* flag = reinterpret_cast<int*>(static_cast<char*>(sink) + (size_t)sms * 32 * sizeof(unsigned));
    if (rc == COMET_OK && cudaMemsetAsync(sink, 0, sink_bytes, stream) != cudaSuccess) rc = COMET_ERR_CUDA;
    if (rc == COMET_OK) {
        for (int i = 0; i < launches; ++i) {
            cudaEventRecord(ev[i], stream);
            if (pipe == COMET_PIPE_TENSOR_I8)
                comet::tensor_i8_probe_kernel<<<sms, pk::THREADS, 0, stream>>>(work, 0x9E3779B9u + i, flag,
                                                                                static_cast<unsigned*>(sink));
            else
                comet::alu_u64_probe_kernel<<<alu_blocks, pk::ALU_THREADS, 0, stream>>>(work, 0x9E3779B97F4A7C15ull + i,
                                                                                         static_cast<u64*>(sink));
        }
        cudaEventRecord(ev[launches], stream);
        if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(stream) != cudaSuccess) rc = COMET_ERR_CUDA;
    }
    if (rc == COMET_OK) {
        for (int i = 0; i < launches; ++i)
            if (cudaEventElapsedTime(&ms_out[i], ev[i], ev[i + 1]) != cudaSuccess) rc = COMET_ERR_CUDA;
        if (pipe == COMET_PIPE_TENSOR_I8) {
            int h_flag = 0;
            if (cudaMemcpy(&h_flag, flag, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = COMET_ERR_CUDA;
            else if (h_flag) rc = COMET_ERR_TIMEOUT;
            *macs_per_launch_out = (double)sms * work * pk::BATCH * ((double)pk::M * pk::N * pk::KC);
        } else {
            *macs_per_launch_out = (double)alu_blocks * pk::ALU_THREADS * pk::ALU_CHAINS * (double)work;
        }
    }
    for (auto e : ev)
        if (e) cudaEventDestroy(e);
    cudaFree(sink);
    if (rc == COMET_ERR_CUDA) cudaGetLastError();
    return rc;
}
