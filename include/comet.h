/*
 * comet.h -- C ABI of the B200 library for the per-party local arithmetic of the
 * sparsity-aware secret-shared feed-forward layer (Comet, arXiv 2505.07239).
 *
 * Both parties of a 2-party additive sharing over Z_{2^64} are simulated on one
 * GPU; the "messages" the two servers would exchange are device buffers owned by
 * the context.  A party's kernels read only that party's shares and the two
 * message buffers.
 *
 * Conventions
 *   - Every word is a uint64_t ring element; arithmetic is mod 2^64.
 *   - Left operands are row-major [tokens, inner].  Right operands (weights,
 *     their masks B and the messages F) are stored OUTPUT-FEATURE-MAJOR, i.e.
 *     as the transpose of the paper's matrix: W1 and WG are [d_ff, d_model],
 *     W2 is [d_model, d_ff], B_UP is [g*n, d_model], B_DN is [d_model, n].
 *     (n = active neurons, g = 1 + `gated` = matrices stacked in the up-projection.)
 *   - Compact column c of the up-projection stands for neuron I[c mod n], I the
 *     ascending list of neurons in active blocks; for g = 2 columns [0,n) are
 *     the gate projection (WG) and [n,2n) the up projection (W1); for g = 3 columns
 *     [2n,3n) belong to W3.
 *   - Parties are 0 and 1 (the paper's P_1, P_2); party 1 carries the public
 *     product term of Eq. 1.
 *   - Every call returns COMET_OK or a negative error code; nothing traps or
 *     aborts, and no exception crosses the ABI.  Arguments are validated on the
 *     host before anything is launched.
 *   - Pointers passed in belong to the caller.  `location` says where they
 *     point: COMET_DEVICE (memory of the context's GPU) or COMET_HOST (pinned or
 *     pageable host memory).  The library copies what it is given into memory
 *     it allocated at comet_init; nothing of the caller's is kept (the one
 *     exception is comet_bind_shares, which reads the caller's device memory in
 *     place).
 *   - All work is enqueued on the CUDA stream given to comet_init.  Calls are
 *     asynchronous with respect to the host except comet_set_mask with a DEVICE
 *     mask and comet_set_token_mask (they return public counts computed on the
 *     device), comet_get/comet_load_shares with host pointers to pageable
 *     memory, comet_synchronize, comet_stats and comet_destroy.
 */
#ifndef COMET_H_
#define COMET_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct comet_ctx comet_ctx;

enum {
    COMET_OK = 0,
    COMET_ERR_INVALID_ARG = -1, /* null pointer, unknown id, bad party / location       */
    COMET_ERR_SHAPE = -2,       /* sizes disagree with the configuration or the mask    */
    COMET_ERR_STATE = -3,       /* call out of order (e.g. ffn_up before its inputs)    */
    COMET_ERR_OOM = -4,         /* device allocation failed in comet_init               */
    COMET_ERR_CUDA = -5,        /* a CUDA runtime call failed; see comet_last_cuda_error */
    COMET_ERR_TIMEOUT = -6,     /* a bounded device-side wait ran out                   */
    COMET_ERR_SCRATCH_LIMIT = -7 /* problem too large for the built-in static scratch array */
};

enum { COMET_DEVICE = 0, COMET_HOST = 1 };

/* matmul_path */
enum {
    COMET_PATH_AUTO = 0,   /* the path the measurements favour                              */
    COMET_PATH_SIMT = 1,   /* 64-bit multiply-add on the integer ALUs                         */
    COMET_PATH_LIMB = 2    /* 8-bit limb planes on the int8 tensor cores, recombined mod 2^64 */
};

/* Tensor ids.  "in" tensors are set with comet_load_shares, "out" tensors are
 * produced by the library; every id can be read back with comet_get.  Shapes
 * are [rows, cols] as stored (see Conventions). */
enum {
    COMET_X = 0,      /* in : activations                [T, d_model]           */
    COMET_W1 = 1,     /* in : up (or fc1) weights        [d_ff, d_model]        */
    COMET_WG = 2,     /* in : gate weights (gated only)  [d_ff, d_model]        */
    COMET_W2 = 3,     /* in : down (or fc2) weights      [d_model, d_ff]        */
    COMET_A_UP = 4,   /* in : triple, masks X            [T, d_model]           */
    COMET_B_UP = 5,   /* in : triple, masks W[:, I]      [g*n, d_model]         */
    COMET_C_UP = 6,   /* in : triple, C = A B            [T, g*n]               */
    COMET_H = 7,      /* in : post-activation hidden     [T, n]                 */
    COMET_A_DN = 8,   /* in : triple, masks H            [T, n]                 */
    COMET_B_DN = 9,   /* in : triple, masks W2[I, :]     [d_model, n]           */
    COMET_C_DN = 10,  /* in : triple                     [T, d_model]           */
    COMET_E_UP = 11,  /* out: message X_i - A_i          [T, d_model]           */
    COMET_F_UP = 12,  /* out: message W_i[:, I] - B_i    [g*n, d_model]  (after a product with at most 32
                         tokens on the tensor-core path the messages F exist as limb planes; comet_get
                         rebuilds the words)                                  */
    COMET_Z_UP = 13,  /* out: up-projection share        [T, g*n]               */
    COMET_E_DN = 14,  /* out: message H_i - A'_i         [T, n]                 */
    COMET_F_DN = 15,  /* out: message W2_i[I, :] - B'_i  [d_model, n]           */
    COMET_Y = 16,     /* out: down-projection share      [T, d_model]           */
    COMET_W3 = 17,    /* in : third weight matrix (gated = 2 only) [d_ff, d_model] */
    COMET_NUM_TENSORS = 18
};

typedef struct {
    int32_t max_tokens;   /* capacity in token rows (T of any later call <= this)       */
    int32_t d_model;      /* multiple of 16                                             */
    int32_t d_ff;         /* multiple of `block`                                        */
    int32_t block;        /* neurons per mask block, multiple of 16                     */
    int32_t frac_bits;    /* fixed-point fractional bits f, 1..31                       */
    int32_t gated;        /* weight matrices of the up-projection that share the mask, minus one:
                             0: W1 alone, Y = act(X W1) W2;  1: [WG || W1], a gated FFN;
                             2: [WG || W1 || W3], e.g. the query, key and value projections of an
                             attention layer under a head mask (block = head size, d_ff = heads *
                             head size, W2 = the output projection): X is still opened once      */
    int32_t device;       /* CUDA device ordinal                                        */
    int32_t max_active;   /* capacity in active neurons, 0 = d_ff                       */
    int32_t matmul_path;  /* COMET_PATH_*                                               */
} comet_config;

/* phases of the path, for the per-phase timers of comet_stats */
enum {
    COMET_PHASE_COMPACT = 0,  /* mask compaction                                   */
    COMET_PHASE_OPEN = 1,     /* E_i = X_i - A_i and F_i = gather(W_i) - B_i        */
    COMET_PHASE_PREP = 2,     /* operand preparation after the exchange (limb path) */
    COMET_PHASE_COMBINE = 3,  /* the gathered ring matmul + Beaver combine          */
    COMET_PHASE_TRUNCATE = 4, /* local truncation                                   */
    COMET_NUM_PHASES = 5
};

typedef struct {
    int64_t message_bytes;   /* bytes of E_i and F_i written by the last ffn_up/ffn_down, both parties:
                                2 * 8 * (T*K + K*N), the communication cost C_1 of the optimality proof */
    int64_t ring_macs;       /* 64-bit multiply-adds of the last ffn_up/ffn_down, both parties: 2 * 2*T*K*N;
                                for ffn_up under a token mask on the tensor-core path with more than 32 tokens,
                                Theorem 1's count: 2 * 2*K * sum over components of rows x columns */
    int32_t n_active;        /* active neurons under the current mask                            */
    int32_t n_active_blocks;
    int32_t tokens;          /* T of the last ffn call                                           */
    int32_t matmul_path;     /* path actually used by the last ffn call                          */
    int64_t kernel_launches; /* kernels launched by this context since comet_init                */
    /* filled only while profiling is on (comet_set_profiling): device time and launch
       count per phase since profiling was switched on, from CUDA events on the stream */
    double phase_ms[COMET_NUM_PHASES];
    int64_t phase_launches[COMET_NUM_PHASES];
    int32_t n_components;    /* connected components under the current token mask (0 without one) */
    int32_t reserved;
    int64_t tensor_tile_macs; /* 64-bit multiply-adds the tensor-core kernel of the last ffn call covered, counted
                                 in whole output tiles (128 x 64, or 32 tokens x 128 for at most 32 tokens) and
                                 32-deep steps, both parties (0 on the CUDA-core path): under a token mask with
                                 several components only the tiles and steps that meet a component */
} comet_stats_t;

/* Create a context: validates the configuration, selects the device, and
 * allocates every buffer the later calls use (shares, triples, messages,
 * results) for the stated capacities.  `cuda_stream` is a cudaStream_t (NULL =
 * the default stream) on which all calls are ordered.  The tensor-core path
 * also owns one internal non-blocking stream, forked from and joined back into
 * `cuda_stream` with events, on which comet_ffn_up opens the weight side of the
 * down-projection early when W2 and B_DN are already loaded.
 * Errors: INVALID_ARG, SHAPE (divisibility rules above), OOM, CUDA. */
int comet_init(const comet_config* config, void* cuda_stream, comet_ctx** out);

/* Release everything comet_init allocated (synchronises the stream first). */
void comet_destroy(comet_ctx* ctx);

/* Section 2.1 / Section 3.3: each server holds its additive share of the input,
 * of the weights, and of the dealer's correlated randomness.  Copies `rows*cols`
 * words of party `party`'s share of tensor `tensor_id` (an "in" id) into the
 * context.  Triples and H are sized by the current mask, so they are loaded
 * after comet_set_mask; a shape that disagrees with the configuration or with
 * the mask is COMET_ERR_SHAPE.  Loading X, A_UP or H fixes T for the next ffn
 * call. */
int comet_load_shares(comet_ctx* ctx, int party, int tensor_id, const uint64_t* ptr, int location,
                      int64_t rows, int64_t cols);

/* As comet_load_shares, but nothing is copied: the library reads party `party`'s
 * share of `tensor_id` in place from `dev_ptr` (device memory of the context's GPU,
 * 16-byte aligned, rows*cols words) whenever a later call needs it.  The caller
 * keeps the memory valid and unchanged until the last call that uses the tensor
 * has completed on the stream (for a triple: the ffn call; for weights: as long as
 * they stay bound).  A later comet_load_shares or comet_bind_shares of the same
 * tensor replaces the binding; comet_set_mask drops the bindings of the triples
 * and of H like their loaded state.  Same shape rules and errors as
 * comet_load_shares, plus INVALID_ARG for an unaligned pointer. */
int comet_bind_shares(comet_ctx* ctx, int party, int tensor_id, const uint64_t* dev_ptr, int64_t rows, int64_t cols);

/* The index-set steps of Protocol 2 and Protocol 3 under a block mask shared by all
 * tokens: turn the plaintext sparsity distribution (one byte per block, non-zero
 * = active) into the ascending list of active blocks, i.e. the index set I.
 * `n_blocks` must equal d_ff / block.  Returns the number of active NEURONS in
 * *n_active_out (the sparsity level is public in the threat model of Section
 * 3.2).  With a HOST mask the library counts the active blocks itself, copies
 * the bytes out of a pinned slot of its own (the caller's buffer may be reused
 * at once) and returns without waiting for the device; with a DEVICE mask the
 * count comes back from the compaction kernel through mapped host memory,
 * which the call waits for.  Zero active blocks is legal.  Invalidates
 * previously loaded triples and H.  Errors: INVALID_ARG, SHAPE (n_blocks; more
 * active neurons than max_active), CUDA, TIMEOUT (an earlier kernel of the
 * context gave up on a bounded wait). */
int comet_set_mask(comet_ctx* ctx, const uint8_t* block_mask, int location, int32_t n_blocks,
                   int32_t* n_active_out);

/* Protocol 2 (SOMM) specialised to one connected component, with Pi_MatMul as
 * the matrix form of Eq. 1: for both parties E_i = X_i - A_i,
 * F_i = W_i[:, I] - B_i (column gather of the paper = row gather of the stored
 * transpose), then after the exchange Z_i = C_i + E B_i + A_i F + i E F over the
 * active columns only, at scale 2f.  Needs X, W1 (and WG), A_UP, B_UP, C_UP.
 * Result in COMET_Z_UP; messages in COMET_E_UP / COMET_F_UP.  With n = 0 it does
 * nothing.
 * On the tensor-core path the call also starts on the down-projection with what
 * is loaded already: with W2 and B_DN it opens that product's weight side
 * (COMET_F_DN), and with C_DN as well it copies C'_i into COMET_Y, the value the
 * down-projection's sums are added to.  So from this call on COMET_F_DN and
 * COMET_Y no longer hold the previous step's values: read those back (or enqueue
 * the comet_get) before the next comet_ffn_up. */
int comet_ffn_up(comet_ctx* ctx, int32_t tokens);

/* Protocols 2 and 3 in general: the sparsity distribution may differ from token to
 * token.  One call sets it for both projections.
 *
 * Up-projection, Protocol 2: the connected components of the bipartite graph
 * (tokens) x (active blocks) are found on the GPU (minimum-label propagation
 * instead of the paper's depth-first search; the partition is the same), each
 * token row and each weight column is opened once (rows / blocks without any
 * edge not at all: their message words are zero), and comet_ffn_up leaves in
 * COMET_Z_UP the result blocks of the components, with every entry whose token
 * and block lie in different components zero in both shares (Merge).  The
 * per-component triples are passed stacked: row r of COMET_A_UP is the mask row
 * of r's component, row c of COMET_B_UP that of c's, COMET_C_UP holds a^t b^t
 * on the blocks (its other words are ignored).  Communication is Theorem 1's
 * minimum.  On the tensor-core path with 33 to 32768 tokens, when there are
 * several components or rows / blocks in none, the products of all components
 * are ONE launch over the component-sorted operands that computes only the
 * 128 x 64 output tiles which meet a component (a separate product for every
 * component, at tile granularity; comet_stats.ring_macs is then Theorem 1's
 * count, tensor_tile_macs what the tiles cover); otherwise one product over
 * [tokens, g*n], masked afterwards.  The shares are the same bits either way.
 *
 * Down-projection, Protocol 3 (its row sets R_j): the sparsity distribution of the hidden
 * state.  `token_mask` is [tokens, n_active_blocks]
 * bytes, row-major; byte (t, b) non-zero means that the neurons of the b-th ACTIVE
 * block (in the ascending order of comet_get_index) are non-zeros of token t, so
 * R_j = {t : token_mask[t, block(j)] != 0}.  It refines the block mask of
 * comet_set_mask (which must precede it and should be the union of the token
 * masks) and applies to the comet_ffn_down calls that follow, until the next
 * comet_set_mask or until it is cleared with token_mask = NULL, tokens = 0,
 * n_active_blocks = 0; comet_ffn_up and comet_ffn_down must then be called with
 * the same `tokens`.  Under a token mask comet_ffn_down opens only the
 * non-zero entries (E'_i is zero elsewhere: those words are not part of the
 * message; likewise the rows of F'_i that belong to an active block no token
 * uses) and ignores whatever COMET_H and COMET_A_DN hold off the support;
 * the dealer's C' is sum_j a_j b_j^T scattered to the rows R_j, i.e.
 * (mask * A') B'.  Communication is Theorem 2's minimum.  Under the same
 * conditions as for the up-projection, rows and contraction index are taken in
 * component order and every tile of 128 rows runs over the blocks of its own
 * components only; otherwise the product runs over [tokens, n].
 * comet_stats.ring_macs is Theorem 2's count either way, tensor_tile_macs what
 * the tiles cover.  *masked_out (may be NULL) receives the number of non-zero
 * entries (neurons, summed over tokens); one kernel, one report of seven words
 * through mapped host memory and a stream synchronise.  Errors: STATE (no block mask yet), SHAPE
 * (tokens out of range, n_active_blocks not the current count), INVALID_ARG. */
int comet_set_token_mask(comet_ctx* ctx, const uint8_t* token_mask, int location, int32_t tokens,
                         int32_t n_active_blocks, int64_t* masked_out);

/* The partition found by comet_set_token_mask: row_label[t] (tokens entries) and
 * blk_label[b] (one per active block) hold the smallest token index of the node's
 * component, -1 for a node without an edge; *n_components_out the number of
 * components.  Errors: STATE (no token mask), INVALID_ARG. */
int comet_get_components(comet_ctx* ctx, int32_t* row_label, int32_t* blk_label, int location,
                         int32_t* n_components_out);

/* Protocol 3 (SIMM) with R_j = all tokens for every active column j, so that
 * Merge&Sum of the per-column products is one matmul with inner size n:
 * E'_i = H_i - A'_i, F'_i = W2_i[I, :] - B'_i, Y_i = C'_i + E' B'_i + A'_i F' +
 * i E' F'.  Needs H, W2, A_DN, B_DN, C_DN.  Result in COMET_Y.  With n = 0 both
 * parties' Y is all zero. */
int comet_ffn_down(comet_ctx* ctx, int32_t tokens);

/* Local fixed-point truncation by f bits, in place, of COMET_Z_UP or COMET_Y for
 * both parties (the paper does not describe truncation; this is the two-party
 * local rule): party 0: s -> s >> f (logical); party 1: s -> -((-s) >> f). */
int comet_truncate(comet_ctx* ctx, int tensor_id);

/* Copy party `party`'s copy of any tensor to caller memory.  `capacity` is in
 * words and must cover the tensor's current size; the number of words written
 * is returned in *written (may be NULL). */
int comet_get(comet_ctx* ctx, int party, int tensor_id, uint64_t* out, int location, int64_t capacity,
              int64_t* written);

/* Device address of the library's own buffer of a RESULT tensor (COMET_Z_UP or
 * COMET_Y) of party `party`, valid until comet_destroy; the tensor's current
 * contents are its first rows*cols words.  For steps that combine results in
 * place between two calls of the path -- when the active neurons are sharded
 * over several GPUs, every GPU's comet_ffn_down leaves a partial sum of Eq. 1
 * in COMET_Y, the partial sums are added over the GPUs (addition of shares is
 * local, Section 2.1 "Addition"; an integer all-reduce, which wraps mod 2^64),
 * and comet_truncate then runs on the sum.  Whatever touches the buffer must be
 * ordered after the producing call and before the next consuming call on the
 * context's stream.  Errors: INVALID_ARG. */
int comet_device_pointer(comet_ctx* ctx, int party, int tensor_id, uint64_t** out);

/* The compacted index list: ascending ids of the active blocks (int32).
 * `capacity` in entries; the count goes to *n_active_blocks_out. */
int comet_get_index(comet_ctx* ctx, int32_t* out, int location, int32_t capacity, int32_t* n_active_blocks_out);

/* Counters of the last calls.  Synchronises nothing unless profiling is on, in
 * which case it waits for the stream and folds the pending event pairs into
 * phase_ms / phase_launches. */
int comet_stats(comet_ctx* ctx, comet_stats_t* out);

/* Switch the per-phase CUDA-event timers on (non-zero) or off; switching on
 * clears phase_ms / phase_launches.  While on, every phase of every call is
 * bracketed by two events recorded on the context's stream. */
int comet_set_profiling(comet_ctx* ctx, int on);

/* Wait for everything this context has enqueued (its stream and its internal
 * stream) and report whether any of its kernels gave up on a bounded wait.
 * Every device-side wait of the tensor-core kernels (on a copy, on the tensor
 * pipe, on the accumulators) ends after about two seconds; the kernel then lets
 * its copies in flight land, frees its tensor memory, returns, and writes an
 * error word that the host reads here.  COMET_ERR_TIMEOUT means that a result
 * of this context holds only part of its sums.  The word is never cleared: a
 * context that has timed out is to be destroyed.  comet_set_mask and comet_get
 * report the same condition as soon as they see it (comet_get does not wait
 * for the copy it enqueues, so only a comet_synchronize after it is a
 * guarantee for that copy).  Errors: INVALID_ARG, CUDA, TIMEOUT. */
int comet_synchronize(comet_ctx* ctx);

/* Test hook: marks the context as if one of its kernels had given up on a
 * bounded wait (it waits for the stream, then sets the error words such a
 * kernel would have set).  Nothing is launched.  It lets a caller exercise its
 * handling of COMET_ERR_TIMEOUT without any kernel actually waiting. */
int comet_inject_timeout(comet_ctx* ctx);

/* Text for an error code; never NULL. */
const char* comet_strerror(int code);

/* cudaError_t of the last failing runtime call of this context (0 if none). */
int comet_last_cuda_error(comet_ctx* ctx);

/* ---------------------------------------------------------------------------
 * Oblivious shuffle, Section 4.2, Protocol 1, online stage, for both parties.
 * It is the step on either side of the sparse FFN: the input matrix is shuffled
 * into the secret order of the revealed sparsity distribution before the
 * up-projection, and the output is unshuffled after the down-projection.
 *
 * A permutation p acts on the ROWS of a [rows, cols] matrix of ring words as the
 * paper's example fixes it, (p(x))[j] = x[p[j]] (0-based).  Party i holds its
 * share X[i], its sub-permutations tau[i], rho[i] (int32, `rows` entries each,
 * with pi = rho_0 o tau_1 = rho_1 o tau_0) and the dealer's masks a[i], b[i]
 * ([rows, cols]; b_0 = rho_0(a_1) + c, b_1 = rho_1(a_0) - c).  The call computes
 *     Y[i] = tau_i(X[i]) + a[i]          (the message party i sends), then
 *     Z[i] = rho_i(Y[1-i]) - b[i]        (party i's share of pi(x)).
 * Unshuffle is the same call with the sub-permutations each party derives
 * locally, tau'_i = rho_i^{-1} and rho'_i = tau_i^{-1} (comet_invert_permutation),
 * and fresh masks.
 *
 * Stateless: no context and no memory of the library's own.  Every pointer is a
 * DEVICE pointer on the current device, owned by the caller; X, a, b are only
 * read, Y and Z are overwritten and must not overlap any other argument.  Two
 * kernels are enqueued on `cuda_stream` (NULL = default stream); the call does
 * not wait for them.  16-byte accesses are used when cols is even and X, a, b,
 * Y, Z are 16-byte aligned, 8-byte accesses otherwise.
 * A permutation entry outside [0, rows) is never followed: the row it would
 * have fetched counts as zero and, if `bad_index_flag` (device int32, may be
 * NULL) is given, it is set to 1.  The caller clears the flag.
 * Errors: INVALID_ARG (null pointer), SHAPE (rows or cols < 1 or >= 2^31), CUDA. */
int comet_shuffle(void* cuda_stream, const uint64_t* const X[2], const int32_t* const tau[2],
                  const int32_t* const rho[2], const uint64_t* const a[2], const uint64_t* const b[2],
                  uint64_t* const Y[2], uint64_t* const Z[2], int64_t rows, int64_t cols, int32_t* bad_index_flag);

/* inverse[perm[j]] = j for j in [0, rows): the local step by which a party turns
 * its (rho_i, tau_i) into the sub-permutations of the unshuffle (Section 4.2,
 * remark (ii)).  Device pointers; entries outside [0, rows) are skipped and
 * reported through `bad_index_flag` as above. */
int comet_invert_permutation(void* cuda_stream, const int32_t* perm, int32_t* inverse, int64_t rows,
                             int32_t* bad_index_flag);

/* Section 2.1 "Addition": a secret-shared bias is added locally, each party adding its
 * own share: Z[i][r, :] += bias[i] for every row r, in place, for both parties.
 * DEVICE pointers on the current device, Z[i] of rows*cols words, bias[i] of cols
 * words, at the same fixed-point scale.  One kernel on `cuda_stream`; stateless.
 * Errors: INVALID_ARG (null pointer), SHAPE (rows or cols < 1), CUDA. */
int comet_add_bias(void* cuda_stream, uint64_t* const Z[2], const uint64_t* const bias[2], int64_t rows, int64_t cols);

/* Truncation by frac_bits with a dealer's pair, for both parties, in place.  The
 * paper has no truncation protocol; this one consists of two of its primitives
 * (Section 2.1): the dealer shares a uniform word r and r' = floor(r / 2^f), r
 * read as a signed 64-bit integer; "Reconstruction" opens m = z - r from the
 * messages M[i] = Z[i] - R[i]; "Addition" of the public value floor(m / 2^f), m
 * read as signed, to the shares of r' gives Z[i] <- RP[i] + i * floor(m / 2^f).
 * Z[0] + Z[1] afterwards is floor(z / 2^f) or one less, unless m + r leaves the
 * signed 64-bit range (probability about |z| / 2^64).  The alternative to
 * comet_truncate, which needs no dealer material and no message.
 * Stateless; DEVICE pointers on the current device to `count` words each, owned
 * by the caller; R, RP are only read, Z is replaced, M is overwritten and must not
 * overlap the others.  Two kernels on `cuda_stream`; the call does not wait.
 * Errors: INVALID_ARG (null pointer), SHAPE (count < 1, frac_bits outside [1, 31]), CUDA. */
int comet_truncate_pair(void* cuda_stream, uint64_t* const Z[2], const uint64_t* const R[2],
                        const uint64_t* const RP[2], uint64_t* const M[2], int64_t count, int32_t frac_bits);

/* ---------------------------------------------------------------------------
 * KV-cache manager, Section 6: which cache entries to compute together with the
 * current token.  Host logic only (HOST pointers, no GPU work): the result is a
 * per-token mask over heads, exactly what comet_set_token_mask takes for the
 * sparse QKV product, so that every token and every head takes part once
 * (Section 6.1, merging).
 *   present [tokens, heads]  non-zero = the (token, head) key/value is cached
 *   active  [heads]          non-zero = head activated for the current token
 *   x, w                     token vector size and size of one head's weight
 *                            matrix, in words (OPT-6.7B: 4096 and 4096*128)
 * request [tokens, heads] (out) gets 1 for every absent entry of an activated
 * head and of every prefetched head; prefetch [heads] (out) gets 1 for the heads
 * that are not activated but are worth refilling now by the rule of Section 6.2,
 * L2 > w/x + max(0, L2 - L1), L2 the head's absent entries and L1 the number of
 * tokens the merged refill of the activated heads sends anyway.  *l1_out (may be
 * NULL) receives L1.  Errors: INVALID_ARG (null pointer), SHAPE (sizes < 1). */
int comet_kv_plan(const uint8_t* present, const uint8_t* active, int32_t tokens, int32_t heads, int64_t x, int64_t w,
                  uint8_t* request, uint8_t* prefetch, int32_t* l1_out);

/* ---------------------------------------------------------------------------
 * Element-wise Beaver product, Section 2.1 "Multiplication", Eq. 1 applied to
 * every element (in a gated FFN: ReLU(gate) times up), for both parties:
 *     D[i] = X[i] - A[i],  E[i] = Y[i] - B[i]            (the two messages), then
 *     Z[i] = C[i] + d*B[i] + e*A[i] + i*d*e,  d = D[0]+D[1], e = E[0]+E[1],
 * element by element mod 2^64, with an element-wise triple c = a*b.  The result
 * is at scale 2f when both factors are at scale f; truncate it afterwards.
 * Stateless; all pointers are DEVICE pointers on the current device to `count`
 * words each, owned by the caller; D, E, Z are overwritten and must not overlap
 * the inputs.  Two kernels are enqueued on `cuda_stream`; the call does not wait.
 * Errors: INVALID_ARG (null pointer), SHAPE (count < 1), CUDA. */
int comet_beaver_mul(void* cuda_stream, const uint64_t* const X[2], const uint64_t* const Y[2],
                     const uint64_t* const A[2], const uint64_t* const B[2], const uint64_t* const C[2],
                     uint64_t* const D[2], uint64_t* const E[2], uint64_t* const Z[2], int64_t count);

/* ---------------------------------------------------------------------------
 * Allocation-free Pi_MatMul.  (The paper has no counterpart; this exists for
 * deployment reasons only.)
 *
 * Some hosts of this library must not, or cannot, allocate device memory at
 * the moment they need a product: a serving process whose framework has
 * already handed all of the GPU's memory to its own pool (a raw cudaMalloc
 * then fails or fights the pool), or a latency-critical loop in which
 * cudaMalloc/cudaFree would stall the whole device.  comet_init allocates, so
 * it is closed to them.  This one call needs no context and allocates nothing,
 * on the host or on the device: it runs one dense Beaver matrix product for
 * both parties,
 *     E_i = X_i - A_i,  F_i = Y_i - B_i,  Z_i = C_i + E B_i + A_i F + i E F,
 * and keeps the four message buffers E_0, E_1, F_0, F_1 -- the only memory the
 * product needs beyond its inputs and outputs -- in an array that is part of
 * the library image itself.  That array is COMET_STATIC_SCRATCH_WORDS 64-bit
 * words (8 MiB); every GPU on which the library is used holds it from the
 * moment the library is loaded there until the process exits.
 *
 * All pointers are DEVICE pointers on the CURRENT device, owned by the caller:
 * X[i], A[i] are [T, K]; Y[i], B[i] are [N, K] (output-feature-major, like the
 * weights above); C[i], Z[i] are [T, N]; i = 0, 1 is the party.  K must be a
 * multiple of 8 and N a multiple of 4, and every one of the twelve pointers
 * must be 16-byte aligned (the kernels move two words at a time; a pointer
 * carved out of a pool at an odd word is refused with INVALID_ARG before
 * anything is launched).  The work is enqueued on `cuda_stream`
 * (NULL = default stream) and the call returns without waiting for it.
 *
 * Limit: 2 * (T*K + N*K) <= COMET_STATIC_SCRATCH_WORDS, otherwise nothing is
 * launched and COMET_ERR_SCRATCH_LIMIT is returned.  Other errors: INVALID_ARG
 * (null or unaligned pointer), SHAPE (non-positive size or the divisibility
 * rule), CUDA.
 *
 * The first call on each device looks up the device address of the array
 * (once per device; no allocation).  Make that first call outside any stream
 * capture.
 *
 * The array is shared by every call in the process and is never cleared:
 * a call overwrites all of the part it uses before reading it, so stale
 * contents are harmless, but two calls whose work overlaps in time on the same
 * GPU (different streams, or different host threads) race on it.  Serialise
 * them, e.g. by using one stream.
 */
#define COMET_STATIC_SCRATCH_WORDS (1u << 20)
int comet_beaver_matmul_static(void* cuda_stream, const uint64_t* const X[2], const uint64_t* const A[2],
                               const uint64_t* const Y[2], const uint64_t* const B[2], const uint64_t* const C[2],
                               uint64_t* const Z[2], int32_t T, int32_t K, int32_t N);

/* ---------------------------------------------------------------------------
 * Measured peak of a multiply pipe.  (Not an operation of the paper: it supports
 * the roofline the benchmark reports, whose compute leg is "multiply-adds at the
 * measured peak of the chosen multiply pipe".)
 *
 * COMET_PIPE_TENSOR_I8: one CTA per SM issues `work` batches of 32
 *   tcgen05.mma kind::i8 instructions (M 128 x N 256 x K 32, u8 x u8 -> s32) on
 *   operand tiles that stay in shared memory, accumulators in tensor memory --
 *   the instruction the limb-plane kernel runs on, without any memory traffic.
 * COMET_PIPE_ALU_U64: two CTAs of 1024 threads per SM run `work` rounds of eight
 *   independent 64-bit multiply-add chains per thread -- the inner loop of the
 *   CUDA-core kernel without its loads.
 * `launches` such kernels are enqueued back to back on `cuda_stream` (NULL =
 * default stream) of the current device, each bracketed by CUDA events, and the
 * call waits for them.  ms_out[launches] (HOST) receives the duration of each
 * launch in milliseconds, *macs_per_launch_out the 8-bit (tensor) or 64-bit
 * (ALU) multiply-adds one launch performs; the first launches show the burst
 * rate, later ones the rate the power limit sustains.  A ring multiply-add
 * costs 36 of the 8-bit ones.  Allocates a small sink buffer and the events for
 * the duration of the call.  Errors: INVALID_ARG, SHAPE (launches outside
 * [1, 4096], work outside [1, 2^24]), OOM, CUDA, TIMEOUT (a bounded wait of the
 * tensor probe ran out). */
enum { COMET_PIPE_TENSOR_I8 = 0, COMET_PIPE_ALU_U64 = 1 };
int comet_pipe_probe(void* cuda_stream, int pipe, int32_t launches, int32_t work, float* ms_out,
                     double* macs_per_launch_out);

#ifdef __cplusplus
}
#endif
#endif /* COMET_H_ */
