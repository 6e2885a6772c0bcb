// TEST INFRASTRUCTURE -- not part of the product.
//
// Plain, slow, single-threaded CPU statement of what the sparse secret-shared
// FFN path computes, written from the paper (arXiv 2505.07239, "Comet") in the
// paper's order and notation.  It shares no code with the CUDA library, is
// never tuned, and is only ever called by the tests, by the smoke check and by
// the benchmark's CPU-baseline leg.
//
// Ring: Z_{2^64}; every value is a uint64_t and C++ unsigned arithmetic is the
// ring arithmetic.  Matrices are row-major in the paper's mathematical shapes
// (X is [rows, inner], Y is [inner, cols]).  Parties: the paper's P_1, P_2 are
// i = 0, 1 here, so the paper's factor (i-1) in Eq. 1 is the factor i.
//
// Pins (see tests/test_oracle_*.py): Eq. 1 reconstructs the plaintext product
// for any triple with c = ab (checked against Python big integers and numpy);
// all-ones mask == dense; masked neurons contribute exactly zero; truncation
// closed forms and the {0,1}-ulp invariant; hand-computed fixtures.
// Parity unpinned: the individual share values Z_i (as opposed to their sum)
// are fixed only by Eq. 1 itself plus this repository's seeded inputs.
// SOMM over connected components (Protocol 2 in general): the partition is
// pinned by a library routine for connected components and by hand-made graphs,
// the result by the plaintext product on the component blocks, the costs by the
// counts of Theorem 1, and the whole by its reduction to the token-shared case.
// SIMM with per-column row sets R_j (Protocol 3 in general): pinned by the masked
// plaintext product, by its reduction to the token-shared case under an
// all-ones distribution, and by the counts of Theorem 2.
// Oblivious shuffle (Protocol 1): pinned by the paper's worked permutation
// example, by z_1 + z_2 = pi(x) against numpy indexing, by the operator
// identities rho_1 o tau_2 = rho_2 o tau_1 = pi, by exhaustive permutations of
// three elements and by unshuffle(shuffle(x)) = x.
// Truncation with a dealer's pair (not a protocol of the paper; built from its
// Reconstruction and Addition, Section 2.1): pinned by the closed forms r = 0 and
// "low f bits of z and r all zero", by the {-1,0}-ulp invariant against Python
// big integers, by [out]_0 = [r']_0 (the public term goes to the party with
// factor i), and by hand-computed words.  Parity unpinned by the paper itself.

#include <cstddef>
#include <cstdint>
#include <vector>

typedef uint64_t u64;

extern "C" {

// ---------------------------------------------------------------------------
// Section 2.1, "Additive secret sharing": reconstruction x = [x]_1 + [x]_2.
// ---------------------------------------------------------------------------
void orc_reconstruct(const u64* s0, const u64* s1, u64* out, size_t count) {
    for (size_t t = 0; t < count; ++t) out[t] = s0[t] + s1[t];
}

// ---------------------------------------------------------------------------
// Index sets.  Protocol 2's I_y of the single connected component and
// Protocol 3's nonzero columns j, for a sparsity distribution
// that is one block mask shared by all tokens: neuron j is active iff
// block_mask[j / bs] != 0.  With `groups` = 2 (gated FFN, Y = [W_gate || W_up]
// of width 2*D) the set is I followed by D + I.  Ascending order.
// Returns the number of indices written.
// ---------------------------------------------------------------------------
int orc_index_set(const uint8_t* block_mask, int nb, int bs, int groups, int32_t* I) {
    int D = nb * bs;
    int count = 0;
    for (int g = 0; g < groups; ++g)
        for (int j = 0; j < D; ++j)
            if (block_mask[j / bs] != 0) I[count++] = g * D + j;
    return count;
}

// Protocol 2: IndexCols(Y, I_y).  Y is [K, D]; out is [K, n].
void orc_index_cols(const u64* Y, int K, int D, const int32_t* I, int n, u64* out) {
    for (int k = 0; k < K; ++k)
        for (int c = 0; c < n; ++c) out[(size_t)k * n + c] = Y[(size_t)k * D + I[c]];
}

// Protocol 3: IndexRow(Y, j) for every j in I.  Y is [D, N]; out is [n, N].
void orc_index_rows(const u64* Y, int N, const int32_t* I, int n, u64* out) {
    for (int r = 0; r < n; ++r)
        for (int c = 0; c < N; ++c) out[(size_t)r * N + c] = Y[(size_t)I[r] * N + c];
}

// Protocol 2, Merge: compact columns back to a dense [T, D] layout,
// zero (in this share) at every inactive position.
void orc_merge_cols(const u64* R, int T, int n, const int32_t* I, int D, u64* Z) {
    for (size_t t = 0; t < (size_t)T * D; ++t) Z[t] = 0;
    for (int r = 0; r < T; ++r)
        for (int c = 0; c < n; ++c) Z[(size_t)r * D + I[c]] = R[(size_t)r * n + c];
}

// ---------------------------------------------------------------------------
// Pi_MatMul, the matrix form of Eq. 1, one party's side.
//
// Step 1 (before the exchange), Section 2.1 "Multiplication" / Section 5.1:
//   [E]_i = [X]_i - [A]_i,   [F]_i = [Y]_i - [B]_i.
// ---------------------------------------------------------------------------
void orc_mask_operand(const u64* share, const u64* mask_share, u64* out, size_t count) {
    for (size_t t = 0; t < count; ++t) out[t] = share[t] - mask_share[t];
}

// Plain ring product P = L * R, L [T,K], R [K,N] (accumulating row by row).
static void ring_product(const u64* L, const u64* R, int T, int K, int N, u64* P) {
    for (size_t t = 0; t < (size_t)T * N; ++t) P[t] = 0;
    for (int r = 0; r < T; ++r)
        for (int k = 0; k < K; ++k) {
            u64 l = L[(size_t)r * K + k];
            const u64* Rrow = R + (size_t)k * N;
            u64* Prow = P + (size_t)r * N;
            for (int c = 0; c < N; ++c) Prow[c] += l * Rrow[c];
        }
}

// Step 2 (after the exchange): E = [E]_0 + [E]_1 and F = [F]_0 + [F]_1 are
// public, and Eq. 1 with d -> E (left), e -> F (right) reads
//   [Z]_i = [C]_i + E * [B]_i + [A]_i * F + i * (E * F),
// three separate products, exactly as the equation is printed.
void orc_beaver_combine(int party, int T, int K, int N, const u64* E, const u64* F,
                        const u64* Ai, const u64* Bi, const u64* Ci, u64* Zi) {
    std::vector<u64> EB((size_t)T * N), AF((size_t)T * N), EF((size_t)T * N);
    ring_product(E, Bi, T, K, N, EB.data());
    ring_product(Ai, F, T, K, N, AF.data());
    ring_product(E, F, T, K, N, EF.data());
    for (size_t t = 0; t < (size_t)T * N; ++t)
        Zi[t] = Ci[t] + EB[t] + AF[t] + (u64)party * EF[t];
}

// The same Eq. 1 evaluated at a list of output positions only (one dot product
// triple per sample), for sizes where the full product is too slow on a CPU.
void orc_beaver_combine_at(int party, int K, int N, const u64* E, const u64* F,
                           const u64* Ai, const u64* Bi, const u64* Ci,
                           int n_samples, const int32_t* rows, const int32_t* cols, u64* out) {
    for (int s = 0; s < n_samples; ++s) {
        int r = rows[s], c = cols[s];
        u64 eb = 0, af = 0, ef = 0;
        for (int k = 0; k < K; ++k) {
            u64 e = E[(size_t)r * K + k], a = Ai[(size_t)r * K + k];
            u64 f = F[(size_t)k * N + c], b = Bi[(size_t)k * N + c];
            eb += e * b;
            af += a * f;
            ef += e * f;
        }
        out[s] = Ci[(size_t)r * N + c] + eb + af + (u64)party * ef;
    }
}

// Both parties of one Pi_MatMul call.  Inputs are pairs of shares (index 0/1).
// Outputs: the four messages and the two result shares.
void orc_pi_matmul(int T, int K, int N,
                   const u64* X0, const u64* X1, const u64* Y0, const u64* Y1,
                   const u64* A0, const u64* A1, const u64* B0, const u64* B1,
                   const u64* C0, const u64* C1,
                   u64* E0, u64* E1, u64* F0, u64* F1, u64* Z0, u64* Z1) {
    size_t nx = (size_t)T * K, ny = (size_t)K * N;
    orc_mask_operand(X0, A0, E0, nx);
    orc_mask_operand(X1, A1, E1, nx);
    orc_mask_operand(Y0, B0, F0, ny);
    orc_mask_operand(Y1, B1, F1, ny);
    std::vector<u64> E(nx), F(ny);
    orc_reconstruct(E0, E1, E.data(), nx);   // the exchange
    orc_reconstruct(F0, F1, F.data(), ny);
    orc_beaver_combine(0, T, K, N, E.data(), F.data(), A0, B0, C0, Z0);
    orc_beaver_combine(1, T, K, N, E.data(), F.data(), A1, B1, C1, Z1);
}

// ---------------------------------------------------------------------------
// Protocol 2 (SOMM) for a token-shared mask: the bipartite graph is complete
// between all T rows of X and the active columns, i.e. one connected
// component with I_x = all rows, I_y = I.  Y is [K, Dy] (Dy = groups * d_ff).
// Outputs are compact: messages E_i [T,K], F_i [K,n]; result R_i [T,n].
// ---------------------------------------------------------------------------
void orc_somm(int T, int K, int Dy, const int32_t* I, int n,
              const u64* X0, const u64* X1, const u64* Y0, const u64* Y1,
              const u64* A0, const u64* A1, const u64* B0, const u64* B1,
              const u64* C0, const u64* C1,
              u64* E0, u64* E1, u64* F0, u64* F1, u64* R0, u64* R1) {
    std::vector<u64> Yt0((size_t)K * n), Yt1((size_t)K * n);
    orc_index_cols(Y0, K, Dy, I, n, Yt0.data());          // IndexCols
    orc_index_cols(Y1, K, Dy, I, n, Yt1.data());
    orc_pi_matmul(T, K, n, X0, X1, Yt0.data(), Yt1.data(), // Pi_MatMul
                  A0, A1, B0, B1, C0, C1, E0, E1, F0, F1, R0, R1);
}

// ---------------------------------------------------------------------------
// Protocol 2, first step: the connected components {G_t} of the bipartite graph whose
// nodes are the T rows of X and the n (compact) columns of Y and whose edges are
// the non-zeros of the sparsity distribution S [T, n], found by depth-first
// search.  Components are numbered in the order in which a scan over the rows
// 0, 1, ... discovers them; row_comp / col_comp give each node's component, -1
// for a node without any edge.  Returns the number of components L.
// ---------------------------------------------------------------------------
int orc_components_dfs(int T, int n, const uint8_t* S, int32_t* row_comp, int32_t* col_comp) {
    for (int r = 0; r < T; ++r) row_comp[r] = -1;
    for (int c = 0; c < n; ++c) col_comp[c] = -1;
    int L = 0;
    std::vector<int> stack;                       // node ids: rows 0..T-1, columns T..T+n-1
    for (int start = 0; start < T; ++start) {
        if (row_comp[start] >= 0) continue;
        bool has_edge = false;
        for (int c = 0; c < n && !has_edge; ++c) has_edge = S[(size_t)start * n + c] != 0;
        if (!has_edge) continue;
        row_comp[start] = L;
        stack.assign(1, start);
        while (!stack.empty()) {
            const int node = stack.back();
            stack.pop_back();
            if (node < T) {
                for (int c = 0; c < n; ++c)
                    if (S[(size_t)node * n + c] != 0 && col_comp[c] < 0) {
                        col_comp[c] = L;
                        stack.push_back(T + c);
                    }
            } else {
                const int c = node - T;
                for (int r = 0; r < T; ++r)
                    if (S[(size_t)r * n + c] != 0 && row_comp[r] < 0) {
                        row_comp[r] = L;
                        stack.push_back(r);
                    }
            }
        }
        ++L;
    }
    return L;
}

// ---------------------------------------------------------------------------
// Protocol 2 (SOMM) in general.  Y is [K, Dy]; compact column c stands for
// column I[c] of Y; S is the sparsity distribution of the compact result [T, n].
// For every component: the index sets I_x, I_y, IndexRows / IndexCols,
// Pi_MatMul with that component's own triple, and Merge puts
// the result block at (I_x, I_y); every other entry of the result is zero in
// both shares, and rows / columns outside all components are neither masked nor
// sent (their message rows stay zero).  The per-component triples arrive
// stacked: A [T, K] holds in row r the mask row of r's component, B [K, n] in
// column c that of c's component, C [T, n] the blocks c^t = a^t b^t at (I_x, I_y)
// (whatever else C holds is ignored).
// cost[0] = rows and columns masked (Theorem 1's communication count, in rows /
// columns), cost[1] = dot products evaluated, sum_t |I_x||I_y|.
// Returns L.
// ---------------------------------------------------------------------------
int orc_somm_components(int T, int K, int Dy, const int32_t* I, int n, const uint8_t* S,
                        const u64* X0, const u64* X1, const u64* Y0, const u64* Y1,
                        const u64* A0, const u64* A1, const u64* B0, const u64* B1,
                        const u64* C0, const u64* C1,
                        u64* E0, u64* E1, u64* F0, u64* F1, u64* R0, u64* R1,
                        int32_t* row_comp, int32_t* col_comp, long long* cost) {
    const int L = orc_components_dfs(T, n, S, row_comp, col_comp);            // the components
    const u64* Xs[2] = {X0, X1};
    const u64* Ys[2] = {Y0, Y1};
    const u64* As[2] = {A0, A1};
    const u64* Bs[2] = {B0, B1};
    const u64* Cs[2] = {C0, C1};
    u64* Es[2] = {E0, E1};
    u64* Fs[2] = {F0, F1};
    u64* Rs[2] = {R0, R1};
    for (int i = 0; i < 2; ++i) {
        for (size_t t = 0; t < (size_t)T * K; ++t) Es[i][t] = 0;
        for (size_t t = 0; t < (size_t)K * n; ++t) Fs[i][t] = 0;
        for (size_t t = 0; t < (size_t)T * n; ++t) Rs[i][t] = 0;
    }
    cost[0] = cost[1] = 0;
    std::vector<int> Ix, Iy;
    for (int t = 0; t < L; ++t) {
        Ix.clear();
        Iy.clear();
        for (int r = 0; r < T; ++r) if (row_comp[r] == t) Ix.push_back(r);    // I_x, I_y
        for (int c = 0; c < n; ++c) if (col_comp[c] == t) Iy.push_back(c);
        const int tx = (int)Ix.size(), ty = (int)Iy.size();
        cost[0] += tx + ty;
        cost[1] += (long long)tx * ty;
        std::vector<u64> xt[2], yt[2], at[2], bt[2], ct[2], et[2], ft[2], rt[2];
        for (int i = 0; i < 2; ++i) {
            xt[i].resize((size_t)tx * K); at[i].resize((size_t)tx * K); et[i].resize((size_t)tx * K);
            yt[i].resize((size_t)K * ty); bt[i].resize((size_t)K * ty); ft[i].resize((size_t)K * ty);
            ct[i].resize((size_t)tx * ty); rt[i].resize((size_t)tx * ty);
            for (int a = 0; a < tx; ++a)                                     // IndexRows
                for (int k = 0; k < K; ++k) {
                    xt[i][(size_t)a * K + k] = Xs[i][(size_t)Ix[a] * K + k];
                    at[i][(size_t)a * K + k] = As[i][(size_t)Ix[a] * K + k];
                }
            for (int k = 0; k < K; ++k)                                      // IndexCols
                for (int b = 0; b < ty; ++b) {
                    yt[i][(size_t)k * ty + b] = Ys[i][(size_t)k * Dy + I[Iy[b]]];
                    bt[i][(size_t)k * ty + b] = Bs[i][(size_t)k * n + Iy[b]];
                }
            for (int a = 0; a < tx; ++a)
                for (int b = 0; b < ty; ++b) ct[i][(size_t)a * ty + b] = Cs[i][(size_t)Ix[a] * n + Iy[b]];
        }
        orc_pi_matmul(tx, K, ty, xt[0].data(), xt[1].data(), yt[0].data(), yt[1].data(),             // Pi_MatMul
                      at[0].data(), at[1].data(), bt[0].data(), bt[1].data(), ct[0].data(), ct[1].data(),
                      et[0].data(), et[1].data(), ft[0].data(), ft[1].data(), rt[0].data(), rt[1].data());
        for (int i = 0; i < 2; ++i) {                                        // Merge
            for (int a = 0; a < tx; ++a)
                for (int k = 0; k < K; ++k) Es[i][(size_t)Ix[a] * K + k] = et[i][(size_t)a * K + k];
            for (int k = 0; k < K; ++k)
                for (int b = 0; b < ty; ++b) Fs[i][(size_t)k * n + Iy[b]] = ft[i][(size_t)k * ty + b];
            for (int a = 0; a < tx; ++a)
                for (int b = 0; b < ty; ++b) Rs[i][(size_t)Ix[a] * n + Iy[b]] = rt[i][(size_t)a * ty + b];
        }
    }
    return L;
}

// ---------------------------------------------------------------------------
// Protocol 3 (SIMM), column by row.  X here is already compact, [T, n], its
// column c standing for neuron I[c]; R_j is all T rows for every nonzero
// column (token-shared mask).  Each column's Pi_MatMul is the outer product of
// a T-vector with row I[c] of Y [D, N]; it uses column c of A' [T,n] and row c
// of B' [n,N] as its (a_j, b_j), and the dealer's C' [T,N] is the sum over j
// of the per-column c_j = a_j b_j^T, added once in Merge&Sum.
// Outputs: messages E_i [T,n], F_i [n,N]; result Z_i [T,N].
// ---------------------------------------------------------------------------
void orc_simm(int T, int n, int N, const int32_t* I,
              const u64* X0, const u64* X1, const u64* Y0, const u64* Y1,
              const u64* A0, const u64* A1, const u64* B0, const u64* B1,
              const u64* C0, const u64* C1,
              u64* E0, u64* E1, u64* F0, u64* F1, u64* Z0, u64* Z1) {
    const u64* Xs[2] = {X0, X1};
    const u64* Ys[2] = {Y0, Y1};
    const u64* As[2] = {A0, A1};
    const u64* Bs[2] = {B0, B1};
    const u64* Cs[2] = {C0, C1};
    u64* Es[2] = {E0, E1};
    u64* Fs[2] = {F0, F1};
    u64* Zs[2] = {Z0, Z1};
    for (int i = 0; i < 2; ++i)
        for (size_t t = 0; t < (size_t)T * N; ++t) Zs[i][t] = Cs[i][t];
    std::vector<u64> e(T), f(N);
    for (int c = 0; c < n; ++c) {                    // the protocol's loop body, one column j = I[c]
        int j = I[c];
        for (int i = 0; i < 2; ++i) {
            for (int r = 0; r < T; ++r)              // IndexCol, IndexRows + masking of x''
                Es[i][(size_t)r * n + c] = Xs[i][(size_t)r * n + c] - As[i][(size_t)r * n + c];
            for (int q = 0; q < N; ++q)              // IndexRow + masking of y
                Fs[i][(size_t)c * N + q] = Ys[i][(size_t)j * N + q] - Bs[i][(size_t)c * N + q];
        }
        for (int r = 0; r < T; ++r) e[r] = E0[(size_t)r * n + c] + E1[(size_t)r * n + c];
        for (int q = 0; q < N; ++q) f[q] = F0[(size_t)c * N + q] + F1[(size_t)c * N + q];
        for (int i = 0; i < 2; ++i)                  // Pi_MatMul (Eq. 1 without c_j) + the sum of Merge&Sum
            for (int r = 0; r < T; ++r) {
                u64 a = As[i][(size_t)r * n + c];
                for (int q = 0; q < N; ++q) {
                    u64 b = Bs[i][(size_t)c * N + q];
                    Zs[i][(size_t)r * N + q] += e[r] * b + a * f[q] + (u64)i * (e[r] * f[q]);
                }
            }
    }
}

// ---------------------------------------------------------------------------
// Protocol 3 (SIMM) with a sparsity distribution S of X that differs from row
// to row: S is [T, n] over the compact columns (non-zero byte = X[r, c] is a
// non-zero), so R_j of compact column c is {r : S[r, c] != 0} (the protocol's first loop).
// A column with empty R_j is not a "nonzero column": nothing of it is masked,
// sent or multiplied, and its message rows stay zero.  For the others, only the
// entries of x'' = X[R_j, j] are masked and sent (E is zero off the support),
// row I[c] of Y is masked once, and the outer product of Eq. 1 is added into the
// rows in R_j (Merge&Sum).  a_j lives in A'[R_j, c] (whatever A' holds off the
// support is ignored); the dealer's C' is the sum over j of a_j b_j^T scattered
// to the rows R_j.  Returns the number of masked entries of X (the nnz of S).
// ---------------------------------------------------------------------------
long long orc_simm_rowsets(int T, int n, int N, const int32_t* I, const uint8_t* S,
                           const u64* X0, const u64* X1, const u64* Y0, const u64* Y1,
                           const u64* A0, const u64* A1, const u64* B0, const u64* B1,
                           const u64* C0, const u64* C1,
                           u64* E0, u64* E1, u64* F0, u64* F1, u64* Z0, u64* Z1) {
    const u64* Xs[2] = {X0, X1};
    const u64* Ys[2] = {Y0, Y1};
    const u64* As[2] = {A0, A1};
    const u64* Bs[2] = {B0, B1};
    const u64* Cs[2] = {C0, C1};
    u64* Es[2] = {E0, E1};
    u64* Fs[2] = {F0, F1};
    u64* Zs[2] = {Z0, Z1};
    for (int i = 0; i < 2; ++i) {
        for (size_t t = 0; t < (size_t)T * N; ++t) Zs[i][t] = Cs[i][t];
        for (size_t t = 0; t < (size_t)T * n; ++t) Es[i][t] = 0;
        for (size_t t = 0; t < (size_t)n * N; ++t) Fs[i][t] = 0;
    }
    long long masked = 0;
    std::vector<int> R;
    std::vector<u64> e, f(N);
    for (int c = 0; c < n; ++c) {
        R.clear();
        for (int r = 0; r < T; ++r)
            if (S[(size_t)r * n + c] != 0) R.push_back(r);         // R_j
        if (R.empty()) continue;                                    // not a nonzero column
        const int j = I[c];
        masked += (long long)R.size();
        e.assign(R.size(), 0);
        for (int i = 0; i < 2; ++i) {
            for (size_t k = 0; k < R.size(); ++k)                   // IndexCol, IndexRows + masking of x''
                Es[i][(size_t)R[k] * n + c] = Xs[i][(size_t)R[k] * n + c] - As[i][(size_t)R[k] * n + c];
            for (int q = 0; q < N; ++q)                             // IndexRow + masking of y
                Fs[i][(size_t)c * N + q] = Ys[i][(size_t)j * N + q] - Bs[i][(size_t)c * N + q];
        }
        for (size_t k = 0; k < R.size(); ++k) e[k] = E0[(size_t)R[k] * n + c] + E1[(size_t)R[k] * n + c];
        for (int q = 0; q < N; ++q) f[q] = F0[(size_t)c * N + q] + F1[(size_t)c * N + q];
        for (int i = 0; i < 2; ++i)                                 // Pi_MatMul and the sum of Merge&Sum
            for (size_t k = 0; k < R.size(); ++k) {
                const u64 a = As[i][(size_t)R[k] * n + c];
                for (int q = 0; q < N; ++q) {
                    const u64 b = Bs[i][(size_t)c * N + q];
                    Zs[i][(size_t)R[k] * N + q] += e[k] * b + a * f[q] + (u64)i * (e[k] * f[q]);
                }
            }
    }
    return masked;
}

// ---------------------------------------------------------------------------
// Local fixed-point truncation by f bits (the paper is silent; two-party local
// truncation on the unsigned words): party 0 shifts its share logically,
// party 1 negates, shifts logically and negates again.
// ---------------------------------------------------------------------------
void orc_truncate(int party, const u64* in, u64* out, size_t count, int f) {
    for (size_t t = 0; t < count; ++t) {
        if (party == 0) out[t] = in[t] >> f;
        else out[t] = (u64)0 - (((u64)0 - in[t]) >> f);
    }
}

// ---------------------------------------------------------------------------
// Section 4.2, "Oblivious shuffle".  A permutation pi acts on a vector as the
// paper's example fixes it: pi = [2,1,3] gives pi(x) = [x_2, x_1, x_3], i.e.
// (pi(x))_j = x_{pi_j} (indices 0-based here).  The shuffled objects are the
// `rows` rows of a [rows, cols] matrix of ring words.
// ---------------------------------------------------------------------------
void orc_apply_permutation(const int32_t* perm, const u64* x, u64* out, int rows, int cols) {
    for (int j = 0; j < rows; ++j)
        for (int c = 0; c < cols; ++c) out[(size_t)j * cols + c] = x[(size_t)perm[j] * cols + c];
}

// p o q as an operator: (p o q)(x) = p(q(x)).  (p(q(x)))_j = (q(x))_{p_j} = x_{q_{p_j}}.
void orc_compose_permutations(const int32_t* p, const int32_t* q, int32_t* out, int rows) {
    for (int j = 0; j < rows; ++j) out[j] = q[p[j]];
}

void orc_invert_permutation(const int32_t* p, int32_t* out, int rows) {
    for (int j = 0; j < rows; ++j) out[p[j]] = j;
}

// Protocol 1, offline stage (the trusted third party): given pi, tau_1, tau_2 and the
// random a_1, a_2, c it derives rho_1 = pi o tau_2^{-1}, rho_2 = pi o tau_1^{-1},
// b_1 = rho_1(a_2) + c and b_2 = rho_2(a_1) - c.  Party index 0/1 = the paper's 1/2.
void orc_shuffle_offline(int rows, int cols, const int32_t* pi, const int32_t* tau0, const int32_t* tau1,
                         const u64* a0, const u64* a1, const u64* c,
                         int32_t* rho0, int32_t* rho1, u64* b0, u64* b1) {
    std::vector<int32_t> inv(rows);
    orc_invert_permutation(tau1, inv.data(), rows);
    orc_compose_permutations(pi, inv.data(), rho0, rows);
    orc_invert_permutation(tau0, inv.data(), rows);
    orc_compose_permutations(pi, inv.data(), rho1, rows);
    const size_t count = (size_t)rows * cols;
    orc_apply_permutation(rho0, a1, b0, rows, cols);
    orc_apply_permutation(rho1, a0, b1, rows, cols);
    for (size_t t = 0; t < count; ++t) {
        b0[t] = b0[t] + c[t];
        b1[t] = b1[t] - c[t];
    }
}

// Protocol 1, online stage, both parties: [y]_i = tau_i([x]_i) + a_i is sent to the
// other party, which computes [z]_i = rho_i([y]_{other}) - b_i.
void orc_shuffle_online(int rows, int cols, const u64* x0, const u64* x1,
                        const int32_t* tau0, const int32_t* tau1, const int32_t* rho0, const int32_t* rho1,
                        const u64* a0, const u64* a1, const u64* b0, const u64* b1,
                        u64* y0, u64* y1, u64* z0, u64* z1) {
    const size_t count = (size_t)rows * cols;
    orc_apply_permutation(tau0, x0, y0, rows, cols);
    orc_apply_permutation(tau1, x1, y1, rows, cols);
    for (size_t t = 0; t < count; ++t) {
        y0[t] = y0[t] + a0[t];
        y1[t] = y1[t] + a1[t];
    }
    orc_apply_permutation(rho0, y1, z0, rows, cols);      // party 0 works on what party 1 sent
    orc_apply_permutation(rho1, y0, z1, rows, cols);
    for (size_t t = 0; t < count; ++t) {
        z0[t] = z0[t] - b0[t];
        z1[t] = z1[t] - b1[t];
    }
}

// ---------------------------------------------------------------------------
// Section 2.1, "Multiplication", Eq. 1 taken element by element (the product
// ReLU(gate) * up of a gated FFN is of this kind): for every element,
// [d]_i = [x]_i - [a]_i and [e]_i = [y]_i - [b]_i are exchanged, d and e
// reconstructed, and [z]_i = [c]_i + d*[b]_i + e*[a]_i + i*d*e.
// ---------------------------------------------------------------------------
void orc_beaver_mul(size_t count, const u64* x0, const u64* x1, const u64* y0, const u64* y1,
                    const u64* a0, const u64* a1, const u64* b0, const u64* b1, const u64* c0, const u64* c1,
                    u64* d0, u64* d1, u64* e0, u64* e1, u64* z0, u64* z1) {
    const u64* xs[2] = {x0, x1};
    const u64* ys[2] = {y0, y1};
    const u64* as[2] = {a0, a1};
    const u64* bs[2] = {b0, b1};
    const u64* cs[2] = {c0, c1};
    u64* ds[2] = {d0, d1};
    u64* es[2] = {e0, e1};
    u64* zs[2] = {z0, z1};
    for (int i = 0; i < 2; ++i)
        for (size_t t = 0; t < count; ++t) {
            ds[i][t] = xs[i][t] - as[i][t];
            es[i][t] = ys[i][t] - bs[i][t];
        }
    for (size_t t = 0; t < count; ++t) {
        const u64 d = d0[t] + d1[t], e = e0[t] + e1[t];
        for (int i = 0; i < 2; ++i) zs[i][t] = cs[i][t] + d * bs[i][t] + e * as[i][t] + (u64)i * (d * e);
    }
}

// ---------------------------------------------------------------------------
// Section 2.1, "Addition": adding a secret-shared vector is local, each party
// adds its own share.  Here a shared bias [N] is added to every row of a shared
// matrix [T, N] (both at the same fixed-point scale).
// ---------------------------------------------------------------------------
void orc_add_bias(int T, int N, const u64* Zi, const u64* bias_i, u64* out) {
    for (int r = 0; r < T; ++r)
        for (int c = 0; c < N; ++c) out[(size_t)r * N + c] = Zi[(size_t)r * N + c] + bias_i[c];
}

// ---------------------------------------------------------------------------
// Truncation by f bits with a dealer's pair.  The paper has no truncation
// protocol; this one is put together from two of its primitives (Section 2.1):
// the dealer shares a uniform word r and r' = floor(r / 2^f) (r read as a signed
// 64-bit integer); "Reconstruction" opens m = z - r from the messages
// [m]_i = [z]_i - [r]_i; "Addition" with the public value c = floor(m / 2^f)
// (m read as signed) gives [out]_i = [r']_i + i*c.
// out_0 + out_1 = floor(m/2^f) + floor(r/2^f), which is floor(z/2^f) or one less
// unless m + r leaves the signed range (probability about |z| / 2^64).
// ---------------------------------------------------------------------------
void orc_truncate_pair(size_t count, int f, const u64* z0, const u64* z1, const u64* r0, const u64* r1,
                       const u64* rp0, const u64* rp1, u64* m0, u64* m1, u64* out0, u64* out1) {
    for (size_t t = 0; t < count; ++t) {
        m0[t] = z0[t] - r0[t];
        m1[t] = z1[t] - r1[t];
    }
    for (size_t t = 0; t < count; ++t) {
        const u64 m = m0[t] + m1[t];                        // reconstruction
        // floor division of the signed reading by 2^f, written without relying on >> of a negative value
        const bool neg = (m >> 63) != 0;
        const u64 c = neg ? ~((~m) >> f) : (m >> f);
        out0[t] = rp0[t];                                   // i = 0: no public term
        out1[t] = rp1[t] + c;                               // i = 1 adds the public value
    }
}

}  // extern "C"
