/*
 * CPU oracle for inference through a fully-connected layer pruned by matrix
 * pivoting (PBP form).  TEST INFRASTRUCTURE ONLY: it exists to check the CUDA
 * library and to be timed as a CPU baseline.  It shares no code, header, table
 * or helper with the CUDA path and must never be called from the product path.
 *
 * Everything is fp64 and written as the plain definition:
 *
 *   Eq. 1   M_sparse = P_row * M_block * P_col.  With index arrays that map a
 *           pivoted index to an original index (Section 4.1.4: gathering "abc"
 *           with [2,0,1] gives "cab"; Listing 1 fetches a_in[P_col[.]] and
 *           stores to a_out[P_row[.]]) this reads
 *               W[row_perm[i]][col_perm[j]] = W_piv[i][j].
 *   Eq. 2   a_out = P_row (M_block (P_col a_in)): gather, block product,
 *           scatter.  ppo_structured_forward evaluates it in exactly that order,
 *           ppo_reconstruct + ppo_dense_forward evaluate the left-hand side
 *           (dense W times x); the two must agree.
 *
 * Conventions where the paper is silent: sizes not divisible by B are padded in
 * pivoted space (phantom rows with row_perm[i] >= M are dropped, phantom
 * columns with col_perm[j] >= N read x as 0); tiles that share a block-row add
 * up (Section 4.1.5); a block-row with no tile yields act(bias); bias is in
 * original row order and is added before the activation.
 *
 * Pinned by tests/test_oracle_pins.py: a 4x4 example worked by hand, the
 * "cab" index-array convention, brute-force P^T W_piv P products on tiny
 * sizes, identity permutations at density 1 against a library matmul, B = 1
 * against an element-wise sparse sum, and Eq. 2 against Eq. 1.  The irregular
 * block form (ppo_reconstruct_blocks, Section 4.1.5) is pinned by a second 4x4
 * example worked by hand, by explicit permutation-matrix products on random
 * rectangles and by its agreement with the uniform-tile form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define PPO_OK 0
#define PPO_BAD_PERM 1
#define PPO_BAD_TILE 2
#define PPO_BAD_ARG 3

static int is_bijection(const int32_t* p, int64_t n) {
    unsigned char* seen = (unsigned char*)calloc((size_t)(n > 0 ? n : 1), 1);
    int ok = 1;
    for (int64_t k = 0; k < n && ok; ++k) {
        if (p[k] < 0 || p[k] >= n || seen[p[k]]) ok = 0; else seen[p[k]] = 1;
    }
    free(seen);
    return ok;
}

static int check_layer(int M, int N, int B, const int32_t* row_perm, const int32_t* col_perm,
                       const int32_t* tile_list, int64_t T) {
    if (M <= 0 || N <= 0 || B <= 0 || T < 0) return PPO_BAD_ARG;
    int64_t Mb = (M + B - 1) / B, Nb = (N + B - 1) / B;
    if (!is_bijection(row_perm, Mb * B) || !is_bijection(col_perm, Nb * B)) return PPO_BAD_PERM;
    unsigned char* seen = (unsigned char*)calloc((size_t)(Mb * Nb), 1);
    int rc = PPO_OK;
    for (int64_t t = 0; t < T && rc == PPO_OK; ++t) {
        int64_t br = tile_list[2 * t], bc = tile_list[2 * t + 1];
        if (br < 0 || br >= Mb || bc < 0 || bc >= Nb || seen[br * Nb + bc]) rc = PPO_BAD_TILE;
        else seen[br * Nb + bc] = 1;
    }
    free(seen);
    return rc;
}

/* Eq. 1: dense W (M x N, row-major, zero where no tile lands). */
int ppo_reconstruct(int M, int N, int B, const int32_t* row_perm, const int32_t* col_perm,
                    const int32_t* tile_list, int64_t T, const double* tile_values, double* W) {
    int rc = check_layer(M, N, B, row_perm, col_perm, tile_list, T);
    if (rc != PPO_OK) return rc;
    memset(W, 0, sizeof(double) * (size_t)M * (size_t)N);
    for (int64_t t = 0; t < T; ++t) {
        int64_t br = tile_list[2 * t], bc = tile_list[2 * t + 1];
        for (int r = 0; r < B; ++r) {
            for (int c = 0; c < B; ++c) {
                int64_t I = row_perm[br * B + r];
                int64_t J = col_perm[bc * B + c];
                if (I < M && J < N) W[I * N + J] = tile_values[(t * B + r) * B + c];
            }
        }
    }
    return PPO_OK;
}

/* Eq. 1 with the irregular block structure of Section 4.1.5: M_block holds
 * rectangles of any size.  Block k covers pivoted rows [r0, r0+h) and pivoted
 * columns [c0, c0+w) (blocks[4k..4k+3] = r0, c0, h, w); its values follow those
 * of block k-1 in block_values, row-major h x w.  Blocks may share rows (their
 * products add up) but no element of M_block belongs to two blocks.  Mp, Np are
 * the lengths of the index arrays (pivoted sizes, >= M, N). */
int ppo_reconstruct_blocks(int M, int N, int Mp, int Np, const int32_t* row_perm, const int32_t* col_perm,
                           const int32_t* blocks, int64_t nb, const double* block_values, double* W) {
    if (M <= 0 || N <= 0 || Mp < M || Np < N || nb < 0) return PPO_BAD_ARG;
    if (!is_bijection(row_perm, Mp) || !is_bijection(col_perm, Np)) return PPO_BAD_PERM;
    unsigned char* taken = (unsigned char*)calloc((size_t)Mp * (size_t)Np, 1);
    memset(W, 0, sizeof(double) * (size_t)M * (size_t)N);
    int rc = PPO_OK;
    int64_t v = 0;
    for (int64_t k = 0; k < nb && rc == PPO_OK; ++k) {
        int64_t r0 = blocks[4 * k], c0 = blocks[4 * k + 1], h = blocks[4 * k + 2], w = blocks[4 * k + 3];
        if (r0 < 0 || c0 < 0 || h <= 0 || w <= 0 || r0 + h > Mp || c0 + w > Np) { rc = PPO_BAD_TILE; break; }
        for (int64_t r = 0; r < h && rc == PPO_OK; ++r) {
            for (int64_t c = 0; c < w; ++c, ++v) {
                int64_t i = r0 + r, j = c0 + c;
                if (taken[i * Np + j]) { rc = PPO_BAD_TILE; break; }
                taken[i * Np + j] = 1;
                int64_t I = row_perm[i], J = col_perm[j];
                if (I < M && J < N) W[I * N + J] = block_values[v];
            }
        }
    }
    free(taken);
    return rc;
}

static double activate(double s, int act) { return (act == 1 && s < 0.0) ? 0.0 : s; }

/* y = act(W x + b) for a dense W; also the pre-activation s and the magnitude
 * a_i = sum_j |W_ij| |x_j| that scales the comparison tolerance.
 * x, y, s, a are [batch][N] / [batch][M] row-major.  s and a may be NULL. */
void ppo_dense_forward(int M, int N, const double* W, const double* bias, const double* x,
                       int batch, int act, double* y, double* s_out, double* a_out, int threads) {
    if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int b = 0; b < batch; ++b) {
            double s = 0.0, a = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                double w = W[i * N + j], v = x[(int64_t)b * N + j];
                s += w * v;
                a += fabs(w) * fabs(v);
            }
            if (bias) s += bias[i];
            if (s_out) s_out[(int64_t)b * M + i] = s;
            if (a_out) a_out[(int64_t)b * M + i] = a;
            y[(int64_t)b * M + i] = activate(s, act);
        }
    }
}

/* Same as ppo_dense_forward but only for the listed original rows (sampled
 * checks at sizes where the full product is too slow). out arrays are [batch][n_rows]. */
void ppo_dense_forward_rows(int M, int N, const double* W, const double* bias, const double* x,
                            int batch, int act, const int32_t* rows, int n_rows,
                            double* y, double* a_out) {
    (void)M;
    for (int k = 0; k < n_rows; ++k) {
        int64_t i = rows[k];
        for (int b = 0; b < batch; ++b) {
            double s = 0.0, a = 0.0;
            for (int64_t j = 0; j < N; ++j) {
                double w = W[i * N + j], v = x[(int64_t)b * N + j];
                s += w * v;
                a += fabs(w) * fabs(v);
            }
            if (bias) s += bias[i];
            y[(int64_t)b * n_rows + k] = activate(s, act);
            if (a_out) a_out[(int64_t)b * n_rows + k] = a;
        }
    }
}

/* Eq. 2, in the paper's order: x_piv = P_col x (gather), y_piv = M_block x_piv
 * (tile by tile, tiles of one block-row add up), y = P_row y_piv (scatter),
 * then bias and activation in original order. */
int ppo_structured_forward(int M, int N, int B, const int32_t* row_perm, const int32_t* col_perm,
                           const int32_t* tile_list, int64_t T, const double* tile_values,
                           const double* bias, const double* x, int batch, int act, double* y) {
    int rc = check_layer(M, N, B, row_perm, col_perm, tile_list, T);
    if (rc != PPO_OK) return rc;
    int64_t Mp = (int64_t)((M + B - 1) / B) * B, Np = (int64_t)((N + B - 1) / B) * B;
    double* x_piv = (double*)malloc(sizeof(double) * (size_t)Np);
    double* y_piv = (double*)malloc(sizeof(double) * (size_t)Mp);
    for (int b = 0; b < batch; ++b) {
        for (int64_t j = 0; j < Np; ++j)
            x_piv[j] = (col_perm[j] < N) ? x[(int64_t)b * N + col_perm[j]] : 0.0;
        for (int64_t i = 0; i < Mp; ++i) y_piv[i] = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            int64_t br = tile_list[2 * t], bc = tile_list[2 * t + 1];
            for (int r = 0; r < B; ++r) {
                double acc = 0.0;
                for (int c = 0; c < B; ++c) acc += tile_values[(t * B + r) * B + c] * x_piv[bc * B + c];
                y_piv[br * B + r] += acc;
            }
        }
        for (int64_t i = 0; i < Mp; ++i) {
            int64_t I = row_perm[i];
            if (I < M) y[(int64_t)b * M + I] = activate(y_piv[i] + (bias ? bias[I] : 0.0), act);
        }
    }
    free(x_piv);
    free(y_piv);
    return PPO_OK;
}
