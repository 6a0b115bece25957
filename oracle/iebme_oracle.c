/*
 * CPU ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain, slow, obviously-correct C for the computation the library accelerates:
 *   - IE-BME encoding of a pruned INT4 weight matrix (paper Sec. V-A: area partition,
 *     shared union mask, Union Bitmaps / Union Value Offsets / Compressed Values),
 *   - its inverse (decode),
 *   - the Payload-to-Metadata Ratio (paper Eq. 1),
 *   - the result the SpMM kernel (paper Alg. 2: "W in IE-BME format, dense X -> Y") must
 *     reach: Y = W * X with INT32 accumulation, computed (a) as a naive triple loop on
 *     the masked dense weight and (b) straight from the encoded arrays,
 *   - the LSPD index rule (paper Sec. VI-B: idx_base + seg_rank),
 *   - bitmap-aware row reordering of one local tile (paper Sec. V-B, Alg. 1).
 *
 * Only tests, the smoke check and the bench's cpu-baseline leg may call this file.
 * It shares no code, header, table or constant with the CUDA library.
 *
 * Conventions (where the paper is silent, the reading taken is the one stated here):
 *   W  : int8 row-major M x K, values in [-8,7], 0 = pruned.
 *   LT : local tile H_L x K_L, index t = rb * (Kp/K_L) + kb (row-block major); M and K are
 *        zero-padded up to multiples of H_L and K_L.
 *   area q = a*C_A + c covers rows [a*H_B,(a+1)*H_B) x cols [c*K_B,(c+1)*K_B) of the LT,
 *        H_B = H_L/R_A, K_B = K_L/C_A.
 *   union mask bit beta = i*K_B + j, word beta/64, bit beta%64 (leftmost column = LSB).
 *   offsets count INT4 values (not bytes); n_lt + 1 entries.
 *   compressed values: two per byte, even index in the low nibble, 4-bit two's complement.
 *   X, Y: token-major, X[n*K + k], Y[n*M + m].
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t M, K;           /* logical shape */
    int64_t Mp, Kp;         /* padded shape */
    int64_t n_lt;           /* number of local tiles */
    int64_t words_per_lt;   /* 64-bit bitmap words per local tile */
    int64_t nnz;            /* true nonzeros */
    int64_t sum_P;          /* sum over tiles of P_t = ||B_t||_0 */
    int64_t n_values;       /* Q * sum_P stored INT4 values */
    int64_t bytes_payload;  /* ceil(n_values / 2) */
    int64_t bytes_bitmap;   /* 8 * words_per_lt * n_lt */
    int64_t bytes_offsets;  /* 4 * (n_lt + 1) */
    double  pmr;            /* Eq. 1: B_w * nnz / Stor_meta, B_w = 0.5 */
    double  fill;           /* n_values / (M*K) */
} orc_stats;

static int8_t w_at(const int8_t *W, int64_t M, int64_t K, int64_t r, int64_t c)
{
    if (r >= M || c >= K) return 0; /* zero padding */
    return W[r * K + c];
}

static void cv_put(uint8_t *cv, int64_t idx, int8_t v)
{
    uint8_t nib = (uint8_t)v & 0xF;
    if (idx & 1) cv[idx >> 1] = (uint8_t)((cv[idx >> 1] & 0x0F) | (nib << 4));
    else         cv[idx >> 1] = (uint8_t)((cv[idx >> 1] & 0xF0) | nib);
}

static int8_t cv_get(const uint8_t *cv, int64_t idx)
{
    uint8_t nib = (idx & 1) ? (cv[idx >> 1] >> 4) : (cv[idx >> 1] & 0xF);
    return (int8_t)((nib & 8) ? (int)nib - 16 : (int)nib);
}

/* Check the format parameters; returns 0 when usable. */
int orc_check_format(int H_L, int K_L, int R_A, int C_A)
{
    if (H_L <= 0 || K_L <= 0 || R_A <= 0 || C_A <= 0) return 1;
    if (H_L % R_A || K_L % C_A) return 2;
    if (((int64_t)(H_L / R_A) * (K_L / C_A)) % 64) return 3; /* whole 64-bit words */
    return 0;
}

/* Sizes the caller must allocate: bitmaps = n_lt*words_per_lt u64, offsets = n_lt+1 u32,
 * cv = Mp*Kp/2 bytes (worst case: every position stored). */
void orc_sizes(int64_t M, int64_t K, int H_L, int K_L, int R_A, int C_A,
               int64_t *n_lt, int64_t *words_per_lt, int64_t *cv_bytes_cap)
{
    int64_t Mp = (M + H_L - 1) / H_L * H_L, Kp = (K + K_L - 1) / K_L * K_L;
    *n_lt = (Mp / H_L) * (Kp / K_L);
    *words_per_lt = ((int64_t)(H_L / R_A) * (K_L / C_A)) / 64;
    *cv_bytes_cap = Mp * Kp / 2 + 1;
}

/* IE-BME encode (Sec. V-A). Returns 0, or <0 on a value outside [-8,7]. */
int orc_encode(const int8_t *W, int64_t M, int64_t K, int H_L, int K_L, int R_A, int C_A,
               uint64_t *bitmaps, uint32_t *offsets, uint8_t *cv, orc_stats *st)
{
    const int Q = R_A * C_A, H_B = H_L / R_A, K_B = K_L / C_A;
    const int64_t Mp = (M + H_L - 1) / H_L * H_L, Kp = (K + K_L - 1) / K_L * K_L;
    const int64_t tiles_k = Kp / K_L, n_lt = (Mp / H_L) * tiles_k;
    const int64_t wpl = ((int64_t)H_B * K_B) / 64;
    int64_t o = 0, nnz = 0, sum_P = 0;

    for (int64_t i = 0; i < M * K; ++i) {
        if (W[i] < -8 || W[i] > 7) return -1;
        if (W[i]) ++nnz;
    }
    memset(bitmaps, 0, (size_t)(n_lt * wpl) * sizeof(uint64_t));
    memset(cv, 0, (size_t)(Mp * Kp / 2 + 1));

    for (int64_t t = 0; t < n_lt; ++t) {
        const int64_t r0 = (t / tiles_k) * H_L, c0 = (t % tiles_k) * K_L;
        uint64_t *bm = bitmaps + t * wpl;
        /* union mask B_t(i,j) = OR_q (W_t^(q)(i,j) != 0) */
        int64_t P = 0;
        for (int i = 0; i < H_B; ++i)
            for (int j = 0; j < K_B; ++j) {
                int any = 0;
                for (int a = 0; a < R_A; ++a)
                    for (int c = 0; c < C_A; ++c)
                        if (w_at(W, M, K, r0 + a * H_B + i, c0 + c * K_B + j)) any = 1;
                if (any) {
                    int64_t beta = (int64_t)i * K_B + j;
                    bm[beta / 64] |= (uint64_t)1 << (beta % 64);
                    ++P;
                }
            }
        /* compressed values: CV[o_t + q*P_t + rho_t(i,j)] = W_t^(q)(i,j) */
        offsets[t] = (uint32_t)o;
        int64_t rho = 0;
        for (int i = 0; i < H_B; ++i)
            for (int j = 0; j < K_B; ++j) {
                int64_t beta = (int64_t)i * K_B + j;
                if (!((bm[beta / 64] >> (beta % 64)) & 1)) continue;
                for (int a = 0; a < R_A; ++a)
                    for (int c = 0; c < C_A; ++c) {
                        int q = a * C_A + c;
                        cv_put(cv, o + (int64_t)q * P + rho,
                               w_at(W, M, K, r0 + a * H_B + i, c0 + c * K_B + j));
                    }
                ++rho;
            }
        o += (int64_t)Q * P;
        sum_P += P;
    }
    offsets[n_lt] = (uint32_t)o;

    if (st) {
        st->M = M; st->K = K; st->Mp = Mp; st->Kp = Kp;
        st->n_lt = n_lt; st->words_per_lt = wpl;
        st->nnz = nnz; st->sum_P = sum_P; st->n_values = o;
        st->bytes_payload = (o + 1) / 2;
        st->bytes_bitmap = 8 * wpl * n_lt;
        st->bytes_offsets = 4 * (n_lt + 1);
        st->pmr = 0.5 * (double)nnz / (double)(st->bytes_bitmap + st->bytes_offsets);
        st->fill = (double)o / ((double)M * (double)K);
    }
    return 0;
}

/* Inverse of orc_encode: walk the union mask in row-major order with a running rank. */
void orc_decode(const uint64_t *bitmaps, const uint32_t *offsets, const uint8_t *cv,
                int64_t M, int64_t K, int H_L, int K_L, int R_A, int C_A, int8_t *W_out)
{
    const int H_B = H_L / R_A, K_B = K_L / C_A;
    const int64_t Mp = (M + H_L - 1) / H_L * H_L, Kp = (K + K_L - 1) / K_L * K_L;
    const int64_t tiles_k = Kp / K_L, n_lt = (Mp / H_L) * tiles_k;
    const int64_t wpl = ((int64_t)H_B * K_B) / 64;
    memset(W_out, 0, (size_t)(M * K));
    for (int64_t t = 0; t < n_lt; ++t) {
        const int64_t r0 = (t / tiles_k) * H_L, c0 = (t % tiles_k) * K_L;
        const uint64_t *bm = bitmaps + t * wpl;
        int64_t P = 0;
        for (int64_t w = 0; w < wpl; ++w) P += __builtin_popcountll(bm[w]);
        int64_t rho = 0;
        for (int i = 0; i < H_B; ++i)
            for (int j = 0; j < K_B; ++j) {
                int64_t beta = (int64_t)i * K_B + j;
                if (!((bm[beta / 64] >> (beta % 64)) & 1)) continue;
                for (int a = 0; a < R_A; ++a)
                    for (int c = 0; c < C_A; ++c) {
                        int q = a * C_A + c;
                        int64_t r = r0 + a * H_B + i, col = c0 + c * K_B + j;
                        int8_t v = cv_get(cv, (int64_t)offsets[t] + (int64_t)q * P + rho);
                        if (r < M && col < K) W_out[r * K + col] = v;
                    }
                ++rho;
            }
    }
}

/* LSPD index rule (Sec. VI-B): payload index of the first active bit of segment g
 * (width G) of mask row r = actives in rows above + actives to the left in the row.
 * mask is H_B x K_B, one byte per bit. */
int64_t orc_lspd_idx_base(const uint8_t *mask, int K_B, int r, int g, int G)
{
    int64_t s = 0;
    for (int u = 0; u < r; ++u)
        for (int v = 0; v < K_B; ++v) s += mask[u * K_B + v];
    for (int v = 0; v < g * G; ++v) s += mask[r * K_B + v];
    return s;
}

/* The plain definition: Y[n][m] = sum_k W[m][k] * X[n][k], INT32 accumulate, on the masked
 * dense weight. X is int8 (values in [-8,7]) token-major N x K; Y is token-major N x M. */
void orc_spmm_dense(const int8_t *W, const int8_t *X, int64_t M, int64_t K, int64_t N, int32_t *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int32_t acc = 0;
            for (int64_t k = 0; k < K; ++k)
                acc += (int32_t)W[m * K + k] * (int32_t)X[n * K + k];
            Y[n * M + m] = acc;
        }
}

/* Second path: multiply straight from the IE-BME arrays (one active union bit selects Q
 * values at the same compact rank, one per area stream). Must agree with orc_spmm_dense. */
void orc_spmm_encoded(const uint64_t *bitmaps, const uint32_t *offsets, const uint8_t *cv,
                      int64_t M, int64_t K, int H_L, int K_L, int R_A, int C_A,
                      const int8_t *X, int64_t N, int32_t *Y)
{
    const int H_B = H_L / R_A, K_B = K_L / C_A;
    const int64_t Mp = (M + H_L - 1) / H_L * H_L, Kp = (K + K_L - 1) / K_L * K_L;
    const int64_t tiles_k = Kp / K_L, n_lt = (Mp / H_L) * tiles_k;
    const int64_t wpl = ((int64_t)H_B * K_B) / 64;
    memset(Y, 0, (size_t)(M * N) * sizeof(int32_t));
    for (int64_t t = 0; t < n_lt; ++t) {
        const int64_t r0 = (t / tiles_k) * H_L, c0 = (t % tiles_k) * K_L;
        const uint64_t *bm = bitmaps + t * wpl;
        int64_t P = 0;
        for (int64_t w = 0; w < wpl; ++w) P += __builtin_popcountll(bm[w]);
        int64_t rho = 0;
        for (int i = 0; i < H_B; ++i)
            for (int j = 0; j < K_B; ++j) {
                int64_t beta = (int64_t)i * K_B + j;
                if (!((bm[beta / 64] >> (beta % 64)) & 1)) continue;
                for (int a = 0; a < R_A; ++a)
                    for (int c = 0; c < C_A; ++c) {
                        int q = a * C_A + c;
                        int64_t r = r0 + a * H_B + i, col = c0 + c * K_B + j;
                        int32_t v = cv_get(cv, (int64_t)offsets[t] + (int64_t)q * P + rho);
                        if (r < M && col < K)
                            for (int64_t n = 0; n < N; ++n)
                                Y[n * M + r] += v * (int32_t)X[n * K + col];
                    }
                ++rho;
            }
    }
}

int orc_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* ------------------------------------------------------------------------------------------
 * Bitmap-aware row reordering (paper Sec. V-B, Eqs. 3-5, Alg. 1), one local tile at a time.
 *
 *   mask   : H_L x K_L bytes, nonzero = the weight at that position survives pruning
 *   group  : R_A rows sharing one union-mask row; its cost (Eqs. 3-4) = number of grouped
 *            columns j in [0, K_L/C_A) at which any of its rows has a nonzero in any of the
 *            C_A column partitions (column j + c*K_L/C_A)
 *   F(S)   : least total cost of splitting the row set S into groups (Eq. 5); memoised
 *            recursion on the subset bitmask, always grouping the lowest row of S first
 *   result : groups with rows ascending, groups in lexicographic order, permutation =
 *            partition-wise concatenation: perm[p*(H_L/R_A) + g] = p-th row of group g.
 *
 * Ties between groupings of equal cost go to the first candidate met when the partners of the
 * lowest row are enumerated in ascending combination order (the paper fixes no tie rule).
 * Returns the optimal cost F(all rows), or -1 on unusable arguments (H_L > 20, R_A not
 * dividing H_L, C_A not dividing K_L).
 * ------------------------------------------------------------------------------------------ */
typedef struct {
    const uint8_t *mask;
    int H_L, K_L, R_A, C_A;
    int64_t *F;        /* 2^H_L entries, -1 = not computed yet */
    uint32_t *choice;  /* the group (as a row bitmask) taken first at state S */
} reorder_ctx;

static int64_t group_cost(const reorder_ctx *c, uint32_t rows)
{
    const int K_B = c->K_L / c->C_A;
    int64_t cost = 0;
    for (int j = 0; j < K_B; ++j) {
        int active = 0;
        for (int r = 0; r < c->H_L && !active; ++r) {
            if (!((rows >> r) & 1u)) continue;
            for (int cc = 0; cc < c->C_A && !active; ++cc)
                if (c->mask[(int64_t)r * c->K_L + j + cc * K_B]) active = 1;
        }
        cost += active;
    }
    return cost;
}

static int64_t reorder_F(reorder_ctx *c, uint32_t S);

/* Extends `group` (already holding `have` rows, the last one `last`) by rows of S above
 * `last`; at R_A rows evaluates cost + F(rest) and keeps the best. */
static void reorder_try(reorder_ctx *c, uint32_t S, uint32_t group, int have, int last,
                        int64_t *best, uint32_t *best_group)
{
    if (have == c->R_A) {
        const int64_t v = group_cost(c, group) + reorder_F(c, S & ~group);
        if (*best < 0 || v < *best) { *best = v; *best_group = group; }
        return;
    }
    for (int r = last + 1; r < c->H_L; ++r)
        if ((S >> r) & 1u) reorder_try(c, S, group | (1u << r), have + 1, r, best, best_group);
}

static int64_t reorder_F(reorder_ctx *c, uint32_t S)
{
    if (S == 0) return 0;
    if (c->F[S] >= 0) return c->F[S];
    int r = 0;
    while (!((S >> r) & 1u)) ++r;
    int64_t best = -1;
    uint32_t best_group = 0;
    reorder_try(c, S, 1u << r, 1, r, &best, &best_group);
    c->F[S] = best;
    c->choice[S] = best_group;
    return best;
}

int64_t orc_reorder_tile(const uint8_t *mask, int H_L, int K_L, int R_A, int C_A, int32_t *perm_out)
{
    if (H_L <= 0 || H_L > 20 || R_A <= 0 || C_A <= 0 || H_L % R_A || K_L <= 0 || K_L % C_A) return -1;
    reorder_ctx c = {mask, H_L, K_L, R_A, C_A, NULL, NULL};
    const size_t n_states = (size_t)1 << H_L;
    c.F = (int64_t *)malloc(n_states * sizeof(int64_t));
    c.choice = (uint32_t *)calloc(n_states, sizeof(uint32_t));
    if (!c.F || !c.choice) { free(c.F); free(c.choice); return -1; }
    for (size_t i = 0; i < n_states; ++i) c.F[i] = -1;
    const uint32_t all = (uint32_t)(n_states - 1);
    const int64_t total = reorder_F(&c, all);

    /* Walk the choices. Each step takes the group holding the lowest remaining row, so the
     * groups come out ordered by their first rows -- which, rows inside a group being ascending
     * and groups disjoint, is the lexicographic order the paper asks for. */
    const int n_groups = H_L / R_A;
    uint32_t S = all;
    for (int g = 0; g < n_groups; ++g) {
        const uint32_t grp = c.choice[S];
        int p = 0;
        for (int r = 0; r < H_L; ++r)
            if ((grp >> r) & 1u) perm_out[p++ * n_groups + g] = r;
        S &= ~grp;
    }
    free(c.F);
    free(c.choice);
    return total;
}
