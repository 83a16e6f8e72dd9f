/*
 * tlo -- TileLens ORACLE (test infrastructure only; see tlo.h).
 * Plain C, fp64 arithmetic, integer division and modulo written out,
 * OpenMP "parallel for" over independent outputs and nothing else.
 */
#include "tlo.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------ Section 4.3: TileLens-HW */

static int is_pow2_i64(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }
static int log2_i64(int64_t x) { int l = 0; while (((int64_t)1 << l) < x) ++l; return l; }

int tlo_hw_box_offsets(const tlo_hw_desc* d, const int64_t* coords, int64_t* out) {
    if (d->rank < 2 || d->rank > 5 || d->s <= 0 || d->strides[0] != 1) return -1;
    if (!is_pow2_i64(d->a) || !is_pow2_i64(d->b) || d->K <= 0 || d->K % d->a != 0) return -1;
    const int64_t u = d->box[0];
    if (!is_pow2_i64(u) || u > d->a) return -1;           /* invariant 1; the section covers a == u and a > u */
    /* Case 2 computes everything "as if the memory tile size is u x b" */
    const int64_t a_eff = u;

    /* Phase 1: split and sum.  Products with a stride below the leading stride add up to i, the rest to K*j. */
    int64_t i = 0, Kj = 0;
    for (int k = 0; k < d->rank; ++k) {
        if (coords[k] < 0 || d->box[k] <= 0) return -1;
        if (d->strides[k] < d->K) i += coords[k] * d->strides[k];
        else Kj += coords[k] * d->strides[k];
    }
    if (i % a_eff != 0 || Kj % (d->K * d->b) != 0) return -1;     /* aligned to memory tiles (Eq. 4's premise) */
    const int64_t tile_base = (Kj + i * d->b) * d->s;             /* Eq. 4 */

    /* Phase 2: the counters.  Every dimension keeps its counter except the one whose stride is K, which becomes
     * an inner counter of b steps of stride a and an outer one of v/b steps of stride b*K (Eq. 5).  A stride below
     * K moves along a column of the matrix by a multiple of the tile width, i.e. over whole memory tiles, each
     * a*b elements further (Eq. 4's i*b term); a stride above K moves over whole tile columns (its K*j term). */
    int64_t ext[6], str[6];
    int n = 0;
    for (int k = 0; k < d->rank; ++k) {
        const int64_t sg = d->strides[k], v = d->box[k];
        if (k == 0) { ext[n] = u; str[n] = 1; ++n; }
        else if (sg == d->K) {
            if (v % d->b != 0) return -1;
            ext[n] = d->b; str[n] = a_eff; ++n;
            ext[n] = v / d->b; str[n] = d->b * d->K; ++n;
        } else if (sg < d->K) {
            if (sg % a_eff != 0) return -1;
            ext[n] = v; str[n] = sg * d->b; ++n;
        } else {
            if (sg % (d->b * d->K) != 0) return -1;
            ext[n] = v; str[n] = sg; ++n;
        }
    }
    /* Case 2: bit permutation of the intra-tile element offset, (sub-tile | col | row) -> (col | sub-tile | row) */
    const int row_bits = log2_i64(u), col_bits = log2_i64(d->b), sub_bits = log2_i64(d->a / u);

    int64_t cnt[6] = {0, 0, 0, 0, 0, 0};
    int64_t total = 1;
    for (int k = 0; k < n; ++k) total *= ext[k];
    for (int64_t t = 0; t < total; ++t) {
        int64_t src = tile_base;
        for (int k = 0; k < n; ++k) src += cnt[k] * str[k] * d->s;
        if (sub_bits > 0) {
            int64_t e = src / d->s;                                  /* element index */
            const int64_t intra_mask = ((int64_t)1 << (row_bits + col_bits + sub_bits)) - 1;
            const int64_t intra = e & intra_mask;
            const int64_t row = intra & (((int64_t)1 << row_bits) - 1);
            const int64_t col = (intra >> row_bits) & (((int64_t)1 << col_bits) - 1);
            const int64_t sub = intra >> (row_bits + col_bits);
            const int64_t fixed = (col << (sub_bits + row_bits)) | (sub << row_bits) | row;
            src = ((e & ~intra_mask) | fixed) * d->s;
        }
        out[t] = src;
        for (int k = 0; k < n; ++k) {                                /* increment the nested counters */
            if (++cnt[k] < ext[k]) break;
            cnt[k] = 0;
        }
    }
    return 0;
}

int tlo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- layouts */

/* Section 2.4: a row is contiguous. */
int64_t tlo_off_row(int64_t r, int64_t c, int64_t rows, int64_t cols, int64_t s) {
    (void)rows;
    return (r * cols + c) * s;
}

/* Section 2.4 / Section 3.2: a column is contiguous, offset (j*K + i)*s. */
int64_t tlo_off_col(int64_t r, int64_t c, int64_t rows, int64_t cols, int64_t s) {
    (void)cols;
    return (c * rows + r) * s;
}

/* Eq. 1 + Eq. 2 in the row flavour: the contiguous direction is the column
 * index c, so (i, a, K) of the printed form become (c, bc, cols) and
 * (j, b, N) become (r, br, rows). */
int64_t tlo_off_tile(int64_t r, int64_t c, int64_t rows, int64_t cols,
                     int64_t br, int64_t bc, int64_t s) {
    (void)rows;
    int64_t Tr = r / br, rp = r % br;          /* Eq. 1 */
    int64_t Tc = c / bc, cp = c % bc;
    int64_t tiles_per_tile_row = cols / bc;
    int64_t linear_tile = Tr * tiles_per_tile_row + Tc;   /* tiles ordered along the contiguous direction first */
    int64_t intra = rp * bc + cp;                          /* same order inside the tile */
    return linear_tile * (br * bc * s) + intra * s;        /* Eq. 2 */
}

int64_t tlo_off(int layout, int64_t r, int64_t c, int64_t rows, int64_t cols,
                int64_t br, int64_t bc, int64_t s) {
    if (layout == TLO_ROW_MAJOR) return tlo_off_row(r, c, rows, cols, s);
    if (layout == TLO_COL_MAJOR) return tlo_off_col(r, c, rows, cols, s);
    /* Eq. 2 as printed: (r, c) = (i, j) of the K x N matrix, a = bc along K, b = br along N */
    if (layout == TLO_TILE_MAJOR_K) return tlo_eq2(r, c, rows, cols, bc, br, s);
    return tlo_off_tile(r, c, rows, cols, br, bc, s);
}

/* Eq. 1 exactly as printed. */
void tlo_eq1(int64_t i, int64_t j, int64_t a, int64_t b, int64_t out[4]) {
    out[0] = i % a;   /* i'  */
    out[1] = j % b;   /* j'  */
    out[2] = i / a;   /* T_i */
    out[3] = j / b;   /* T_j */
}

/* Eq. 2 exactly as printed: K x N matrix, K contiguous, memory tile a x b. */
int64_t tlo_eq2(int64_t i, int64_t j, int64_t K, int64_t N, int64_t a, int64_t b, int64_t s) {
    (void)N;
    int64_t q[4];
    tlo_eq1(i, j, a, b, q);
    int64_t ip = q[0], jp = q[1], Ti = q[2], Tj = q[3];
    return (Tj * (K / a) + Ti) * (a * b * s) + (jp * a + ip) * s;
}

/* Eq. 3: shape (a, b, K/a, N/b), stride (1, a, ab, Kb) in elements. */
int64_t tlo_eq3(int64_t i, int64_t j, int64_t K, int64_t N, int64_t a, int64_t b, int64_t s) {
    (void)N;
    int64_t q[4];
    tlo_eq1(i, j, a, b, q);
    int64_t stride[4] = {1, a, a * b, K * b};
    int64_t e = 0;
    for (int d = 0; d < 4; ++d) e += q[d] * stride[d];
    return e * s;
}

/* --------------------------------------------------------------- relayout */

int tlo_relayout(const void* src, void* dst, int64_t rows, int64_t cols, int64_t s,
                 int64_t br, int64_t bc, int direction) {
    if (rows < 0 || cols < 0 || s <= 0 || br <= 0 || bc <= 0) return -1;
    if (rows % br != 0 || cols % bc != 0) return -1;       /* Section 3.3 */
    const unsigned char* in = (const unsigned char*)src;
    unsigned char* out = (unsigned char*)dst;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t c = 0; c < cols; ++c) {
            int64_t o_row = tlo_off_row(r, c, rows, cols, s);
            int64_t o_tile = tlo_off_tile(r, c, rows, cols, br, bc, s);
            if (direction == TLO_TO_TILE_MAJOR)
                memcpy(out + o_tile, in + o_row, (size_t)s);
            else
                memcpy(out + o_row, in + o_tile, (size_t)s);
        }
    }
    return 0;
}

/* ----------------------------------------------------------------- matmul */

double tlo_bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Section 2.3: one output element, the sum over k written out. */
static void dot_at(const uint16_t* A, const uint16_t* B, int layout, int64_t br, int64_t bc,
                   int64_t N, int64_t K, int64_t i, int64_t j, double* c_out, double* s_out) {
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double a = tlo_bf16_to_double(A[i * K + k]);
        int64_t off = tlo_off(layout, k, j, K, N, br, bc, 2);
        double b = tlo_bf16_to_double(B[off / 2]);
        double p = a * b;
        acc += p;
        abs_acc += fabs(p);
    }
    *c_out = acc;
    *s_out = abs_acc;
}

int tlo_matmul_at(const uint16_t* A, const uint16_t* B, int layout, int64_t br, int64_t bc,
                  int64_t M, int64_t N, int64_t K, int64_t n,
                  const int64_t* idx_i, const int64_t* idx_j, double* C, double* S) {
    if (layout == TLO_TILE_MAJOR && (br <= 0 || bc <= 0 || K % br != 0 || N % bc != 0)) return -1;
    if (layout == TLO_TILE_MAJOR_K && (br <= 0 || bc <= 0 || K % bc != 0 || N % br != 0)) return -1;
    for (int64_t t = 0; t < n; ++t)
        if (idx_i[t] < 0 || idx_i[t] >= M || idx_j[t] < 0 || idx_j[t] >= N) return -1;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < n; ++t)
        dot_at(A, B, layout, br, bc, N, K, idx_i[t], idx_j[t], &C[t], &S[t]);
    return 0;
}

int tlo_matmul(const uint16_t* A, const uint16_t* B, int layout, int64_t br, int64_t bc,
               int64_t M, int64_t N, int64_t K, double* C, double* S) {
    if (layout == TLO_TILE_MAJOR && (br <= 0 || bc <= 0 || K % br != 0 || N % bc != 0)) return -1;
    if (layout == TLO_TILE_MAJOR_K && (br <= 0 || bc <= 0 || K % bc != 0 || N % br != 0)) return -1;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t t = 0; t < M * N; ++t)
        dot_at(A, B, layout, br, bc, N, K, t / N, t % N, &C[t], &S[t]);
    return 0;
}

/* FP8 in the E4M3 encoding GPUs use for inference (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no
 * infinities, S.1111.111 is NaN): the value written out from its fields. */
double tlo_fp8_e4m3_to_double(uint8_t h) {
    int sign = h >> 7, e = (h >> 3) & 15, m = h & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);           /* subnormal: 0.m x 2^(1-bias) */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Section 2.3 with s = 1 (Section 3.1 treats FP8 beside the 16-bit types): the same sum over k on FP8 operands. */
static void dot_at_fp8(const uint8_t* A, const uint8_t* B, int layout, int64_t br, int64_t bc,
                       int64_t N, int64_t K, int64_t i, int64_t j, double* c_out, double* s_out) {
    double acc = 0.0, abs_acc = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double a = tlo_fp8_e4m3_to_double(A[i * K + k]);
        double b = tlo_fp8_e4m3_to_double(B[tlo_off(layout, k, j, K, N, br, bc, 1)]);
        double p = a * b;
        acc += p;
        abs_acc += fabs(p);
    }
    *c_out = acc;
    *s_out = abs_acc;
}

int tlo_matmul_at_fp8(const uint8_t* A, const uint8_t* B, int layout, int64_t br, int64_t bc,
                      int64_t M, int64_t N, int64_t K, int64_t n,
                      const int64_t* idx_i, const int64_t* idx_j, double* C, double* S) {
    if (layout == TLO_TILE_MAJOR && (br <= 0 || bc <= 0 || K % br != 0 || N % bc != 0)) return -1;
    if (layout == TLO_TILE_MAJOR_K && (br <= 0 || bc <= 0 || K % bc != 0 || N % br != 0)) return -1;
    for (int64_t t = 0; t < n; ++t)
        if (idx_i[t] < 0 || idx_i[t] >= M || idx_j[t] < 0 || idx_j[t] >= N) return -1;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < n; ++t)
        dot_at_fp8(A, B, layout, br, bc, N, K, idx_i[t], idx_j[t], &C[t], &S[t]);
    return 0;
}

/* ----------------------------------------------------- read amplification */

/* One weight-tile load: rows k in [k0,k1), columns n in [n0,n1) of the K x N
 * operand.  Visits every element, marks the block of its first and of its
 * last byte, counts marks that were new, then clears them again. */
static uint64_t blocks_touched(unsigned char* mark, int layout, int64_t K, int64_t N,
                               int64_t br, int64_t bc, int64_t s, int64_t G,
                               int64_t k0, int64_t k1, int64_t n0, int64_t n1) {
    uint64_t count = 0;
    for (int64_t k = k0; k < k1; ++k)
        for (int64_t n = n0; n < n1; ++n) {
            int64_t off = tlo_off(layout, k, n, K, N, br, bc, s);
            int64_t first = off / G, last = (off + s - 1) / G;
            if (!mark[first]) { mark[first] = 1; ++count; }
            if (!mark[last])  { mark[last] = 1;  ++count; }
        }
    for (int64_t k = k0; k < k1; ++k)
        for (int64_t n = n0; n < n1; ++n) {
            int64_t off = tlo_off(layout, k, n, K, N, br, bc, s);
            mark[off / G] = 0;
            mark[(off + s - 1) / G] = 0;
        }
    return count;
}

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* All weight-tile loads issued by ONE row of CTA tiles (one m-tile): every
 * n-tile, every K iteration.  per_ntile_* (length n-tiles) may be NULL. */
static int weight_loads_one_mtile(int64_t N, int64_t K, int64_t BN, int64_t BK,
                                  int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                                  uint64_t* fetched, uint64_t* used, uint64_t* requests,
                                  uint64_t* per_ntile_fetched, uint64_t* per_ntile_used) {
    int64_t nt = ceil_div(N, BN), kt = ceil_div(K, BK);
    int64_t total_blocks = ceil_div(K * N * s, G) + 1;
    uint64_t f_sum = 0, u_sum = 0, q_sum = 0;
    int failed = 0;
#pragma omp parallel reduction(+ : f_sum, u_sum, q_sum)
    {
        unsigned char* mark = (unsigned char*)calloc((size_t)total_blocks, 1);
        if (!mark) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t tn = 0; tn < nt; ++tn) {
            if (!mark) continue;
            int64_t n0 = tn * BN, n1 = n0 + BN < N ? n0 + BN : N;
            uint64_t f_tile = 0, u_tile = 0;
            for (int64_t tk = 0; tk < kt; ++tk) {
                int64_t k0 = tk * BK, k1 = k0 + BK < K ? k0 + BK : K;
                uint64_t blocks = blocks_touched(mark, layout, K, N, br, bc, s, G, k0, k1, n0, n1);
                f_tile += blocks * (uint64_t)G;
                u_tile += (uint64_t)((k1 - k0) * (n1 - n0) * s);
                q_sum += blocks;
            }
            f_sum += f_tile;
            u_sum += u_tile;
            if (per_ntile_fetched) per_ntile_fetched[tn] = f_tile;
            if (per_ntile_used) per_ntile_used[tn] = u_tile;
        }
        free(mark);
    }
    if (failed) return -2;
    *fetched = f_sum;
    *used = u_sum;
    *requests = q_sum;
    return 0;
}

static int read_amp_args_ok(int64_t N, int64_t K, int64_t BM, int64_t BN, int64_t BK,
                            int layout, int64_t G, int64_t br, int64_t bc, int64_t s) {
    if (N <= 0 || K <= 0 || BM <= 0 || BN <= 0 || BK <= 0 || G <= 0 || s <= 0) return 0;
    if (layout == TLO_TILE_MAJOR) {
        if (br <= 0 || bc <= 0 || br * bc * s != G) return 0;     /* Section 3.1: h*w*s = G */
        if (K % br != 0 || N % bc != 0) return 0;                 /* Section 3.3 */
    } else if (layout == TLO_TILE_MAJOR_K) {
        if (br <= 0 || bc <= 0 || br * bc * s != G) return 0;
        if (K % bc != 0 || N % br != 0) return 0;
    } else if (layout != TLO_ROW_MAJOR && layout != TLO_COL_MAJOR) {
        return 0;
    }
    return 1;
}

int tlo_read_amp(int64_t M, int64_t N, int64_t K, int64_t BM, int64_t BN, int64_t BK,
                 int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                 uint64_t* fetched, uint64_t* used, uint64_t* requests,
                 uint64_t* per_tile_fetched, uint64_t* per_tile_used) {
    if (M < 0 || !read_amp_args_ok(N, K, BM, BN, BK, layout, G, br, bc, s)) return -1;
    int64_t mt = ceil_div(M, BM), nt = ceil_div(N, BN);
    uint64_t f = 0, u = 0, q = 0;
    uint64_t* pf = NULL;
    uint64_t* pu = NULL;
    if (per_tile_fetched && per_tile_used && mt > 0) { pf = per_tile_fetched; pu = per_tile_used; }
    int rc = weight_loads_one_mtile(N, K, BN, BK, layout, G, br, bc, s, &f, &u, &q, pf, pu);
    if (rc) return rc;
    /* every m-tile's CTAs issue the same weight loads */
    for (int64_t tm = 1; tm < mt && pf; ++tm)
        for (int64_t tn = 0; tn < nt; ++tn) {
            pf[tm * nt + tn] = pf[tn];
            pu[tm * nt + tn] = pu[tn];
        }
    *fetched = f * (uint64_t)mt;
    *used = u * (uint64_t)mt;
    if (requests) *requests = q * (uint64_t)mt;
    return 0;
}

int tlo_read_amp_grouped(const int32_t* offsets, int E, int64_t N, int64_t K,
                         int64_t BM, int64_t BN, int64_t BK,
                         int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                         uint64_t* fetched, uint64_t* used, uint64_t* requests) {
    if (E < 0 || !read_amp_args_ok(N, K, BM, BN, BK, layout, G, br, bc, s)) return -1;
    uint64_t f1 = 0, u1 = 0, q1 = 0;
    /* every expert's weight has the same shape and starts on a G boundary,
     * so one expert's one-m-tile count serves all of them */
    int rc = weight_loads_one_mtile(N, K, BN, BK, layout, G, br, bc, s, &f1, &u1, &q1, NULL, NULL);
    if (rc) return rc;
    uint64_t f = 0, u = 0, q = 0;
    for (int e = 0; e < E; ++e) {
        int64_t Me = (int64_t)offsets[e + 1] - (int64_t)offsets[e];
        if (Me < 0) return -1;
        if (Me == 0) continue;                    /* an expert with no token launches no CTA */
        uint64_t mt = (uint64_t)ceil_div(Me, BM);
        f += f1 * mt;
        u += u1 * mt;
        q += q1 * mt;
    }
    *fetched = f;
    *used = u;
    if (requests) *requests = q;
    return 0;
}

/* Sections 2.5 and 6.5 (requests shared between CTAs): the count when the CTAs that are resident together step
 * through K together and a block wanted by several of them at the same step is fetched once.  CTA tiles are
 * numbered n-tile major, m-tile minor; wave w holds tiles [w*P, (w+1)*P).  For every wave and every K iteration
 * the blocks of all its tiles' weight rectangles are marked element by element in one set. */
int tlo_read_amp_shared(int64_t M, int64_t N, int64_t K, int64_t BM, int64_t BN, int64_t BK, int64_t P,
                        int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                        uint64_t* fetched, uint64_t* needed, uint64_t* requests) {
    if (M < 0 || P <= 0 || !read_amp_args_ok(N, K, BM, BN, BK, layout, G, br, bc, s)) return -1;
    const int64_t mt = ceil_div(M, BM), nt = ceil_div(N, BN), kt = ceil_div(K, BK);
    const int64_t T = mt * nt, waves = ceil_div(T, P);
    const int64_t total_blocks = ceil_div(K * N * s, G) + 1;
    uint64_t f_sum = 0, u_sum = 0, q_sum = 0;
    int failed = 0;
#pragma omp parallel reduction(+ : f_sum, u_sum, q_sum)
    {
        unsigned char* mark = (unsigned char*)calloc((size_t)total_blocks, 1);
        unsigned char* col_seen = (unsigned char*)calloc((size_t)N, 1);
        if (!mark || !col_seen) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < waves; ++w) {
            if (!mark || !col_seen) continue;
            const int64_t t0 = w * P, t1 = t0 + P < T ? t0 + P : T;
            for (int64_t tk = 0; tk < kt; ++tk) {
                const int64_t k0 = tk * BK, k1 = k0 + BK < K ? k0 + BK : K;
                uint64_t blocks = 0, cols = 0;
                for (int64_t t = t0; t < t1; ++t) {               /* every CTA tile of the wave */
                    const int64_t tn = t / mt;
                    const int64_t n0 = tn * BN, n1 = n0 + BN < N ? n0 + BN : N;
                    for (int64_t k = k0; k < k1; ++k)
                        for (int64_t n = n0; n < n1; ++n) {
                            int64_t off = tlo_off(layout, k, n, K, N, br, bc, s);
                            int64_t first = off / G, last = (off + s - 1) / G;
                            if (!mark[first]) { mark[first] = 1; ++blocks; }
                            if (!mark[last])  { mark[last] = 1;  ++blocks; }
                        }
                    for (int64_t n = n0; n < n1; ++n)
                        if (!col_seen[n]) { col_seen[n] = 1; ++cols; }
                }
                for (int64_t t = t0; t < t1; ++t) {               /* clear the marks again */
                    const int64_t tn = t / mt;
                    const int64_t n0 = tn * BN, n1 = n0 + BN < N ? n0 + BN : N;
                    for (int64_t k = k0; k < k1; ++k)
                        for (int64_t n = n0; n < n1; ++n) {
                            int64_t off = tlo_off(layout, k, n, K, N, br, bc, s);
                            mark[off / G] = 0;
                            mark[(off + s - 1) / G] = 0;
                        }
                    for (int64_t n = n0; n < n1; ++n) col_seen[n] = 0;
                }
                f_sum += blocks * (uint64_t)G;
                q_sum += blocks;
                u_sum += cols * (uint64_t)(k1 - k0) * (uint64_t)s;
            }
        }
        free(mark);
        free(col_seen);
    }
    if (failed) return -2;
    *fetched = f_sum;
    *needed = u_sum;
    *requests = q_sum;
    return 0;
}

/* Section 5.2, Eq. 6: prefetch degree.  BL = bandwidth * latency / G requests keep the bus busy; a wave issues
 * p_wave = n_sm * ctas_per_sm * p_tile demand requests per K iteration; d = min(floor(c * BL / p_wave), K / TILE_K)
 * with c = 1 as printed (the text then doubles the first term in practice: c = 2). */
int64_t tlo_prefetch_degree(double bandwidth_bytes_per_s, double latency_s, int64_t G, int64_t n_sm, int64_t ctas_per_sm,
                            int64_t p_tile, int64_t K, int64_t tile_k, double collision_factor) {
    if (G <= 0 || n_sm <= 0 || ctas_per_sm <= 0 || p_tile <= 0 || K <= 0 || tile_k <= 0) return -1;
    const double BL = bandwidth_bytes_per_s * latency_s / (double)G;
    const double p_wave = (double)n_sm * (double)ctas_per_sm * (double)p_tile;
    int64_t d = (int64_t)floor(collision_factor * BL / p_wave);
    const int64_t cap = K / tile_k;
    return d < cap ? d : cap;
}

/* Section 6.5 ("Straggler-Induced CTA Stalls"): a CTA issues the n requests of a compute tile together and can
 * start only when the last one has arrived; the section measures the time to the first arrival ("queueing") and the
 * time between the first and the last ("straggler wait"), and explains the gap between layouts by the chance that
 * the slowest of n requests falls in the tail of the per-request latency distribution.
 * The paper gives that distribution only as figures, so none is assumed here: the caller passes a sample of
 * per-request latencies (a measurement, a trace), read as the distribution that puts probability 1/N on each
 * sample value, and the n requests of a tile are read as independent draws from it.  Then, with the sample sorted,
 *   P(last arrival <= x_(i)) = (i/N)^n,    P(first arrival > x_(i)) = ((N - i)/N)^n,
 * which give the two expectations below as plain sums over the sorted sample, and
 *   P(last arrival > t) = 1 - (#{x <= t} / N)^n.
 * Returns 0, or -1 for bad arguments. */
static int tlo_cmp_double(const void* a, const void* b) {
    const double x = *(const double*)a, y = *(const double*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}
int tlo_tile_arrival(const double* samples, int64_t N, int64_t n, double threshold, double* first, double* last,
                     double* p_late) {
    if (!samples || N <= 0 || n <= 0 || !first || !last) return -1;
    double* x = (double*)malloc((size_t)N * sizeof(double));
    if (!x) return -1;
    for (int64_t i = 0; i < N; ++i) x[i] = samples[i];
    qsort(x, (size_t)N, sizeof(double), tlo_cmp_double);
    long double e_max = 0.0L, e_min = 0.0L;
    int64_t below = 0;
    for (int64_t i = 1; i <= N; ++i) {
        /* probability that the largest of n draws is exactly the i-th smallest sample value, and the same for the
         * smallest of n draws */
        const long double p_max = powl((long double)i / (long double)N, (long double)n) -
                                  powl((long double)(i - 1) / (long double)N, (long double)n);
        const long double p_min = powl((long double)(N - i + 1) / (long double)N, (long double)n) -
                                  powl((long double)(N - i) / (long double)N, (long double)n);
        e_max += p_max * (long double)x[i - 1];
        e_min += p_min * (long double)x[i - 1];
        if (x[i - 1] <= threshold) ++below;
    }
    *first = (double)e_min;
    *last = (double)e_max;
    if (p_late) *p_late = (double)(1.0L - powl((long double)below / (long double)N, (long double)n));
    free(x);
    return 0;
}

/* ------------------------------------------- MoE expert FFN (Section 2.3 names the workload; epilogues are ours)
 *
 * The paper's MoE kernel is the two grouped products of an expert FFN; it does not describe what happens between
 * them.  What is computed here is the usual gated form: h = silu(x W_gate) * (x W_up), rounded once to bf16 (the
 * intermediate dtype), y = h W_down, everything else in fp64. */

/* double -> bf16 bit pattern, round to nearest, ties to even (through binary32, which holds every bf16 exactly:
 * the double is first rounded to binary32 by the C conversion, then the low 16 bits are rounded away). */
uint16_t tlo_double_to_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);     /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

double tlo_silu(double x) { return x / (1.0 + exp(-x)); }

/* h[j] for one row of one expert: gate/up columns interleaved (column 2j = gate_j, 2j+1 = up_j) in the K x 2I weight. */
static uint16_t ffn_h_at(const uint16_t* x_row, const uint16_t* W_gu, int layout, int64_t br, int64_t bc,
                         int64_t K, int64_t I, int64_t j) {
    double g = 0.0, u = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double a = tlo_bf16_to_double(x_row[k]);
        g += a * tlo_bf16_to_double(W_gu[tlo_off(layout, k, 2 * j, K, 2 * I, br, bc, 2) / 2]);
        u += a * tlo_bf16_to_double(W_gu[tlo_off(layout, k, 2 * j + 1, K, 2 * I, br, bc, 2) / 2]);
    }
    return tlo_double_to_bf16(tlo_silu(g) * u);
}

/* Rows listed in `rows` (indices into the expert-sorted X): H_out[r][0..I) as bf16 bits, Y_out[r][0..hidden) and
 * S_out[r][.] = sum_j |h_j * Wd[j][c]| in fp64.  offsets: E+1 row offsets of the experts.  Each expert's W_gate_up is
 * K x 2I, its W_down I x hidden, both in `layout` with memory tile br x bc, experts laid end to end. */
int tlo_moe_ffn_rows(const uint16_t* X, const uint16_t* W_gu, const uint16_t* W_down, const int32_t* offsets, int E,
                     int64_t hidden, int64_t I, int layout, int64_t br, int64_t bc,
                     int64_t n_rows, const int64_t* rows, uint16_t* H_out, double* Y_out, double* S_out) {
    if (layout == TLO_TILE_MAJOR && (br <= 0 || bc <= 0 || hidden % br || (2 * I) % bc || I % br || hidden % bc)) return -1;
    for (int64_t t = 0; t < n_rows; ++t)
        if (rows[t] < 0 || rows[t] >= offsets[E]) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < n_rows; ++t) {
        int e = 0;
        while (!(offsets[e] <= rows[t] && rows[t] < offsets[e + 1])) ++e;
        const uint16_t* x_row = X + rows[t] * hidden;
        const uint16_t* wgu = W_gu + (int64_t)e * hidden * 2 * I;
        const uint16_t* wd = W_down + (int64_t)e * I * hidden;
        uint16_t* h = H_out + t * I;
        for (int64_t j = 0; j < I; ++j) h[j] = ffn_h_at(x_row, wgu, layout, br, bc, hidden, I, j);
        for (int64_t c = 0; c < hidden; ++c) {
            double acc = 0.0, sab = 0.0;
            for (int64_t j = 0; j < I; ++j) {
                double p = tlo_bf16_to_double(h[j]) * tlo_bf16_to_double(wd[tlo_off(layout, j, c, I, hidden, br, bc, 2) / 2]);
                acc += p;
                sab += fabs(p);
            }
            Y_out[t * hidden + c] = acc;
            S_out[t * hidden + c] = sab;
        }
    }
    return 0;
}
