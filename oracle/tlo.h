/*
 * tlo -- TileLens ORACLE.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct CPU statement of what the tile-major hot
 * path computes: the layout index functions, the relayout permutation, the
 * fp64 matrix product and the brute-force count of G-byte blocks touched by
 * every weight-tile load.  Nothing here is blocked, fused or reordered beyond
 * what the paper's definitions state, and nothing here is shared with the
 * CUDA library (no common header, helper, table or constant).  Only tests,
 * the smoke check and the CPU-baseline leg of the benchmark may call it; the
 * product path never does.
 *
 * Orientation (one reading used everywhere): the weight operand B is logically
 * K x N and is stored with N contiguous ("row-major" as in Section 2.4 and the
 * 128x256 example of Section 6.5, where each tile row is one contiguous strip).
 * The paper writes its equations for the K-contiguous (column-major) flavour
 * and states that the other flavour follows by exchanging rows and columns
 * (Section 3.2); tlo_off_tile is that exchanged form, tlo_eq2 is the literal
 * printed form, and the tests check one against the other.
 *
 * Pins (see tests/test_oracle_*.py): every function below is pinned to values
 * the paper prints, to closed forms, to invariants or to brute force on tiny
 * inputs.  No function here is "parity unpinned".
 */
#ifndef TLO_H
#define TLO_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* TLO_TILE_MAJOR_K is the tile-major layout exactly as the paper prints it (Eq. 2): the K x N weight with K
 * contiguous, memory tile a (along K) x b (along N); there br/bc of the calls below carry (b, a). */
enum { TLO_ROW_MAJOR = 0, TLO_COL_MAJOR = 1, TLO_TILE_MAJOR = 2, TLO_TILE_MAJOR_K = 3 };
enum { TLO_TO_TILE_MAJOR = 0, TLO_TO_ROW_MAJOR = 1 };

/* Section 2.4: byte offset of element (r,c) of a rows x cols matrix of s-byte
 * elements when a row / a column is contiguous. */
int64_t tlo_off_row(int64_t r, int64_t c, int64_t rows, int64_t cols, int64_t s);
int64_t tlo_off_col(int64_t r, int64_t c, int64_t rows, int64_t cols, int64_t s);

/* Eq. 1 + Eq. 2 with rows and columns exchanged (Section 3.2, first sentence):
 * memory tile = br rows x bc contiguous columns; tiles ordered row-major over
 * the tile grid, elements row-major inside a tile. */
int64_t tlo_off_tile(int64_t r, int64_t c, int64_t rows, int64_t cols,
                     int64_t br, int64_t bc, int64_t s);

/* One switch over the three layouts (layout = TLO_*_MAJOR). */
int64_t tlo_off(int layout, int64_t r, int64_t c, int64_t rows, int64_t cols,
                int64_t br, int64_t bc, int64_t s);

/* Eq. 1 as printed: out = {i', j', T_i, T_j} for memory tile a x b. */
void tlo_eq1(int64_t i, int64_t j, int64_t a, int64_t b, int64_t out[4]);
/* Eq. 2 as printed (K x N matrix, K contiguous, memory tile a x b). */
int64_t tlo_eq2(int64_t i, int64_t j, int64_t K, int64_t N, int64_t a, int64_t b, int64_t s);
/* Eq. 3: the 4-D coordinate of Eq. 1 dotted with stride (1, a, ab, Kb), in bytes. */
int64_t tlo_eq3(int64_t i, int64_t j, int64_t K, int64_t N, int64_t a, int64_t b, int64_t s);

/* Section 4.3 "Default tile-major for LGMS allocations" / Section 5.1: the
 * weights are rewritten once into tile-major order; same bytes, new places.
 * Copies every element through the index functions.  Returns 0, or -1 when
 * br/bc do not divide rows/cols (Section 3.3 requires divisibility). */
int tlo_relayout(const void* src, void* dst, int64_t rows, int64_t cols, int64_t s,
                 int64_t br, int64_t bc, int direction);

/* bf16 bit pattern -> double (exact: bf16 is a prefix of binary32). */
double tlo_bf16_to_double(uint16_t h);

/* Section 2.3: C = A x B with A M x K (bf16, row-major) and B K x N (bf16,
 * stored in `layout` with memory tile br x bc), evaluated only at the n listed
 * (idx_i[t], idx_j[t]) positions, as the plain sum over k in fp64.
 * C[t] = sum_k A[i][k]*B[k][j];  S[t] = sum_k |A[i][k]*B[k][j]|. */
int tlo_matmul_at(const uint16_t* A, const uint16_t* B, int layout, int64_t br, int64_t bc,
                  int64_t M, int64_t N, int64_t K, int64_t n,
                  const int64_t* idx_i, const int64_t* idx_j, double* C, double* S);
/* The same at every (i,j): C and S are M x N row-major. */
int tlo_matmul(const uint16_t* A, const uint16_t* B, int layout, int64_t br, int64_t bc,
               int64_t M, int64_t N, int64_t K, double* C, double* S);

/* FP8 (E4M3, the no-infinity encoding: bias 7, S.1111.111 = NaN) bit pattern -> double, exact. */
double tlo_fp8_e4m3_to_double(uint8_t h);
/* tlo_matmul_at on FP8 operands (s = 1; Section 3.1 and Figure 1(c) use FP8 with 64 x 64 memory tiles). */
int tlo_matmul_at_fp8(const uint8_t* A, const uint8_t* B, int layout, int64_t br, int64_t bc,
                      int64_t M, int64_t N, int64_t K, int64_t n,
                      const int64_t* idx_i, const int64_t* idx_j, double* C, double* S);

/* Sections 1, 2.5, 6.5: read amplification of the weight operand under access
 * granularity G.  The tiled product has ceil(M/BM) x ceil(N/BN) CTA tiles and
 * ceil(K/BK) iterations; each (CTA tile, iteration) loads the clipped BK x BN
 * rectangle of B.  For every such load, the set of distinct G-byte blocks that
 * hold any byte of the rectangle is built element by element; fetched += |set|*G,
 * used += elements*s, requests += |set|.  No sharing is credited between loads.
 * If per_tile_fetched/used are non-NULL they receive one entry per
 * (m-tile, n-tile), m-tile major. */
int tlo_read_amp(int64_t M, int64_t N, int64_t K, int64_t BM, int64_t BN, int64_t BK,
                 int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                 uint64_t* fetched, uint64_t* used, uint64_t* requests,
                 uint64_t* per_tile_fetched, uint64_t* per_tile_used);

/* Section 2.3 (MoE: every expert performs the same product): the same count
 * summed over experts e with offsets[e+1]-offsets[e] > 0 rows, each expert's
 * K x N weight its own G-aligned allocation. */
int tlo_read_amp_grouped(const int32_t* offsets, int E, int64_t N, int64_t K,
                         int64_t BM, int64_t BN, int64_t BK,
                         int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                         uint64_t* fetched, uint64_t* used, uint64_t* requests);

/* Sections 2.5 / 6.5 (CTAs share requests): as tlo_read_amp, but the P CTA tiles resident together (tiles numbered
 * n-tile major, m-tile minor; wave w = tiles [w*P, (w+1)*P)) step through K together and fetch a block once per
 * step however many of them want it.  needed = distinct weight bytes the wave's tiles use per step, summed.
 * P = 1 reproduces tlo_read_amp.  The paper's 10.1x / 3.9x come from its simulator's caches and are not this
 * count: the function is pinned to closed forms and to tlo_read_amp, not to those figures. */
int tlo_read_amp_shared(int64_t M, int64_t N, int64_t K, int64_t BM, int64_t BN, int64_t BK, int64_t P,
                        int layout, int64_t G, int64_t br, int64_t bc, int64_t s,
                        uint64_t* fetched, uint64_t* needed, uint64_t* requests);

/* Eq. 6 (Section 5.2): stride-prefetch degree d = min(floor(c*B*L/p_wave), K/TILE_K), B*L in requests of G bytes,
 * p_wave = n_sm * ctas_per_sm * p_tile; c = 1 as printed, 2 "in practice".  Pinned by the inequality the paper
 * derives it from (p_wave*(d+1) >= B*L > p_wave*d when not capped) and its monotonicity, not by a printed value. */
/* Section 6.5: expected time to the first and to the last arrival of the n requests of a compute tile, and the
 * probability that the last one arrives after `threshold`, for per-request latencies drawn independently from the
 * caller's sample (probability 1/N per value). */
int tlo_tile_arrival(const double* samples, int64_t N, int64_t n, double threshold, double* first, double* last,
                     double* p_late);
int64_t tlo_prefetch_degree(double bandwidth_bytes_per_s, double latency_s, int64_t G, int64_t n_sm, int64_t ctas_per_sm,
                            int64_t p_tile, int64_t K, int64_t tile_k, double collision_factor);

/* Section 4.3 (tile-major aware TMA): a tensor-map-like descriptor of a VIEW of the column-major K x N matrix
 * (dims/strides/box in elements, strides[0] == 1, dimension 0 contiguous) extended by the two fields the paper
 * adds: the memory tile (a, b), a contiguous, and the leading stride K. */
typedef struct {
    int32_t rank;            /* 2..5 */
    int32_t s;               /* element bytes */
    int64_t dims[5];
    int64_t strides[5];
    int64_t box[5];          /* the TMA tile; box[0] = u, and v = the extent in the dimension whose stride is K */
    int64_t a, b;            /* field 1 */
    int64_t K;               /* field 2 */
} tlo_hw_desc;

/* The source byte offset of every element of one box load at `coords`, in the order the engine's counters
 * produce them (dimension 0 fastest), computed the way Section 4.3 describes the hardware: split-and-sum of
 * coordinate x stride products into i and K*j, tileBase by Eq. 4, the stride-K counter replaced by two nested
 * counters (Eq. 5), and for a > u (Case 2) everything as if the memory tile were u x b followed by the bit
 * permutation of the intra-tile offset.  out holds prod(box) entries.  Returns 0, or -1 for a descriptor or
 * coordinate the section does not cover (u > a, v not a multiple of b, unaligned coordinates, a stride that is
 * neither below K and a multiple of u, equal to K, nor a multiple of b*K). */
int tlo_hw_box_offsets(const tlo_hw_desc* d, const int64_t* coords, int64_t* out);

/* double -> bf16 bits (round to nearest even) and silu(x) = x / (1 + exp(-x)). */
uint16_t tlo_double_to_bf16(double x);
double tlo_silu(double x);
/* Gated expert FFN around the two grouped products of the MoE workload (Section 2.3; the paper is silent on what
 * lies between them): h = bf16(silu(x Wg) * (x Wu)), y = h Wd, gate/up columns interleaved (2j, 2j+1) in the
 * hidden x 2I weight, for the listed rows of the expert-sorted X.  H_out: n_rows x I bf16 bits, Y_out and
 * S_out (sum of |h * w| terms): n_rows x hidden doubles. */
int tlo_moe_ffn_rows(const uint16_t* X, const uint16_t* W_gu, const uint16_t* W_down, const int32_t* offsets, int E,
                     int64_t hidden, int64_t I, int layout, int64_t br, int64_t bc,
                     int64_t n_rows, const int64_t* rows, uint16_t* H_out, double* Y_out, double* S_out);

/* Threads the parallel loops above will use. */
int tlo_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
