/*
 * tilelens.h -- C ABI of the B200 (sm_100a) tile-major GEMM hot path.
 *
 * The operations are the ones the TileLens paper states: a weight matrix is
 * rewritten once into tile-major order (Section 3), a tiled matmul reads it
 * through tensor-map (TMA) views (Sections 2.3, 4.1, 4.2), and the read
 * amplification a G-byte-granular memory would see is counted per CTA tile
 * load (Sections 1, 2.5, 6.5).
 *
 * Conventions that hold for every call
 *   - Orientation.  The weight operand B is logically K x N.  "Row-major"
 *     keeps N contiguous; a memory tile ("block") is block_rows K-rows by
 *     block_cols contiguous N-columns, block_rows*block_cols*elem_bytes == G.
 *     Blocks are packed row-major over the block grid and are row-major
 *     inside (Eq. 1 and Eq. 2 with rows and columns exchanged, as Section 3.2
 *     allows).  The paper's (a, b) is (block_cols, block_rows).
 *   - Pointers named d_* or documented "device" are CUDA device pointers of
 *     the current device; h_* are host pointers.  The caller owns every
 *     buffer it passes.  Nothing the library allocates has to be freed by
 *     the caller.
 *   - Streams are `cudaStream_t` passed as void*; NULL is the default stream.
 *     Calls that take a stream enqueue work and return without waiting.
 *   - Every function returns a tl_status (0 = TL_OK).  Argument errors are
 *     found on the host before anything is enqueued.  A device-side wait that
 *     ran out (every wait in the kernels is bounded) raises a flag that
 *     tl_device_status() reports after synchronising.
 *   - Threads.  Host threads may call concurrently (the library serialises its own host-side work).  The stream
 *     and the workspace set by tl_set_stream() / tl_set_workspace() belong to the calling thread, like CUDA's
 *     current device; the internal split-K workspace belongs to the device, so calls that can run at the same
 *     time on one GPU (two streams, two threads) must each bring their own workspace.
 *   - Stream capture.  Every call that only enqueues work (the relayouts, the device-buffer products, tl_moe_ffn,
 *     tl_read_amp_async / tl_read_amp_batch, tl_hw_*) may be issued on a stream that is being captured into a CUDA
 *     graph, and the graph replays the same launches with the same bits: nothing a launch needs lives in host state
 *     that a replay would miss.  Two conditions.  The library's first use of a device, a kernel or a problem shape
 *     allocates and configures (control block, shared-memory attributes, tensor maps), which a capture forbids: make
 *     the same calls once before capturing.  And a captured launch whose schedule needs split-K scratch takes it only
 *     from the calling thread's workspace (tl_set_workspace), which must then live as long as the graph; without one
 *     it returns TL_ERR_WORKSPACE, because the internal workspace is replaced when a later call needs a larger one.
 *     tl_moe_ffn always runs as two launches while its stream is being captured.  tl_gemm_host, tl_read_amp and
 *     tl_device_status synchronise and are not for capture.
 *   - Divisibility (Section 3.3): rows % block_rows == 0 and
 *     cols % block_cols == 0, otherwise TL_ERR_INVALID_ARG; the caller pads.
 *     block_rows and block_cols must be powers of two (Section 3.2), otherwise
 *     TL_ERR_UNSUPPORTED.
 */
#ifndef TILELENS_H
#define TILELENS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TL_OK = 0,
    TL_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, G != rows*cols*s of the block, divisibility */
    TL_ERR_UNSUPPORTED = 2,   /* valid request outside what the kernels instantiate */
    TL_ERR_ALIGNMENT = 3,     /* pointer or pitch not aligned as the call requires */
    TL_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed: see tl_last_cuda_error() */
    TL_ERR_TIMEOUT = 5,       /* a bounded device-side wait expired, or a kernel refused an input (detail code) */
    TL_ERR_WORKSPACE = 6      /* caller-supplied workspace too small (or none, for a captured launch that needs scratch) */
} tl_status;

typedef enum { TL_TO_TILE_MAJOR = 0, TL_TO_ROW_MAJOR = 1 } tl_direction;
/* TL_LAYOUT_TILE_MAJOR_K: the K-contiguous flavour, Eq. 2 exactly as printed; block_rows x block_cols is then
 * the memory tile of the stored [N][K] array: b rows along N by a contiguous columns along K. */
typedef enum { TL_LAYOUT_ROW_MAJOR = 0, TL_LAYOUT_COL_MAJOR = 1, TL_LAYOUT_TILE_MAJOR = 2,
               TL_LAYOUT_TILE_MAJOR_K = 3 } tl_layout;

/* ------------------------------------------------------------------ misc */

const char* tl_status_string(int status);
/* Last cudaError_t / CUresult seen by a call that returned TL_ERR_CUDA (0 if none). */
int tl_last_cuda_error(void);
/* Stream used by the calling thread's calls that take none (tl_relayout, tl_read_amp*).  Default: NULL stream. */
int tl_set_stream(void* cuda_stream);
/* Synchronises the device, then returns TL_ERR_TIMEOUT if any kernel since the
 * last call gave up on a bounded wait (and clears the flag), else TL_OK.
 * *detail (may be NULL) receives a code saying which wait expired. */
int tl_device_status(uint32_t* detail);

/*
 * Switches of the library, process-wide.  None changes a result; they select between code paths that compute the
 * same thing (for measurement, and so that tests can reach every path), bound the device-side waits, or arm the
 * test hook below.  The paper has no counterpart.  Initial values may be preset through environment variables of the
 * names given in brackets (read once).
 */
typedef enum {
    TL_OPT_PDL = 0,          /* 1 (default): launches use programmatic stream serialisation, 0: plain stream order [TL_NO_PDL=1] */
    TL_OPT_PREFETCH_STAGES,  /* weight stages a GEMM CTA asks into L2 before it waits for its predecessor; -1 (default): up to 4 [TL_PREFETCH_STAGES] */
    TL_OPT_PAIR_KERNEL,      /* 1 (default): large dense products run on CTA pairs, 0: single-CTA kernel [TL_NO_PAIR=1] */
    TL_OPT_PAIR_512,         /* 1 (default): the pair kernel uses 512-token tiles where they fill whole waves, 0: 256-token tiles [TL_PAIR_HALVES=1] */
    TL_OPT_BOX_PER_BLOCK,    /* 0 (default): one TMA box per pipeline stage, 1: one box per memory tile [TL_BOX_PER_BLOCK] */
    TL_OPT_MAX_STAGES,       /* 0 (default): as many pipeline stages as fit, n >= 2: at most n [TL_MAX_STAGES] */
    TL_OPT_UMMA_M128,        /* 0 (default): 64-row MMAs for tiles of up to 64 tokens, 1: always 128 rows [TL_UMMA_M128] */
    TL_OPT_RELAYOUT_TMA,     /* 1 (default): copy-engine relayout where the shape allows, 0: shared-memory kernel [TL_RELAYOUT_NO_TMA=1] */
    TL_OPT_LOG,              /* 1: every GEMM launch prints the plan it chose to stderr [TL_LOG] */
    TL_OPT_WAIT_LIMIT_US,    /* bound of every device-side barrier wait, microseconds; default 2 000 000, accepted 100 .. 60 000 000 */
    TL_OPT_STALL_ONCE,       /* test hook: 1 = the next tl_gemm* launch, 2 = the next copy-engine relayout launch arms the
                                first pipeline stage of every CTA for 16 bytes more than its copies deliver, so that
                                the wait on that stage runs out after TL_OPT_WAIT_LIMIT_US, the kernel gives up (drains
                                its copies, frees tensor memory, returns) and tl_device_status() reports TL_ERR_TIMEOUT.
                                3 = in the next one-launch tl_moe_ffn CTA 0 does not arrive at the grid barrier, so every
                                CTA's bounded wait there runs out (detail 0x800); in the counter form
                                (TL_OPT_FFN_ONE_LAUNCH = 2) CTA 0 does not raise the counters of the m-tiles it stores,
                                so the waits of the producers that load them run out (detail 0x900).
                                That launch's output is undefined.
                                4 = the next grouped launch builds the tile tables it prepares ahead of its stream
                                predecessor's completion from wrong expert offsets, so that its check after the wait
                                must find them wrong and build them again; the output is the ordinary one.
                                The option resets itself to 0 when it is consumed. */
    TL_OPT_MOE_ROW_CAP,      /* grouped products: most token rows per tile; 0 (default): the library's choice (32, or 64 / 128 when
                                the experts average more than 24 / 48 rows and there are enough such tiles), else 16/32/64/128 */
    TL_OPT_REDUCE_SPLIT,     /* 1 (default): a split tile's partial sums are added by all reduction CTAs inside it, 0: by one */
    TL_OPT_SM_LIMIT,         /* 0 (default): GEMM grids use every SM; n > 0: at most n CTAs (leaves SMs to concurrent work) */
    TL_OPT_NO_SCRATCH_PLANS, /* 1 (default): dense decode-sized products prefer schedules without partial tiles in global
                                memory (whole tiles on a grid that divides the tile count, or split-K inside clusters);
                                0: always the stream-K cut */
    TL_OPT_FFN_ONE_LAUNCH,   /* 0 (default): tl_moe_ffn runs its two grouped products as two launches; where it can, 1: as two
                                phases of one cooperative launch with grid-wide barriers, 2: as one cooperative launch in which
                                the second product's loads wait, m-tile by m-tile, for the first product's rows (measured on the
                                Qwen-3 expert FFN: 203 us with two launches, 241 us and 220 us in one) */
    TL_OPT_GENERIC_RAW,      /* 1 (default): memory tiles of at least 8 rows whose rows are 16, 8, 4 or 2 bytes long are copied into
                                shared memory as stored (and, for 8- and 4-byte rows, transposed there in place) and read by the
                                MMA through a no-swizzle or K-major descriptor; 0: they take the permuting generic-address path */
    TL_OPT_PAIR_TMA_STORE,   /* 1 (default): the CTA-pair kernel writes C through shared memory with tiled bulk stores, 0: with
                                plain stores straight from the accumulator registers (same values either way) */
    TL_OPT_PLAN_AS_IF_SMS,   /* test hook, 0 (default) = off: n > 0 makes tl_gemm_plan answer as if the current device had n SMs,
                                without asking the CUDA runtime anything (co-resident clusters of S CTAs: those of a B200 when
                                n is 148, else n / S), so that the planning rules can be tested on a machine without a GPU.
                                Launches refuse to run while it is set (TL_ERR_INVALID_ARG). */
    TL_OPT_COUNT_
} tl_option;
/* TL_ERR_INVALID_ARG for an unknown option or a value outside the option's range. */
int tl_set_option(int option, int64_t value);
/* Current value; -1 for an unknown option. */
int64_t tl_get_option(int option);

/* -------------------------------------------------------------- relayout */

/*
 * Row-major <-> tile-major rewrite of a rows x cols matrix of elem_bytes-wide
 * elements (Section 3: same bytes, every contiguous G-byte block becomes a
 * block_rows x block_cols rectangle; Section 5.1: done once at weight load).
 *   d_src, d_dst  device, rows*cols*elem_bytes bytes each, must not overlap.
 *   elem_bytes    1, 2 or 4.          G == block_rows*block_cols*elem_bytes.
 *   direction     tl_direction.
 * Enqueues one kernel on the tl_set_stream() stream.  When cols*elem_bytes is
 * a multiple of 16 and both pointers are 16-byte aligned, block rows of 32
 * bytes to 1 KB in memory tiles of at most 32 KB are moved by the copy engine
 * (tensor copy on the row-major side, bulk copy on the tile-major side) and
 * every other shape by a 16-byte-vectorised kernel staged through shared
 * memory; otherwise an element-wise kernel runs (same result, slower).
 * rows == 0 or cols == 0 is a no-op.
 */
int tl_relayout(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int elem_bytes,
                int64_t G, int block_rows, int block_cols, int direction);
/* The same on an explicit stream. */
int tl_relayout_on(const void* d_src, void* d_dst, int64_t rows, int64_t cols, int elem_bytes,
                   int64_t G, int block_rows, int block_cols, int direction, void* cuda_stream);

/*
 * The same rewrite for n matrices that share element size, memory tile and direction (the weights of a layer at
 * load time, Section 5.1), in stream order.  d_srcs, d_dsts, rows, cols: HOST arrays of n entries (device
 * pointers, extents); each pair as in tl_relayout, no destination overlapping any other buffer of the call.
 * Matrices that can take the copy-engine path are moved by ONE launch per run of up to 8 of them, without a kernel
 * boundary in between; the others go through tl_relayout_on one by one.  The first matrix that fails
 * tl_relayout's argument checks ends the call with that error, the ones before it already enqueued.
 */
int tl_relayout_batch(int n, const void* const* d_srcs, void* const* d_dsts, const int64_t* rows, const int64_t* cols,
                      int elem_bytes, int64_t G, int block_rows, int block_cols, int direction, void* cuda_stream);

/* ------------------------------------------------------------------ GEMM */

/*
 * C[M x N] (fp32, row-major) = A[M x K] (bf16, row-major) x B[K x N] (bf16),
 * Section 2.3.  B is tile-major with G-byte blocks of block_rows x block_cols
 * (Section 3; read through the multi-dimensional tensor-map view of Section
 * 4.2, one TMA box per memory tile or per part of it inside the CTA tile), or
 * plain row-major when block_rows == 0 (then G and block_cols are ignored).
 * Products are accumulated in fp32 in tensor memory.
 *   d_A, d_B     device, 16-byte aligned (d_B 128-byte aligned when tile-major).
 *   d_C          device, 16-byte aligned, M*N floats, fully overwritten.
 *   cta_m/n/k    the CTA tile: cta_m token rows x cta_n weight columns per CTA,
 *                cta_k weight rows per pipeline stage.  0,0,0 lets the library
 *                choose (by M: M x 256 x 64 up to 64 rows, 128 x 128 x 128,
 *                128 x 256 x 64 or 256 x 256 x 64 up to 512 rows, whichever its
 *                planner ranks ahead for the shape, CTA pairs on 256- or 512-row tiles for
 *                prefill; tl_gemm_plan() tells).  Instantiated: cta_n in {64, 128, 256}, cta_k in {64, 128},
 *                cta_m in {16, 32, 64, 128, 256} (cta_n == 256: at most 128, or
 *                256 x 256 x 64 for dense problems whose tiles need no split
 *                of K: two 128-row token blocks share each weight slab).
 *                Tiles may overhang M, N and K.
 *   K % 8 == 0 (16-byte row pitch of A); tile-major: K % block_rows == 0,
 *   N % block_cols == 0; row-major: N % 64 == 0.  N % 4 == 0 (C is written in
 *   16-byte vectors; only the hand-addressed memory tiles of one or two
 *   columns could ask for less), else TL_ERR_UNSUPPORTED.
 *   Memory tiles whose rows are at least 32 bytes (16 columns) are read by
 *   TMA, whatever their height.  Narrower ones (block rows down to 2 bytes)
 *   are the generic-address case of Section 4.4.  With at least 8 rows they
 *   are still fetched by the copy engine as stored: 16-byte rows are read by
 *   the MMA as they are, single-column tiles as panels of a K-major operand,
 *   8- and 4-byte rows (up to 64 and 128 rows) after an in-place transpose in
 *   shared memory; block_rows | cta_k except for single-column tiles.  Tiles
 *   of fewer rows (and all of them when TL_OPT_GENERIC_RAW is 0) are permuted
 *   in shared memory with Eq. 1-2 arithmetic; there the memory tile must fit
 *   inside the CTA tile (block_rows | cta_k, block_cols | cta_n), G >= 16, and
 *   the CTA tile must leave room in shared memory for two raw images of a
 *   stage's weights beside two operand stages (cta_n * cta_k < 256 * 128),
 *   else TL_ERR_UNSUPPORTED.  One-row tiles are row-major.
 * When the output tiles do not fill the SMs (decode, small or grouped
 * problems) the K loops are cut: inside thread-block clusters whose CTAs
 * add their partial tiles through distributed shared memory where such a
 * schedule exists (no workspace), else stream-K fashion over all SMs, with
 * partial tiles going through a workspace and a second small kernel adding
 * them.  Either way the order of every sum is fixed: results are
 * reproducible run to run.  tl_gemm_plan() tells which schedule a call runs.
 * The workspace is the caller's (tl_set_workspace) or one the library grows
 * on demand; calls that may run concurrently on one GPU must not share a
 * workspace.
 * M == 0 is a no-op.
 */
int tl_gemm(const void* d_A_rowmajor, const void* d_B_tilemajor, float* d_C,
            int64_t M, int64_t N, int64_t K,
            int64_t G, int block_rows, int block_cols,
            int cta_m, int cta_n, int cta_k, void* cuda_stream);

/*
 * Grouped (mixture-of-experts) form, Section 2.3: rows of A are sorted by
 * expert; expert e owns rows [offsets[e], offsets[e+1]) and multiplies them
 * with its own K x N weight.  The E weights are separate tile-major (or
 * row-major) buffers of K*N*2 bytes laid end to end in d_B_experts.
 *   d_offsets    device, E+1 int32, non-decreasing, offsets[0] == 0,
 *                offsets[E] == total_rows.  Experts with no row cost nothing.
 *   d_C          total_rows x N floats; every row is written.
 * cta_m is an upper bound: each tile uses the smallest instantiated token
 * count that covers its rows.
 */
int tl_gemm_grouped(const void* d_A_sorted, const void* d_B_experts, float* d_C,
                    const int32_t* d_offsets, int E, int64_t total_rows,
                    int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                    int cta_m, int cta_n, int cta_k, void* cuda_stream);

/*
 * The expert FFN around the two grouped products (the paper names the fused MoE kernel as its workload, Section
 * 2.3 and 6.2, and is silent on what lies between the products; the gated form below is this library's choice).
 * tl_gemm_grouped_swiglu: tl_gemm_grouped whose N = 2*I weight columns hold gate_j in column 2j and up_j in column
 * 2j+1; instead of C it writes H[row][j] = bf16(silu(g) * u) (fp32 arithmetic, one rounding to nearest even),
 * d_H_bf16: total_rows x I bf16, 16-byte aligned.  N % 64 == 0; tiles of at most 128 rows (cta_m <= 128), else
 * TL_ERR_UNSUPPORTED.
 * tl_moe_ffn: that product followed by the grouped product of H and the experts' I x hidden down weights:
 * Y (fp32, total_rows x hidden) = H x W_down, no host synchronisation; d_H_bf16 is caller-owned scratch that holds H
 * afterwards.  Two launches in stream order (the second overlaps the first one's end through programmatic stream
 * serialisation).  With TL_OPT_FFN_ONE_LAUNCH = 1 and TMA-readable weights both products run as two phases of ONE
 * cooperative launch instead (a grid-wide barrier with a bounded wait between them; the split tiles of the first
 * product are summed inside the kernel, those of the second by the small reduction kernel that follows): same bits
 * as two launches.  With TL_OPT_FFN_ONE_LAUNCH = 2 the one launch has no barrier: the first product runs whole tiles
 * only, its epilogue counts every m-tile of H it has stored, and the second product's loads of an m-tile wait (with
 * a bound) for that count; a sum of H may then be taken in another order than with two launches (same tolerance).
 * Both one-launch forms are measured slower than two launches and need every CTA of their grid resident at once.
 */
/* tl_gemm / tl_gemm_grouped with C written as bf16 (fp32 accumulation, one rounding to nearest even): d_C_bf16
 * M x N (total_rows x N) bf16, 16-byte aligned, N % 8 == 0.  The paper leaves the output type open. */
int tl_gemm_bf16(const void* d_A_rowmajor, const void* d_B_tilemajor, void* d_C_bf16,
                 int64_t M, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                 int cta_m, int cta_n, int cta_k, void* cuda_stream);
int tl_gemm_grouped_bf16(const void* d_A_sorted, const void* d_B_experts, void* d_C_bf16,
                         const int32_t* d_offsets, int E, int64_t total_rows,
                         int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                         int cta_m, int cta_n, int cta_k, void* cuda_stream);
int tl_gemm_grouped_swiglu(const void* d_A_sorted, const void* d_B_experts_gate_up, void* d_H_bf16,
                           const int32_t* d_offsets, int E, int64_t total_rows,
                           int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                           int cta_m, int cta_n, int cta_k, void* cuda_stream);
int tl_moe_ffn(const void* d_X_sorted, const void* d_W_gate_up, const void* d_W_down, void* d_H_bf16, float* d_Y,
               const int32_t* d_offsets, int E, int64_t total_rows, int64_t hidden, int64_t inter,
               int64_t G, int block_rows, int block_cols, void* cuda_stream);

/*
 * The same products for weights stored the way deployments keep them (Section 2.4): [N][K] with K contiguous
 * (the "column-major" K x N matrix), tile-major exactly as Eq. 2 prints it: memory tiles of tile_k contiguous
 * K-elements (the paper's a) by tile_n rows along N (the paper's b), tile_n*tile_k*2 == G, tiles ordered along
 * K first.  tile_n == 0: the plain [N][K] array.  tl_relayout(rows = N, cols = K, block_rows = tile_n,
 * block_cols = tile_k) produces this buffer.  The weights are then the K-major operand of the MMA.
 *   tile_k >= 16 (a tile row is one swizzle row of 128, 64 or 32 bytes); N % tile_n == 0, K % tile_k == 0; the
 *   plain array needs K % 64 == 0; otherwise as tl_gemm and tl_gemm_grouped (experts laid end to end).  Shorter
 *   tile rows return TL_ERR_UNSUPPORTED: there is no generic-address path in this flavour.
 */
int tl_gemm_kmajor(const void* d_A_rowmajor, const void* d_B_nk_tilemajor, float* d_C,
                   int64_t M, int64_t N, int64_t K,
                   int64_t G, int tile_n, int tile_k,
                   int cta_m, int cta_n, int cta_k, void* cuda_stream);
int tl_gemm_grouped_kmajor(const void* d_A_sorted, const void* d_B_experts_nk, float* d_C,
                           const int32_t* d_offsets, int E, int64_t total_rows,
                           int64_t N, int64_t K, int64_t G, int tile_n, int tile_k,
                           int cta_m, int cta_n, int cta_k, void* cuda_stream);

/*
 * FP8 form (Section 3.1 and Figure 1(c): a 4 KB block of 8-bit elements is a 64 x 64 memory tile): A is M x K and
 * the weights are [N][K], both E4M3 bytes (bias 7, no infinities); C = A x B^T in fp32, products exact,
 * accumulation in fp32.  tile_n * tile_k == G; tile_k >= 32; the plain array (tile_n == 0) needs K % 128 == 0.
 * cta_k counts K elements and is 0, 128 or 256.  Everything else as tl_gemm_kmajor / tl_gemm_grouped_kmajor.
 */
int tl_gemm_fp8_kmajor(const void* d_A_rowmajor_fp8, const void* d_B_nk_tilemajor_fp8, float* d_C,
                       int64_t M, int64_t N, int64_t K,
                       int64_t G, int tile_n, int tile_k,
                       int cta_m, int cta_n, int cta_k, void* cuda_stream);
int tl_gemm_grouped_fp8_kmajor(const void* d_A_sorted_fp8, const void* d_B_experts_nk_fp8, float* d_C,
                               const int32_t* d_offsets, int E, int64_t total_rows,
                               int64_t N, int64_t K, int64_t G, int tile_n, int tile_k,
                               int cta_m, int cta_n, int cta_k, void* cuda_stream);

/* Bytes of workspace tl_gemm, or tl_gemm_grouped with any number of experts and M rows in total, may need for
 * these sizes on the current device (an upper bound: the grouped schedule of many experts cuts K over every SM). */
size_t tl_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k);
/* Hands the library a caller-owned device workspace (256-byte aligned) for the CALLING THREAD's GEMM calls;
 * (NULL, 0) returns to the device's internal one.  The buffer must stay valid until the last call using it has
 * finished. */
int tl_set_workspace(void* d_ptr, size_t bytes);

/*
 * The schedule a GEMM call with these sizes runs on the current device: the CTA grid of Section 2.3 as this
 * library cuts it.  Host-only; no pointer is needed and nothing is enqueued.  The same code chooses the plan of a
 * real launch, so feeding tl_read_amp* with (cta_m, cta_n, cta_k) from here counts exactly the tile loads the
 * kernel issues (Sections 2.5, 6.5).  E == 0: dense (tl_gemm*); E >= 1: grouped with E experts and M rows in
 * total.  flavour 0: N-contiguous bf16 weights (tl_gemm), 1: K-contiguous bf16 (tl_gemm_kmajor: block_rows =
 * tile_n, block_cols = tile_k), 2: K-contiguous FP8 (tl_gemm_fp8_kmajor).  Errors as the GEMM call itself
 * would return them for these sizes.
 */
typedef struct tl_gemm_plan_info {
    int32_t cta_m, cta_n, cta_k;   /* token rows x weight columns of one CTA's tile, weight rows (K elements) per stage.
                                      CTA-pair kernel: each CTA of a pair owns 128 of the pair's 256 columns and loads them
                                      once per tile of cta_m = 512 (or 256) token rows */
    int32_t pair_kernel;           /* 1: CTA pairs (cta_group::2), 0: single-CTA kernel */
    int32_t stream_k;              /* 1: K ranges cut over the CTAs + reduction kernel; 0: whole tiles */
    int32_t grid;                  /* CTAs launched */
    int32_t stages;                /* pipeline depth */
    int32_t weights_on_n;          /* 1: weights on the N side of the MMA (token tiles of up to 128 rows, or 256 x 256 x 64:
                                      two 128-row token blocks per tile) */
    int32_t generic_path;          /* 1: weights loaded by the generic-address path of Section 4.4 (permuted in shared
                                      memory); 2: memory tiles fetched as stored and read by the MMA as they are (16-byte
                                      rows, single-column tiles); 3: fetched as stored, 8- or 4-byte rows transposed in place */
    int32_t cluster_k;             /* S > 1: one tile per cluster of S CTAs that split its K loop (sums through distributed
                                      shared memory, no workspace); else 1 */
    int64_t pair_tiles_512, pair_tiles_256;   /* pair kernel: tiles of 512 and of 256 token rows (x 256 columns) */
    int32_t chained;               /* tl_gemm_last_plan after tl_moe_ffn: 1 when both products ran in one launch */
    int32_t reserved;
    uint64_t workspace_bytes;      /* split-K scratch the launch uses */
} tl_gemm_plan_info;
int tl_gemm_plan(int64_t M, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                 int cta_m, int cta_n, int cta_k, int E, int flavour, tl_gemm_plan_info* out);
/* What the calling thread's most recent GEMM launch ran (zeros before the first). */
int tl_gemm_last_plan(tl_gemm_plan_info* out);

/*
 * End-to-end form with host buffers: copies A and the ROW-MAJOR weight to the
 * device, rewrites the weight into tile-major blocks (block_rows == 0: keeps
 * it row-major), multiplies, copies C back and waits for it.
 *   h_A, h_B_rowmajor, h_C   host (pinned memory makes the copies asynchronous).
 *   d_scratch                device, at least tl_gemm_host_scratch_bytes() bytes, 256-byte aligned.
 */
int tl_gemm_host(const void* h_A, const void* h_B_rowmajor, float* h_C,
                 int64_t M, int64_t N, int64_t K, int64_t G, int block_rows, int block_cols,
                 int cta_m, int cta_n, int cta_k,
                 void* d_scratch, size_t scratch_bytes, void* cuda_stream);
size_t tl_gemm_host_scratch_bytes(int64_t M, int64_t N, int64_t K);

/*
 * tl_gemm for callers that must not allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the product above, same kernel;
 * to keep its scratch small it may pick a narrower CTA tile than tl_gemm, so
 * results agree with tl_gemm within the GEMM tolerance, exactly for inputs
 * whose partial sums are exact.)
 *
 * Who needs it: a serving process that hands all of HBM to its own pool at
 * start-up, so that any later cudaMalloc fails; a plug-in host or sandbox that
 * forbids allocation calls after initialisation; a latency-critical loop that
 * cannot afford the device-wide synchronisation an allocation or a free may
 * imply.  tl_gemm grows an internal workspace with cudaMalloc the first time a
 * decode-shaped problem needs split-K scratch; this entry point never calls
 * cudaMalloc, cudaFree or any allocating routine.  Its scratch (the partial
 * tiles of the split-K schedule) is a fixed array of TL_NOALLOC_SCRATCH_BYTES inside the
 * library image; every GPU that loads the library holds that much memory
 * until the process exits.
 *
 *   arguments     as tl_gemm, plus d_timeout_flag: a device uint32 the caller
 *                 owns and has zeroed, raised (non-zero) if a bounded wait in
 *                 the kernel expires; NULL keeps the flag in the array, unread.
 *   limit         problems whose split-K scratch exceeds the array return
 *                 TL_ERR_WORKSPACE and enqueue nothing.  The scratch is
 *                 2 * (number of SMs) * cta_m * cta_n * 4 bytes when the K
 *                 loops are cut over all SMs, which happens when the output
 *                 tiles do not fill the SMs evenly (fewer tiles than SMs, or
 *                 a last wave less than 92 % full) and no schedule without
 *                 partial tiles in global memory exists (tl_gemm_plan tells);
 *                 else 0; products that run on CTA pairs need none.  The
 *                 default tile here is 128 columns wide: on a 148-SM B200 that
 *                 admits every M <= 32; M in (32, 64] needs 9.3 MB when it is
 *                 cut and is then refused.
 *   first call    the first call on each device looks up the array's device
 *                 address (with that device current).  Make that call before
 *                 starting any stream capture.
 *   sharing       all calls share the one array, and it keeps the previous
 *                 call's contents; nothing in it has to start at zero, because
 *                 every partial tile is written by the GEMM kernel before the
 *                 reduction kernel of the same call reads it.  Two calls that can run at
 *                 the same time on one GPU (different streams, or different
 *                 host threads) race on the array and give wrong results:
 *                 serialise them.
 */
#define TL_NOALLOC_SCRATCH_BYTES (8u << 20)
int tl_gemm_noalloc(const void* d_A_rowmajor, const void* d_B_tilemajor, float* d_C,
                    int64_t M, int64_t N, int64_t K,
                    int64_t G, int block_rows, int block_cols,
                    int cta_m, int cta_n, int cta_k,
                    uint32_t* d_timeout_flag, void* cuda_stream);

/* ------------------------------------- tile-major aware box loads (TileLens-HW) */

/*
 * Section 4.3 proposes to extend the TMA's source-address computation so that kernels keep their tensor views and
 * only the descriptor changes.  These two calls emulate that engine in software on a tile-major buffer.
 * The descriptor is a tensor-map-like VIEW of the column-major K x N matrix (K contiguous): extents, strides and
 * box in ELEMENTS, strides[0] == 1, the other dimensions in any order, plus the two fields the section adds:
 * the memory tile (tile_a contiguous K-elements x tile_b columns, Eq. 1-2) and the leading stride K.
 * Covered, as in the section: box[0] = u a power of two with u == tile_a (case 1) or u dividing tile_a (case 2);
 * the box extent in the dimension whose stride equals K a multiple of tile_b; every other stride either below K
 * and a multiple of u, or a multiple of tile_b*K.  Anything else returns TL_ERR_UNSUPPORTED (TL_ERR_INVALID_ARG
 * for malformed descriptors).  Coordinates must be tile-aligned (Eq. 4) and the box inside the tensor; a box that
 * is not raises the status word (tl_device_status() -> TL_ERR_TIMEOUT with detail 0x900) and is skipped.
 */
typedef struct tl_hw_desc {
    int32_t rank;              /* 2..5 */
    int32_t elem_bytes;        /* s: 1, 2 or 4 */
    int64_t dims[5];
    int64_t strides[5];
    int32_t box[5];
    int32_t tile_a, tile_b;    /* field 1: memory tile, tile_a * tile_b * s = G */
    int64_t leading_stride;    /* field 2: K */
} tl_hw_desc;

/*
 * Source byte offsets (into the tile-major buffer) of every element of n_boxes box loads, in the order the
 * engine's counters produce them (dimension 0 fastest): d_offsets[box * prod(box) + t].  Skipped boxes are
 * filled with ~0.  desc: host.  d_coords: device, n_boxes x rank int32.  d_offsets: device.  Asynchronous.
 */
int tl_hw_box_offsets(const tl_hw_desc* desc, const int32_t* d_coords, int64_t n_boxes, uint64_t* d_offsets,
                      void* cuda_stream);
/*
 * The loads themselves: box i lands densely at d_dst + i * prod(box) * s in coordinate order (the destination
 * address "simply increments", Section 4.3), read from the tile-major buffer d_src_tilemajor of src_bytes bytes
 * (the K x N matrix as tl_relayout(rows = N, cols = K, block_rows = tile_b, block_cols = tile_a) writes it).
 * Nothing outside [0, src_bytes) is read.  Asynchronous on cuda_stream.
 */
int tl_hw_box_load(const tl_hw_desc* desc, const void* d_src_tilemajor, uint64_t src_bytes, const int32_t* d_coords,
                   int64_t n_boxes, void* d_dst, void* cuda_stream);

/* --------------------------------------------------- read amplification */

/*
 * Read amplification of the weight operand under access granularity G
 * (Sections 1, 2.5; "requests per compute tile" of Section 6.5).  The schedule
 * is the GEMM's: ceil(M/cta_m) x ceil(N/cta_n) CTA tiles, ceil(K/cta_k)
 * iterations, each loading the clipped cta_k x cta_n rectangle of B.  Per
 * load, the distinct G-byte blocks holding any byte of the rectangle are
 * counted (B starts on a G boundary); nothing is shared between loads.
 *   bytes_fetched = sum of blocks * G,  bytes_used = sum of rectangle bytes,
 *   requests (may be NULL) = sum of blocks.  All host out-parameters; exact.
 * layout is a tl_layout; block_rows/block_cols only matter for the two tile-major flavours.
 * Any positive tile sizes are accepted (not only the GEMM's).  Runs one small
 * kernel (one warp per CTA tile) on the tl_set_stream() stream and waits.
 */
int tl_read_amp(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                uint64_t* bytes_fetched, uint64_t* bytes_used, uint64_t* requests);

/*
 * The same count when CTAs share requests (Section 2.5: CTAs that want the same 4 KB request; Section 6.5: a
 * request another CTA already issued): the wave_ctas CTA tiles resident together (tiles numbered n-tile major,
 * m-tile minor, wave w = tiles [w*wave_ctas, (w+1)*wave_ctas)) step through K together, and a block several of
 * them want at the same step is fetched once.  bytes_needed = the distinct weight bytes a wave uses per step,
 * summed.  wave_ctas == 1 gives tl_read_amp's numbers.  Host out-parameters, exact; waits like tl_read_amp.
 */
int tl_read_amp_shared(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k, int64_t wave_ctas,
                       int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                       uint64_t* bytes_fetched, uint64_t* bytes_needed, uint64_t* requests);

/*
 * Eq. 6 (Section 5.2): the stride-prefetch degree that keeps a bus of the given bandwidth busy over the given
 * read latency: d = min(floor(c * B*L / p_wave), K / cta_k), B*L counted in requests of G bytes, p_wave = n_sm *
 * ctas_per_sm * requests_per_tile (the per-tile request count tl_read_amp reports, divided by tiles and
 * iterations); c = 1 as printed, 2 as the text uses in practice.  Host arithmetic only; -1 for bad arguments.
 */
int64_t tl_prefetch_degree(double bandwidth_bytes_per_s, double latency_s, int64_t G, int64_t n_sm,
                           int64_t ctas_per_sm, int64_t requests_per_tile, int64_t K, int64_t cta_k,
                           double collision_factor);

/*
 * What the request count of a tile costs in time (Section 6.5, "Straggler-Induced CTA Stalls"): a CTA issues the
 * requests of a compute tile together and starts when the LAST one has arrived; the more requests, the likelier that
 * the slowest falls in the tail of the per-request latency distribution.  The paper shows its distribution only in
 * figures, so the caller supplies one: h_latencies, `count` measured per-request latencies (any unit), read as the
 * distribution that gives each sample value probability 1/count, the `requests` requests of a tile as independent
 * draws from it (requests = tl_read_amp's request count divided by tile loads).  Returns the expected time to the
 * first arrival (the section's "queueing" phase), to the last arrival (first + "straggler wait"), and, if p_late
 * is not NULL, the probability that the last arrival comes after `threshold`.  Host arithmetic only.
 * TL_ERR_INVALID_ARG for an empty sample, a NaN, or requests <= 0.
 */
int tl_tile_arrival_latency(const double* h_latencies, int64_t count, int64_t requests, double threshold,
                            double* first_arrival, double* last_arrival, double* p_late);

/*
 * tl_read_amp without the wait: the three totals (bytes_fetched, bytes_used, requests) are written to d_totals,
 * 3 uint64 in DEVICE memory (or mapped pinned host memory), by the kernel's last CTA.  Asynchronous on
 * cuda_stream; successive counter calls must be ordered by one stream (they share their accumulators).
 */
int tl_read_amp_async(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                      int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                      uint64_t* d_totals, void* cuda_stream);

/*
 * Up to 16 tl_read_amp_async configurations in one kernel launch (the counters of all products of a step).
 * h_cfgs: HOST array of n configurations; d_totals: DEVICE, n x 3 uint64 in the order of h_cfgs.  Asynchronous.
 */
typedef struct tl_read_amp_cfg {
    int64_t M, N, K;
    int32_t cta_m, cta_n, cta_k, layout;
    int64_t G;
    int32_t block_rows, block_cols, elem_bytes, reserved;
} tl_read_amp_cfg;
int tl_read_amp_batch(const tl_read_amp_cfg* h_cfgs, int n, uint64_t* d_totals, void* cuda_stream);

/* Grouped form: sum over experts with rows; h_offsets is a HOST array of E+1 int32. */
int tl_read_amp_grouped(const int32_t* h_offsets, int E, int64_t N, int64_t K,
                        int cta_m, int cta_n, int cta_k,
                        int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                        uint64_t* bytes_fetched, uint64_t* bytes_used, uint64_t* requests);

/* Per-CTA-tile form: d_fetched / d_used are DEVICE arrays of
 * ceil(M/cta_m)*ceil(N/cta_n) uint64, m-tile major.  Asynchronous on cuda_stream. */
int tl_read_amp_per_cta(int64_t M, int64_t N, int64_t K, int cta_m, int cta_n, int cta_k,
                        int layout, int64_t G, int block_rows, int block_cols, int elem_bytes,
                        uint64_t* d_fetched, uint64_t* d_used, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* TILELENS_H */
