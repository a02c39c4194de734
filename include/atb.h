/* atb.h - C ABI of the asymmetric-tile-buffered BFP16 x BF16 GEMM library for NVIDIA B200 (sm_100a).
 *
 * The library computes C = A x B (Section 1 of "Can Asymmetric Tile Buffering Be Beneficial?")
 * with A in BFP16 block floating point (Section 2.4: blocks of 8 values share one 8-bit
 * exponent, 8-bit mantissas, 9 bytes per block), B in BF16, FP32 accumulation and BF16 output,
 * tiled with asymmetric tile buffering (Section 3): the output tile keeps T_MC rows live while A
 * is buffered only T_MA <= T_MC rows at a time.
 *
 * General rules
 *   - Plain C.  Every pointer named *_dev is DEVICE memory owned by the caller (any allocator);
 *     pointers without that suffix are HOST memory.  The library never allocates or frees device
 *     memory and keeps no reference to caller memory after a call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Device work is
 *     asynchronous on that stream; the calls return as soon as it is enqueued.  They only enqueue kernels
 *     (tensor maps travel by value as kernel parameters), so a sequence of calls can be captured into a
 *     CUDA graph and replayed on the same buffers.
 *   - Argument errors are returned synchronously and nothing is launched.  No exception or abort
 *     crosses this boundary.  atb_last_error_message() gives a per-thread detail string.
 *   - The device must have compute capability 10.0; there is no fallback of any kind.
 *
 * BFP16 storage (the logical format is the paper's; the planar device layout is this library's)
 *   - mantissa plane: int8  mant[M][K], row-major, two's complement in [-127, 127];
 *   - exponent plane: uint8 exp[ceil(K/64)][M_pad][8], M_pad = M rounded up to a multiple of 32:
 *     the 8 block exponents of row m that cover columns 64p .. 64p+63 sit in 8 consecutive bytes
 *     at ((p * M_pad) + m) * 8.  Entries of padded rows / blocks are zero.
 *   - value of element (m, k) = mant[m][k] * 2^(E - 133), E = exponent of block (m, k / 8).
 */
#ifndef ATB_H_
#define ATB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ATB_OK = 0,
    ATB_ERR_NULL_POINTER = 1,
    ATB_ERR_BAD_SHAPE = 2,          /* M, N, K or a leading dimension is not acceptable        */
    ATB_ERR_BAD_TILING = 3,         /* the (T_MA, T_MC, T_K, T_N) tuple is not supported        */
    ATB_ERR_MISALIGNED = 4,         /* a pointer or stride breaks the 16-byte rules below       */
    ATB_ERR_UNSUPPORTED_DEVICE = 5, /* current device is not compute capability 10.0            */
    ATB_ERR_CUDA = 6,               /* a CUDA runtime / driver call failed (see the message)    */
    ATB_ERR_BUFFER_TOO_SMALL = 7,   /* an output array given by the caller is too short         */
    ATB_ERR_DEVICE_TIMEOUT = 8      /* a kernel gave up a bounded wait (reported by atb_device_status) */
} atb_status_t;

/* Name of a status code; never NULL. */
const char* atb_status_string(atb_status_t status);
/* Detail of the calling thread's most recent failing call ("" if none); never NULL. */
const char* atb_last_error_message(void);

/* Asymmetric tiling 4-tuple of Section 3: A is buffered T_MA x T_K, B T_K x T_N, C T_MC x T_N;
 * rho = T_MC / T_MA >= 1, rho = 1 is conventional symmetric buffering. */
typedef struct { int T_MA, T_MC, T_K, T_N; } atb_tiling_t;

/* Sizes in bytes of the two BFP16 planes of an M x K matrix (K a multiple of 8). */
size_t atb_bfp16_mant_bytes(int64_t M, int64_t K);   /* M * K                                  */
size_t atb_bfp16_exp_bytes(int64_t M, int64_t K);    /* ceil(K/64) * roundup(M, 32) * 8        */

/* BFP16 quantisation (format: Section 2.4; the paper leaves the algorithm open, so this is the
 * library's definition).  For every row m and block kb (columns 8kb .. 8kb+7):
 *   amax = largest |x| of the block, NaNs ignored;
 *   E    = biased fp32 exponent field of amax, 0 if amax is zero or subnormal, at most 254;
 *   m_k  = round-to-nearest-even(x_k / 2^(E-133)) saturated to [-127, 127]; NaN -> 0, +-Inf -> +-127.
 * A_dev:    fp32 A[M][lda], row-major, lda >= K elements, 16-byte aligned, lda % 4 == 0.
 * mant_dev: atb_bfp16_mant_bytes(M, K) bytes, 16-byte aligned.
 * exp_dev:  atb_bfp16_exp_bytes(M, K) bytes, 16-byte aligned; padding entries are written as 0.
 * Requires M >= 0, K >= 0, K % 8 == 0.  M == 0 or K == 0 is a no-op returning ATB_OK. */
atb_status_t atb_quantize_bfp16(const float* A_dev, int64_t M, int64_t K, int64_t lda,
                                int8_t* mant_dev, uint8_t* exp_dev, void* stream);

/* C = dequant(A) x B with the asymmetric tile buffering schedule of Section 3 (output-stationary:
 * per K-step the T_K x T_N tile of B is loaded once and rho = T_MC / T_MA slabs of A are streamed
 * through it; the T_MC x T_N FP32 accumulator is written out once, after K / T_K steps).
 * FP32 accumulation, one round-to-nearest-even to BF16 at the end.
 *   A_mant_dev, A_exp_dev: the planes described above (16-byte aligned); every exponent byte is
 *               taken as written (element = m * 2^(E-133), exactly, as a bf16 operand: bf16-subnormal for
 *               E < 7, +-Inf where E = 255 takes it beyond bf16); mantissa -128, which the quantiser never
 *               writes, is not a valid input;
 *   B_bf16_dev: bf16 B[K][ldb] row-major, ldb >= N, ldb % 8 == 0, 16-byte aligned;
 *   C_bf16_dev: bf16 C[M][ldc] row-major, ldc >= N, ldc % 8 == 0, 16-byte aligned (written).
 * Shapes: M >= 1 (any value), N >= 8 with N % 8 == 0, K >= 16 with K % 16 == 0.  Edge tiles in M, N and
 *         K are handled (TMA zero-fills loads past the edge and clips stores).
 * Tilings: T_MC in {128, 256, 384}; T_N in {64, 128, 256, 512}; T_K in {64, 128};
 *          T_MA in {32, 64, 128, 256} dividing T_MC (rho = T_MC / T_MA is 1, 2, 3, 4, 6, 8 or 12:
 *          T_MC = 384 gives the ratios that are not powers of two); (T_MC / 128) * T_N <= 512 (the FP32
 *          accumulator must fit the 512 TMEM columns); the shared-memory rings must fit 227 KB.
 *          atb_tiling_supported() tells in advance.
 *          (T_MC, T_K, T_N) = (256, 64, 512) runs on a pair of SMs (tcgen05 cta_group::2): each SM holds 128
 *          rows of the tile and the whole 512-column accumulator for them, the B tile is shared by the two
 *          (the array-level sharing of Eq. 2).  Per SM - the paper's "core" - the accumulator is 128 rows
 *          tall, so T_MA = 128 is this tiling's SYMMETRIC form (rho per core = 128 / T_MA), only
 *          T_MA in {32, 64} buffer asymmetrically, and T_MA = 256 does not exist (ATB_ERR_BAD_TILING).
 *          (T_MC, T_K, T_N) = (128, 128, 256) runs on a pair of SMs too where M > 128: the pair computes two
 *          128 x 256 tiles, one above the other, one per SM, and shares their B tiles between them (Eq. 2 again);
 *          each SM keeps its 128 x 256 accumulator twice, so the write-out of a tile runs beside the K loop of the
 *          next one - the tiling of choice where K is shallow or the output is small.  T_MA = 128 is its symmetric
 *          form, T_MA in {32, 64} buffer asymmetrically.  Where M <= 128 there is one tile row and nothing to share:
 *          the tiling then runs on single SMs.  atb_tiling_plan() reports the pair's plan.
 * For fixed (T_MC, T_K, T_N) the result is bit-identical for every T_MA, and every call with the same
 * arguments on the same GPU model gives the same bits.  Between different (T_MC, T_K, T_N) results agree
 * within FP32 rounding, not bit for bit: a persistent CTA walks K upwards for one of its tiles and downwards
 * for the next (the next wave of tiles then starts on data the L2 still holds), so the order of a tile's
 * additions depends on its place in the walk; only where no CTA computes more than one tile do all
 * tilings with the same T_K add in the same order.
 * Errors: NULL_POINTER, BAD_SHAPE, BAD_TILING, MISALIGNED, UNSUPPORTED_DEVICE, CUDA. */
atb_status_t atb_gemm(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                      const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                      const void* B_bf16_dev, int64_t ldb,
                      void* C_bf16_dev, int64_t ldc, void* stream);

/* Split-K variant of atb_gemm for shapes with few output tiles (M x N small, K large): every
 * T_MC x T_N tile is computed as `splits` partial tiles over disjoint K ranges, written in FP32 to a
 * caller-provided workspace and summed (FP32) into the BF16 result by a second kernel on the same
 * stream.  The paper's hardware cannot do this - Section 2.2: an AIE core has no way to bring partial
 * sums back, so every output tile is fully accumulated in L1 - here partial sums go through L2/HBM.
 * Same operands and rules as atb_gemm.  Tilings: T_K = 64, T_MC in {128, 256}, T_N in {128, 256},
 * T_MA in {64, 128}.  splits in [1, min(64, ceil(K / T_K))]; splits * roundup(M, T_MC) must stay below 2^31
 * (the row coordinate of the partial tiles is a 32-bit TMA coordinate), else ATB_ERR_BAD_SHAPE.
 *   workspace_dev: device memory, 16-byte aligned, at least atb_gemm_splitk_workspace_bytes() bytes;
 *                  fully overwritten; may be reused by the next call on the same stream.
 * Errors: as atb_gemm, plus ATB_ERR_BUFFER_TOO_SMALL. */
size_t atb_gemm_splitk_workspace_bytes(int64_t M, int64_t N, int T_MC, int splits);
atb_status_t atb_gemm_splitk(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                             const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                             const void* B_bf16_dev, int64_t ldb,
                             void* C_bf16_dev, int64_t ldc,
                             int splits, float* workspace_dev, size_t workspace_bytes, void* stream);
/* Number of K splits (a power of two, 1 = use atb_gemm) that the host heuristic expects to be
 * fastest for this shape and tile: fills the SMs, keeps >= 8 K-steps per split, and charges the FP32
 * partials' traffic.  Host only. */
int atb_select_splits(int64_t M, int64_t N, int64_t K, int T_MC, int T_K, int T_N);

/* atb_gemm_splitk for callers that must not allocate.  (The paper has no counterpart: this is an
 * integration convenience of this library, not part of the method.)
 *
 * Who needs it: code that sits under somebody else's memory manager - an operator plugged into an
 * inference server or a framework whose pool has claimed the device memory, where a stray cudaMalloc
 * can fail, fragment the pool or stall every stream with its implicit synchronisation - and
 * latency-bound loops that are simply forbidden to call an allocator after start-up.  Such callers
 * still pass the operands and the result; what they are spared is finding room for the FP32 partial
 * sums.  Those go to a fixed array of ATB_NOALLOC_SCRATCH_BYTES that is linked into the library: every
 * GPU that loads the library keeps that much memory reserved until the process ends, used or not.
 *
 * Same arguments, tilings and results as atb_gemm_splitk (bit for bit), minus the workspace pair.
 *   - Limit: atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits) must not exceed
 *     ATB_NOALLOC_SCRATCH_BYTES, else ATB_ERR_BUFFER_TOO_SMALL and nothing is launched (e.g. 1024 x 1024
 *     with up to 16 splits, 2048 x 2048 with up to 4).
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - The first call on each device looks the array's device address up (cudaGetSymbolAddress, with
 *     that device current) and remembers it; make that first call before starting any stream capture.
 *   - When the array's memory is actually set aside: when the CUDA runtime loads the library's GEMM module
 *     on a device.  With lazy module loading (the default of recent CUDA versions) that happens inside the
 *     first GEMM-family call of this library on that device - possibly this one - and it can fail there
 *     with ATB_ERR_CUDA if the device has less than ATB_NOALLOC_SCRATCH_BYTES free.  So make one priming
 *     call (any small atb_gemm or this entry point) per device at start-up, BEFORE handing the rest of the
 *     device memory to a pool; after it, no call of this entry point changes the amount of free memory.
 *   - All calls share the one array and it keeps whatever the last call left there.  Nothing has to be
 *     cleared: every partial sum the reduction reads is written earlier by the same call.  For the same
 *     reason two calls whose kernels can run at the same time on one GPU (different streams, or
 *     different host threads) would trample each other's partial sums: order them on one stream or
 *     with events. */
#define ATB_NOALLOC_SCRATCH_BYTES (64u * 1024u * 1024u)
atb_status_t atb_gemm_splitk_noalloc(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                     const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                     const void* B_bf16_dev, int64_t ldb,
                                     void* C_bf16_dev, int64_t ldc, int splits, void* stream);

/* atb_gemm with a quantising epilogue: C is written in BFP16 (the C format of the all-BFP16
 * configurations of Section 6.1, Table 2), in the very layout atb_quantize_bfp16 produces for an
 * M x N matrix, so that C can be the A operand of the next atb_gemm (its blocks run along N, the K of
 * that product).  Every block of 8 consecutive columns of a row is quantised from the FP32
 * accumulators with the rule of atb_quantize_bfp16 (E = exponent of the block's largest magnitude,
 * m = RNE(x / 2^(E-133)) saturated to +-127): the result equals atb_quantize_bfp16 applied to the FP32
 * accumulators bit for bit.
 *   C_mant_dev: int8 [M][N] row-major (contiguous), 16-byte aligned (written);
 *   C_exp_dev:  exponent plane of atb_bfp16_exp_bytes(M, N) bytes, 16-byte aligned (written; the
 *               plane's padding rows get exponent 0).
 * Shapes: M >= 1, N % 16 == 0, K % 16 == 0.  Tilings: T_MA in {64, 128} with T_K = 64, T_MC in {128, 256} and
 * T_N in {128, 256}; with (T_MC, T_K, T_N) = (256, 64, 512), the CTA-pair tiling; and with (128, 128, 256), which
 * runs as two stacked tiles on a CTA pair where M > 128, as in atb_gemm.  Other arguments, conventions and errors
 * as for atb_gemm. */
atb_status_t atb_gemm_bfp16_out(int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                const int8_t* A_mant_dev, const uint8_t* A_exp_dev,
                                const void* B_bf16_dev, int64_t ldb,
                                int8_t* C_mant_dev, uint8_t* C_exp_dev, void* stream);

/* The precision configurations the paper evaluates (Section 6.1, Table 2), with the BFP16 operand on
 * the B side as the paper has it: the B tile stays in the core for the rho slabs of a K-step and is
 * converted ONCE per K-step; the slabs of A stream through it (Section 3.1).
 *   config 1: A in BF16 (streamed as is), B in BFP16, C in BF16;
 *   config 2: A, B and C in BFP16 (the paper's configurations 2 and 3; accumulation is FP32 here).
 * Operands (device memory, 16-byte aligned, caller-owned):
 *   A_dev:       config 1: bf16 A[M][lda] row-major (lda >= K, lda % 8 == 0), A_exp_dev = NULL;
 *                config 2: int8 mantissas [M][K] with their exponent plane in A_exp_dev (the planes
 *                of atb_quantize_bfp16; lda is ignored);
 *   Bt_mant_dev, Bt_exp_dev: the BFP16 planes of B TRANSPOSED, i.e. of the N x K matrix whose row n is
 *                column n of B, as atb_quantize_bfp16 produces them for that matrix - the blocks of 8
 *                run along K, as the paper's do;
 *   C_dev:       config 1: bf16 C[M][ldc] (ldc >= N, ldc % 8 == 0), C_exp_dev = NULL;
 *                config 2: int8 mantissas [M][N] and the exponent plane in C_exp_dev, as
 *                atb_gemm_bfp16_out writes them (ldc is ignored).
 * Shapes: M >= 1, N % 16 == 0, K % 16 == 0.  atb_gemm_config runs T_MA = 128, T_K = 64, T_N = 256 on a pair of SMs
 * (T_MC = 512, see atb_gemm_config_tiled) where M > 256 and on one SM (T_MC = 256) otherwise; the result does
 * not depend on that choice.  Errors as for atb_gemm; an unknown config is ATB_ERR_BAD_TILING. */
atb_status_t atb_gemm_config(int config, int64_t M, int64_t N, int64_t K,
                             const void* A_dev, const uint8_t* A_exp_dev, int64_t lda,
                             const int8_t* Bt_mant_dev, const uint8_t* Bt_exp_dev,
                             void* C_dev, uint8_t* C_exp_dev, int64_t ldc, void* stream);
/* The same with the asymmetric-buffering knob of Section 3 in the paper's own orientation (the experiment
 * of Section 6.1 / Table 1: the BFP16 tile of B stays put, A streams through it in slabs of T_MA rows):
 * T_MA in {32, 64, 128, 256} is the height of the slabs A is loaded and buffered in - one TMA box and, for a
 * BFP16 A, one raw buffer with its own barrier per slab.  T_K = 64 and T_N = 256 are fixed; T_MC is
 *   256: one SM holds the 256 x 256 accumulator and converts the whole B tile once per K-step;
 *   512: a pair of SMs (tcgen05 cta_group::2) holds 256 rows each and shares the B tile - each converts half of
 *        it, so a converted B element feeds 512 rows (the array-level sharing of Section 3.2, Eq. 2, applied to
 *        the resident operand) and the conversions per FLOP halve.
 * Per SM - the paper's "core" - the accumulator is 256 rows tall in both forms, so rho per core = 256 / T_MA
 * and T_MA = 256 is the symmetric form of both.  Any other (T_MC, T_K, T_N) is ATB_ERR_BAD_TILING.
 * For fixed operands the result is bit-identical for every T_MA and for both values of T_MC. */
atb_status_t atb_gemm_config_tiled(int config, int64_t M, int64_t N, int64_t K, int T_MA, int T_MC, int T_K, int T_N,
                                   const void* A_dev, const uint8_t* A_exp_dev, int64_t lda,
                                   const int8_t* Bt_mant_dev, const uint8_t* Bt_exp_dev,
                                   void* C_dev, uint8_t* C_exp_dev, int64_t ldc, void* stream);

/* 1 if atb_gemm accepts the tiling (kernel exists, TMEM and shared-memory budgets met), else 0.
 * Host only; touches no device. */
int atb_tiling_supported(int T_MA, int T_MC, int T_K, int T_N);

/* How atb_gemm lays a tiling out on the SM (host only; for documentation, tests and tuning).
 * The rings are the B200 counterpart of the buffers of Eq. 1: B tiles of T_K x T_N, raw BFP16 A
 * slabs of T_MA x T_K, and dequantised BF16 A in 128-row groups of T_K columns. */
typedef struct {
    int n_b_stages;      /* depth of the B-tile ring                                              */
    int n_raw_stages;    /* depth of the raw A-slab ring                                          */
    int n_a_groups;      /* depth of the dequantised-A ring, in 128-row groups                    */
    int dequant_groups;  /* groups the 16 dequantiser warps are split into; slabs take turns      */
    int acc_buffers;     /* T_MC x T_N FP32 accumulators resident in TMEM (1 or 2)                */
    int tmem_columns;    /* TMEM columns allocated (power of two <= 512)                          */
    int smem_bytes;      /* dynamic shared memory of the launch                                   */
} atb_plan_t;
/* Returns ATB_ERR_BAD_TILING if atb_gemm does not support the tiling. */
atb_status_t atb_tiling_plan(int T_MA, int T_MC, int T_K, int T_N, atb_plan_t* plan);

/* Waits for `stream` and reports whether any kernel of this library launched by this process on
 * the current device gave up a bounded wait since the last call (every wait on an mbarrier in the
 * kernels gives up after 2 s of the GPU's global timer, so that a fault cannot hang a shared GPU; the
 * CTA then sets an abort flag, all its roles leave their loops and it frees its tensor memory).
 * The flag is kept per device and read for the CURRENT device only: call with the device that ran
 * the kernels current.  Returns ATB_OK, ATB_ERR_DEVICE_TIMEOUT (and clears the flag) or ATB_ERR_CUDA.
 * Debug / test helper: it synchronises. */
atb_status_t atb_device_status(void* stream);

/* Parameters of the analytical model of Sections 3-5.  One "unit" is what the paper calls a core
 * (an AIE core there, an SM here). */
typedef struct {
    double peak_flops_per_cycle;  /* Perf_core^peak per unit, FLOP per cycle (Eq. 14-15)          */
    double clock_hz;              /* cycles per second                                            */
    int    n_units;               /* N_core of Eq. 12                                             */
    double bw_bytes_per_s;        /* BW_offchip of Eq. 12                                         */
    double a_bytes, b_bytes, c_bytes;              /* per-element byte costs in AI (Section 3.1)  */
    double a_buf_bytes, b_buf_bytes, c_buf_bytes;  /* per-element byte costs in Eq. 1             */
    double a_scratch_bytes;       /* bytes per A-slab element of one converted copy (0 = none)    */
    double buf_capacity_bytes;    /* S of Eq. 1 for the A and B terms (+ the C term if acc_capacity_bytes == 0) */
    double acc_capacity_bytes;    /* > 0: the C term c_buf*T_MC*T_N is budgeted here instead (TMEM) */
    int    share_rows, share_cols;/* array-level sharing factors of Eq. 2 (4 and 8 in the paper)  */
    double eta, eps_cycles, ii;   /* Eq. 13: Eff_micro = eta T_K / (eps + eta II T_K)             */
    double delta_cycles;          /* per-slab switching cost of Eq. 14                            */
    /* Refinements beyond the paper (0 switches each one off; all 0 in the XDNA2 presets): */
    int    mma_rows;              /* M extent of one MMA: a larger slab is consumed in pieces of this size, so Eq. 14-15
                                     count rho_eff = T_MC / min(T_MA, mma_rows) switches (0: rho_eff = rho)          */
    double load_latency_cycles;   /* atb_select_tiling: free-to-landed latency of a tile load; a B ring whose
                                     look-ahead is shorter scales the compute bound down                    */
    double pair_efficiency;       /* atb_select_tiling: measured factor on the compute bound of CTA-pair tilings */
    double launch_seconds;        /* atb_select_tiling: fixed cost per kernel launch              */
    double tile_fixed_cycles;     /* atb_select_tiling: pipeline fill per output tile that no other tile hides    */
    double drain_cycles_per_column; /* atb_select_tiling: where the accumulator is not double-buffered the UMMAs wait
                                     while the epilogue drains it: cycles per FP32 accumulator column of a unit  */
    double pair_tile_cycles;      /* atb_select_tiling: extra per-tile cost of a CTA pair (both units must finish) */
    double thin_slab_cost;        /* with mma_rows > 0: slabs thinner than mma_rows are converted and signalled in bundles
                                     of mma_rows rows, so a slab beyond the first of its bundle costs only this fraction of
                                     a switch: rho_eff = T_MC / mma_rows + (rho - T_MC / mma_rows) * thin_slab_cost
                                     (1 = every slab is a full switch, as in Eq. 14)                                 */
    double coarse_slab_factor;    /* with mma_rows > 0: factor on Eff_core of slabs larger than mma_rows: their raw ring has
                                     fewer, larger buffers and pipelines at coarser grain (0 or 1 = none)              */
    double deep_kstep_factor;     /* with mma_rows > 0: factor on Eff_core of tilings with T_K > 64 (0 or 1 = none; 0 in
                                     every preset: since A moves in 64-column units whatever T_K is, a deeper K-step
                                     no longer changes the conversion pipeline)                                        */
    /* The conversion of A (BFP16 -> BF16 in shared memory) that precedes every UMMA, on the compute side of
     * Eq. 12.  One unit = mma_rows rows x 64 columns of A; it feeds 2 * mma_rows * 64 * T_N FLOP, i.e.
     * t_mma = that / peak_flops_per_cycle cycles of tensor time.  Eff_core is multiplied by
     * t_mma / max(t_mma + convert_exposed_cycles, convert_cycles).  Both 0 = no conversion (XDNA2 presets). */
    double convert_cycles;        /* cycles per unit at the dequantisers' full throughput (binds where T_N is small)  */
    double convert_exposed_cycles;/* cycles per unit that the pipeline does not hide behind the UMMAs                  */
    double convert_latency_cycles;/* atb_select_tiling: latency from a free operand buffer to a converted unit; a ring of n
                                     converted units, each in use for t = max(t_mma + convert_exposed_cycles,
                                     convert_cycles) cycles, sustains n * t / (latency + t) of the rate                  */
    int    a_unit_cols;           /* > 0: A is buffered in units of this many columns whatever T_K is (64 on B200), so the A
                                     and scratch terms of Eq. 1 use min(T_K, a_unit_cols) in place of T_K (0: T_K)    */
} atb_hw_params_t;

typedef struct {
    atb_tiling_t t;
    int    feasible;              /* Eq. 1 / Eq. 3 satisfied                                      */
    double buf_bytes_used;        /* left-hand side of Eq. 1 (A, B and scratch terms; + C if not split) */
    double acc_bytes_used;        /* C term                                                       */
    double ai;                    /* Eq. 2, FLOP per byte                                         */
    double eff_micro, eff_core;   /* Eq. 13, Eq. 15                                               */
    double mem_bound_flops;       /* AI * BW                                                      */
    double compute_bound_flops;   /* Eff_core * peak * N_core                                     */
    double predicted_flops;       /* Eq. 12: the smaller of the two                               */
} atb_tiling_score_t;

/* Parameter presets: this library's B200 calibration, and the paper's XDNA2 evaluation
 * (Section 5 and Table 2; precision_config 1, 2 or 3 selects the byte costs of Section 6.1). */
void atb_hw_params_b200(atb_hw_params_t* hw);
void atb_hw_params_xdna2(atb_hw_params_t* hw, int precision_config);

/* Scores one tiling for problem depth K with the formulas of Sections 3 and 5 (Eq. 1, 2, 12-15).
 * Pure host arithmetic; returns ATB_ERR_NULL_POINTER / ATB_ERR_BAD_TILING (non-positive sizes or
 * T_MC not a multiple of T_MA). */
atb_status_t atb_score_tiling(const atb_hw_params_t* hw, int64_t K, atb_tiling_t t,
                              atb_tiling_score_t* out);

/* Tiling selection (Section 5: the trade-off between arithmetic intensity, which wants small T_K
 * and large rho, and core efficiency, which wants the opposite): enumerates the tilings atb_gemm
 * supports, scores each with atb_score_tiling for this (M, N, K) - including the loss from
 * partially filled waves of output tiles over n_units - and returns them best first.  A CTA-pair
 * tiling (T_MC = 256, T_N = 512) is rated per CTA: feasible, buf_bytes_used, acc_bytes_used, eff_core
 * and the compute bound are those of the 128-row half tile one CTA holds, with the B tile shared by two.
 * The stacked pair tiling (T_MC = 128, T_K = 128, T_N = 256, where M > 128) is rated as it is - a CTA holds a
 * whole 128 x 256 tile - with the B tile shared by two and the tiles counted in stripes of 256 rows.
 *   hw:       NULL = atb_hw_params_b200().
 *   best:     receives the top feasible tiling (may be NULL).
 *   scores:   optional array of *n_scores entries, filled best first; *n_scores receives the
 *             number written.  Pass scores = NULL, n_scores = NULL to get only `best`.
 * Returns ATB_ERR_BAD_SHAPE if no supported tiling is feasible. */
atb_status_t atb_select_tiling(int64_t M, int64_t N, int64_t K, const atb_hw_params_t* hw,
                               atb_tiling_t* best, atb_tiling_score_t* scores, int* n_scores);

#ifdef __cplusplus
}
#endif
#endif /* ATB_H_ */
