/*
 * mmasim -- bit-accurate evaluation of GPU matrix-multiply-accumulate arithmetic models on a B200.
 *
 * The library evaluates D = Phi(A, B, C) (the paper's Equation 2) where Phi is one of the arithmetic
 * behaviour models of Section 4 (Table 1: Phi_FTZ-AddMul, Phi_FMA, Phi_E/T/ST/GST/TR/GTR-FDPA), chosen by
 * (architecture, input type, accumulator type) exactly as Tables 3-7 map instructions to models.
 * Every output word is a pure function of the input words; there is exactly one correct answer.
 *
 * Conventions for every entry point
 *   - Data pointers are DEVICE pointers owned by the caller unless the name ends in _host.
 *   - The library never synchronises and enqueues work only on the given stream
 *     (a cudaStream_t passed as void*; NULL is the default stream).  _host calls are synchronous.
 *   - No CPU fallback exists: without a CUDA device the compute entry points return MMASIM_ERR_CUDA.
 *   - Return value: an mmasim_status; mmasim_last_error() gives a thread-local message for the last failure.
 *   - A is M x K row-major; B is N x K row-major, i.e. the paper's K x N matrix stored column-major
 *     (both operands are contiguous along K); C and D are M x N row-major in the accumulator type.
 *   - Element storage: FP64 8 bytes; FP32 and TF32 4 bytes (TF32: the low 13 bits are ignored);
 *     BF16/FP16 2 bytes; FP8, FP6 and FP4 of the T-/ST-FDPA models one element per byte in the low bits;
 *     FP4 of the GST-FDPA models (MXF4_GST, NVF4_GST) two per byte, element 2i in the low nibble.
 *   - K must be a multiple of min(K, L_max) (Algorithm 5 would silently drop a remainder; zero padding of A
 *     and B is exactly neutral for every FDPA model), of P for Phi_FTZ-AddMul, and of 32 for GST models.
 */
#ifndef MMASIM_H
#define MMASIM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mmasim_model mmasim_model; /* opaque, host side, immutable, may be shared between threads */

typedef enum {
    MMASIM_OK = 0,
    MMASIM_ERR_INVALID_ARG = 1, /* null pointer, bad enum, host pointer where a device pointer is needed */
    MMASIM_ERR_UNSUPPORTED = 2, /* the (arch, input, accumulator) triple is not in Tables 3-7 */
    MMASIM_ERR_SHAPE = 3,       /* M, N, K < 1, K not a multiple of the model's block, bad k_chunk or ld */
    MMASIM_ERR_ALIGN = 4,       /* pointer or leading dimension not aligned as documented */
    MMASIM_ERR_CUDA = 5,        /* a CUDA runtime call failed (message holds the CUDA error string) */
    MMASIM_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up (mmasim_hw_umma's status word, mmasim_gemm_host, mmasim_copy_timeouts) */
} mmasim_status;

/* The ten architectures of Section 3.2. */
typedef enum {
    MMASIM_VOLTA = 0, MMASIM_TURING, MMASIM_AMPERE, MMASIM_ADA, MMASIM_HOPPER, MMASIM_BLACKWELL,
    MMASIM_RTX_BLACKWELL, MMASIM_CDNA1, MMASIM_CDNA2, MMASIM_CDNA3, MMASIM_ARCH_COUNT
} mmasim_arch;

/* Input types (first column of Tables 3-7).  MX* are the block-scaled variants of Algorithm 8 (one E8M0
 * scale per 32 elements); MXF4_GST / NVF4_GST are the group-scaled FP4 variants of Algorithm 9 (E8M0 per 32
 * elements / UE4M3 per 16 elements).  BF16_1K is the CDNA2 "_1k" BF16 instruction class (P = 4). */
typedef enum {
    MMASIM_F64 = 0, MMASIM_F32, MMASIM_TF32, MMASIM_BF16, MMASIM_BF16_1K, MMASIM_F16,
    MMASIM_E4M3, MMASIM_E5M2, MMASIM_E3M2, MMASIM_E2M3, MMASIM_E2M1,
    MMASIM_MXE4M3, MMASIM_MXE5M2, MMASIM_MXE3M2, MMASIM_MXE2M3, MMASIM_MXE2M1,
    MMASIM_MXF4_GST, MMASIM_NVF4_GST, MMASIM_FMT_COUNT
} mmasim_fmt;

typedef enum { MMASIM_ACC_F32 = 0, MMASIM_ACC_F16, MMASIM_ACC_F64, MMASIM_ACC_COUNT } mmasim_acc;

/* Model families (Table 1) and conversion functions (Table 2). */
typedef enum {
    MMASIM_FAM_FMA = 0, MMASIM_FAM_FTZ_ADDMUL, MMASIM_FAM_E_FDPA, MMASIM_FAM_T_FDPA, MMASIM_FAM_ST_FDPA,
    MMASIM_FAM_GST_FDPA, MMASIM_FAM_TR_FDPA, MMASIM_FAM_GTR_FDPA
} mmasim_family;
typedef enum { MMASIM_RHO_NONE = 0, MMASIM_RZ_FP32, MMASIM_RZ_E8M13, MMASIM_RNE_FP32, MMASIM_RNE_FP16 } mmasim_rho;

/* Parameters of a model as the paper's tables give them (0 where a parameter does not apply). */
typedef struct {
    int32_t family;       /* mmasim_family */
    int32_t l_max;        /* L_max of Algorithm 5 (Tables 4, 5, 6, 7) */
    int32_t F;            /* fractional bits of the fused sum */
    int32_t F2;           /* TR-/GTR-FDPA second-stage precision (Table 7) */
    int32_t rho;          /* mmasim_rho */
    int32_t P;            /* Phi_FTZ-AddMul group size (Table 6) */
    int32_t G;            /* GST-FDPA group size (Table 5) */
    int32_t k_block;      /* elements per scale factor: 32 (MX), 16 (NVFP4), 0 = unscaled */
    int32_t a_bits;       /* storage bits per A element: 64, 32, 16, 8 or 4 */
    int32_t b_bits;       /* storage bits per B element */
    int32_t acc_bytes;    /* bytes per C / D element: 8, 4 or 2 */
    int32_t inner_round;  /* 0 = as in the paper; 1 = TR-FDPA second stage uses RZ (Section 6.2.4 experiment) */
} mmasim_info;

/* Hypothetical-model overrides for mmasim_create_model_ex (design-space exploration, Section 7).
 * A negative field keeps the table value. */
typedef struct {
    int32_t l_max, F, F2, rho, inner_round;
    int32_t literal_emax;       /* 1: the maximum exponent of the fused sum runs over every term as Algorithms 7-11 print
                                   it (a zero product counts with Exp(a) + Exp(b), a zero accumulator with its exponent
                                   field's value, every GST group with its scale exponents) instead of over the nonzero
                                   terms, which is what the B200 does; FDPA models other than E-FDPA; generic kernels */
} mmasim_overrides;

/* Optional arguments of mmasim_gemm_ex.  Zero-initialise, then set what is needed. */
typedef struct {
    int64_t lda, ldb, ldc, ldd; /* leading dimensions in ELEMENTS (GST FP4: in elements, even); 0 = packed */
    const void* sfa;            /* device, M x ceil(K/k_block) bytes row-major: scale factors of A (ST/GST models) */
    const void* sfb;            /* device, N x ceil(K/k_block) bytes row-major: scale factors of B */
    int64_t k_chunk;            /* 0, or a multiple of the model's block: every k_chunk elements of K the model is
                                   run from a +0 accumulator and its FP32 result is added to an FP32 running sum
                                   with an IEEE-754 RNE addition (the FP32-promotion workaround the paper motivates
                                   in Sections 2.2 and 6.3; FP32-accumulator FDPA models only) */
    const float* row_scale;     /* device, M floats or NULL */
    const float* col_scale;     /* device, N floats or NULL: D = fl32(fl32(row_scale[i]*col_scale[j]) * d) */
    int32_t flags;              /* MMASIM_GEMM_FORCE_GENERIC: skip the tuned kernels (used to cross-check them) */
} mmasim_gemm_opts;
#define MMASIM_GEMM_FORCE_GENERIC 1

/* Registry lookup (Tables 3-7).  Returns NULL and sets the error message if the triple is not in the paper. */
mmasim_model* mmasim_create_model(int arch, int in_fmt, int acc_fmt);

/* As above with different A and B element types (Algorithm 7 allows F_A != F_B; both must select the same
 * table row class, e.g. E4M3 x E5M2) and optional overrides; ov may be NULL. */
mmasim_model* mmasim_create_model_ex(int arch, int a_fmt, int b_fmt, int acc_fmt, const mmasim_overrides* ov);

void mmasim_destroy_model(mmasim_model* model);

/* Fills *out with the model's parameters. */
int mmasim_model_info(const mmasim_model* model, mmasim_info* out);

/* D = Phi(A, B, C) (Equation 2; Algorithms 2, 4, 5).  C may be NULL (= +0) and may alias D.
 * All pointers 16-byte aligned.  Enqueues on stream and returns. */
int mmasim_gemm(const mmasim_model* model, int64_t M, int64_t N, int64_t K,
                const void* A, const void* B, const void* C, void* D, void* stream);

/* As mmasim_gemm with leading dimensions, scale factors (Algorithms 8, 9), FP32 promotion of partial sums
 * and a dequantisation epilogue.  opts may be NULL. */
int mmasim_gemm_ex(const mmasim_model* model, int64_t M, int64_t N, int64_t K,
                   const void* A, const void* B, const void* C, void* D,
                   const mmasim_gemm_opts* opts, void* stream);

/* mmasim_gemm_ex without any device-memory allocation, for callers that cannot allocate when they call: code inside a
 * region where the allocator must not be touched (a latency-critical loop, a thread that may not take the allocator's
 * locks, a process whose memory budget is fixed at start-up), where mmasim_gemm_ex would take stream-ordered scratch
 * out of the library's pool.  The paper has no counterpart; this is a property of the library, not of a model.
 *   - Serves the FP8 models with F = 13 (the Ada and Hopper FP8 rows of Table 4, A and B in E4M3 or E5M2), K a multiple
 *     of 32, row strides of A and B multiples of 16 bytes; anything else returns MMASIM_ERR_UNSUPPORTED.  Inputs,
 *     outputs and opts (k_chunk, row_scale / col_scale, leading dimensions) as for mmasim_gemm_ex; results are the same
 *     words.
 *   - The scratch (the decoded operands: about (ceil(M/128) + ceil(N/128)) * K/32 * 27 KiB, with 64-column tiles of B
 *     for FP16 accumulators and k_chunk) lives in a fixed 32 MiB device array that every GPU loading the library holds
 *     until the process ends.  A problem that needs more returns MMASIM_ERR_SHAPE and the message states both sizes
 *     (1024 x 1024 x 1024 needs 14 MiB; 2048 x 2048 x 512 fits, 2048^3 does not).
 *   - The first call on each device looks the array's address up (with that device current); make that first call
 *     outside any stream capture.  No call allocates or frees device memory.
 *   - All calls share the one array, which keeps the previous call's contents; every call rewrites the part it reads,
 *     so nothing has to be cleared.  Two calls whose work overlaps on the GPU (different streams, or one stream of each
 *     of two host threads) race on it: order them on one stream or with events. */
int mmasim_gemm_noalloc(const mmasim_model* model, int64_t M, int64_t N, int64_t K,
                        const void* A, const void* B, const void* C, void* D,
                        const mmasim_gemm_opts* opts, void* stream);

/* n independent dot-product-accumulates d_t = Phi(a_t, b_t, c_t) (Equation 4), the shape of the paper's probe
 * vectors (Section 3.1): A, B are n x K row-major, C (may be NULL) and D hold n accumulator words.
 * Unscaled models only. */
int mmasim_dot_batch(const mmasim_model* model, int64_t n, int64_t K,
                     const void* A, const void* B, const void* C, void* D, void* stream);

/* mmasim_gemm_ex on HOST buffers: allocates device memory, copies A, B, C (and scales) to the device, runs,
 * copies D back and frees; synchronous.  Fields of opts that are pointers are host pointers here.
 * The device buffers are stream-ordered allocations on a stream of the call's own, out of a memory pool that the
 * library creates per device on first use and that keeps up to 1 GiB between calls, so repeated calls do not pay
 * for allocation; mmasim_host_release() destroys the pools and returns the memory.  The device's default memory
 * pool and its attributes are not touched.  Pinned host buffers make the copies asynchronous.
 * Problems of 1024 rows and 32 MiB or more are cut into up to eight row panels of D (outputs are independent,
 * Section 3.1 Step 1): B is copied once, then each panel's rows of A and C go in, its kernel runs and its rows of D
 * come back on separate streams, so that with pinned buffers the copies run beside the arithmetic.
 * With opts->ldd > N only the N words of every row of D are written; the words between rows stay the caller's.
 * Returns MMASIM_ERR_TIMEOUT if a kernel of the call gave up a bounded wait (see mmasim_copy_timeouts): D is then incomplete. */
int mmasim_gemm_host(const mmasim_model* model, int64_t M, int64_t N, int64_t K,
                     const void* A, const void* B, const void* C, void* D, const mmasim_gemm_opts* opts);

/* Destroys the memory pools mmasim_gemm_host created (every device); no mmasim_gemm_host call may be in flight.
 * The next mmasim_gemm_host call creates a new pool.  No counterpart in the paper. */
int mmasim_host_release(void);

/* The hardware's own matrix multiply-accumulate, for differential runs of the models against the machine they
 * describe (Section 3.1, Step 4; Section 3.2: an MMA interface is D = MMA(A, B, C) on one instruction).  Runs the
 * warp-level `mma.sync` instruction of the given kind on every tile of 16 rows of A (8 for MMASIM_HW_F64):
 *   D (M x 8) = A (M x K, row-major) * B^T (B is 8 x K, row-major, shared by all tiles) + C (M x 8, may be NULL = +0),
 * K a multiple of the instruction's K; a longer K chains instructions through the accumulator in ascending k, as
 * Algorithm 5 does.  Element layouts as for mmasim_gemm (TF32 in 32-bit words, FP8 one element per byte); all
 * pointers are device pointers; M a multiple of the tile height.  Results are whatever the B200 computes:
 * comparing them with a model is the caller's business. */
typedef enum {
    MMASIM_HW_F16_F32 = 0,      /* m16n8k16, FP16 inputs, FP32 accumulator */
    MMASIM_HW_F16_F16 = 1,      /* m16n8k16, FP16 inputs, FP16 accumulator */
    MMASIM_HW_BF16_F32 = 2,     /* m16n8k16 */
    MMASIM_HW_TF32_F32 = 3,     /* m16n8k8 */
    MMASIM_HW_E4M3_F32 = 4,     /* m16n8k32 */
    MMASIM_HW_E5M2_F32 = 5,     /* m16n8k32 */
    MMASIM_HW_F64 = 6,          /* m8n8k4, FP64 throughout */
    MMASIM_HW_F16_F32_K8 = 7,   /* m16n8k8 */
    MMASIM_HW_TF32_F32_K4 = 8,  /* m16n8k4 */
    MMASIM_HW_E4M3_F16 = 9,     /* m16n8k32, FP8 inputs, FP16 accumulator */
    MMASIM_HW_E5M2_F16 = 10,    /* m16n8k32 */
    MMASIM_HW_E4M3_E5M2_F32 = 11, /* m16n8k32, A in E4M3, B in E5M2 */
    MMASIM_HW_E4M3_F32_K16 = 12  /* m16n8k16 */
} mmasim_hw_kind;
int mmasim_hw_mma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D, void* stream);

/* The same for the B200's fifth-generation matrix instruction, tcgen05.mma (the instruction class of the paper's Blackwell
 * FP8 / FP6 / FP4 rows, Table 3's UTC*MMA entries; Section 3.2, Section 3.1 Step 4).  One instruction tile of 128 rows:
 *   D (M x 16) = A (M x K, row-major) * B^T (B is 16 x K, row-major, shared by all tiles) + C (M x 16, may be NULL = +0),
 * accumulator words (FP32; 16-bit FP16 words for the kinds 17-20), M a multiple of 128, K a multiple of the instruction's K (16 for FP16 / BF16, 8 for TF32, 32
 * for the 8-bit kinds); a longer K chains instructions through the accumulator in tensor memory, ascending k.  Element
 * layouts as for mmasim_gemm (TF32 in 32-bit words; FP8, FP6 and FP4 one element per byte in the low bits); all
 * pointers are device pointers.  `status` (device, 4 bytes, zeroed by the caller) receives MMASIM_ERR_TIMEOUT if the
 * kernel's bounded wait for the instruction ran out; the kernel then stores nothing, releases what it holds and
 * returns.  MMASIM_UMMA_SELFTEST_TIMEOUT issues nothing, so that this wait runs out after about a millisecond: the
 * test of the give-up path (A, B, D are still needed as valid buffers). */
typedef enum {
    MMASIM_UMMA_F16_F32 = 0, MMASIM_UMMA_BF16_F32 = 1, MMASIM_UMMA_TF32_F32 = 2, MMASIM_UMMA_E4M3_F32 = 3,
    MMASIM_UMMA_E5M2_F32 = 4, MMASIM_UMMA_E4M3_E5M2_F32 = 5, MMASIM_UMMA_E2M3_F32 = 6, MMASIM_UMMA_E3M2_F32 = 7,
    MMASIM_UMMA_E2M1_F32 = 8, MMASIM_UMMA_SELFTEST_TIMEOUT = 9,
    /* block-scaled kinds: sfa (M x K/k_block bytes) and sfb (16 x K/k_block bytes), device, row-major, as for mmasim_gemm_ex */
    MMASIM_UMMA_MXE4M3 = 10, MMASIM_UMMA_MXE5M2 = 11, MMASIM_UMMA_MXE2M3 = 12, MMASIM_UMMA_MXE3M2 = 13, MMASIM_UMMA_MXE2M1 = 14,
    MMASIM_UMMA_MXF4 = 15,      /* packed FP4, E8M0 scale per 32 elements, K a multiple of 64 */
    MMASIM_UMMA_NVF4 = 16,      /* packed FP4, UE4M3 scale per 16 elements, K a multiple of 64 */
    /* FP16 accumulator (C and D are M x 16 16-bit words): kind::f16 with FP16 inputs, kind::f8f6f4 with E4M3 / E5M2 /
     * E2M1 inputs - the Blackwell FP16-accumulator rows of Tables 3 and 4 (T-FDPA with rho = RNE-FP16) */
    MMASIM_UMMA_F16_F16 = 17, MMASIM_UMMA_E4M3_F16 = 18, MMASIM_UMMA_E5M2_F16 = 19, MMASIM_UMMA_E2M1_F16 = 20
} mmasim_umma_kind;
int mmasim_hw_umma(int kind, int64_t M, int64_t K, const void* A, const void* B, const void* C, void* D,
                   const void* sfa, const void* sfb, int32_t* status, void* stream);

/* Error statistics of n model outputs D (accumulator words, acc_fmt MMASIM_ACC_F32 or MMASIM_ACC_F16) against an
 * FP64 reference `ref` (n doubles): the reduction behind the accuracy analysis of Section 6 - the deviation
 * delta = D - D_real of Figure 3 (Section 6.2.4), its sign balance and its size.  `stats` (device, 8 doubles) is
 * ACCUMULATED into (the caller zeroes it; several calls may share it):
 *   [0] outputs counted (pairs where D or ref is NaN or infinite are skipped)   [1] sum of delta
 *   [2] sum of |delta|   [3] sum of delta^2   [4] number of delta < 0   [5] number of delta > 0
 *   [6] max |delta|      [7] sum of |delta| / |ref| over ref != 0
 * All pointers are device pointers. */
int mmasim_error_stats(int acc_fmt, int64_t n, const void* D, const double* ref, double* stats, void* stream);

/* Issue-rate micro-benchmarks, the roofline denominators (no counterpart in the paper).  Launches `blocks` CTAs of
 * 256 threads; every thread runs `iters` (rounded up to a multiple of 8) times 8 rounds of independent operations of
 * the given kind.  `sink` (device, >= 4 bytes) receives a value that keeps the work alive.  The caller times the
 * launch; counted operations per launch = blocks * 256 * iters * 8 * (*ops_per_round).  Kinds:
 *    0 iadd3          3-input integer add              1 lop3           3-input logic
 *    2 shf            funnel shift                     3 imad           32-bit integer multiply-add
 *    4 macmix         add / max / sub / shift / add of one emulated term (5 operations per round)
 *    5 viaddmax       fused add-max, 32-bit            6 viaddmax16x2   fused add-max on two 16-bit lanes
 *    7 f2i            float -> int conversion          8 fmul           FP32 multiply
 *    9 popc           population count + add          10 imad+alu       one multiply-add and one add per round
 *   11 fmul+alu       FP32 multiply and integer add   12 imad.wide      32 x 32 -> 64-bit multiply
 *   13 mac_d1, 14 mac_d2   two integer forms of one emulated term
 *   15 dp4a           4-way byte dot product          16 dfma           FP64 multiply-add, 8 dependent chains
 *   17 dfma+alu       FP64 multiply-add and add-max   18 ffma.rm        FP32 multiply-add toward -inf, 8 chains
 *   19 ffma2.rm       packed two-lane fma.rm.f32x2, 8 chains
 *   20 ffma.rn.x16, 21 ffma.rn.x32, 22 ffma.rm.x16, 23 ffma2.rm.x16 (lanes counted), 24 dfma.rn.x16, 25 dfma.rn.x32,
 *   26 dfma.rm.x16    the same instructions with 16 / 32 independent accumulators per thread and loop-invariant
 *                     multiplicands (no operand-fetch conflicts): the second witness of the pipe rates.
 *   27 dmma.rm.k4, 28 dmma.rm.k16   the FP64 matrix instruction rounding toward -inf (mma.sync m8n8k4 / m16n8k16),
 *                     multiply-adds counted.
 *   29 cvt.f32.f64 (FP32 -> FP64 -> FP32), 30 cvt.s32.f64 (s32 -> FP64 -> s32): conversion pairs, both counted;
 *   31 dadd.rm.x16    add.rm.f64 with 16 independent accumulators.
 *   32 ffma2.rm.x16+alu   kind 23 with one independent integer addition beside every packed multiply-add (the
 *                     multiply-add lanes are counted): whether the FP32 and the integer pipe issue side by side. */
int mmasim_int_peak(int kind, int64_t blocks, int64_t iters, void* sink, int32_t* ops_per_round, void* stream);

/* Name of the kernel variant the last mmasim_gemm* call on this thread dispatched to ("generic", ...). */
const char* mmasim_last_kernel(void);

/* The tuned fused-summation kernels bring decoded operand blocks into shared memory with bulk copies and wait for each
 * with a bounded number of polls.  A CTA whose wait runs out (never in a healthy run) stores none of its outputs and
 * counts itself in a per-device counter; this call synchronises the current device and returns the counter's value
 * since the library was loaded in *count (host pointer).  0 means that every output of every finished call was
 * stored.  No counterpart in the paper. */
int mmasim_copy_timeouts(uint64_t* count);

/* Thread-local message of the last failing call on this thread ("" if none). */
const char* mmasim_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MMASIM_H */
