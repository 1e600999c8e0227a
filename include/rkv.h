/*
 * rkv.h -- C ABI of librkv: bulk verification of candidate-kernel outputs on
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the numerical-correctness step of the robust-kbench
 * evaluation loop (arxiv 2509.14279): the outputs of K candidate kernels are
 * compared with one reference output, for seeded test inputs drawn from several
 * value distributions, and outputs that exploit a loophole are flagged.
 *
 *   - App. "Kernel Evaluation Environment": a kernel is correct iff it passes
 *     all tests (input sizes x initialisation settings x seeds); absolute and
 *     relative tolerance 1e-5.  -> rkv_verify_batch / rkv_verify_multi, the
 *     per-element rule |c - r| <= atol + rtol*|r| and the joint verdict.
 *   - Sec. 5 "Kernel Translation & Optimization": the candidate's result is
 *     compared with the torch reference.  -> one reference, K candidates.
 *   - Sec. 3 (harness): "diverse initialization states to prevent hardcoding";
 *     forward and backward passes (a backward candidate returns several
 *     gradient tensors).  -> rkv_gen_inputs, rkv_verify_multi.
 *   - Sec. 3, App. A.1 and the listing "Level 2 - Task 13": constant outputs,
 *     pass-through of the input, low-magnitude outputs.  -> the flags.
 *
 * Conventions.  Every function returns an rkv_status (0 = RKV_OK, < 0 = error)
 * unless stated otherwise; none throws, aborts or prints.  Unless a parameter is
 * marked HOST, a data pointer is caller-owned DEVICE memory of the current CUDA
 * device, 16-byte aligned; the library reads inputs and writes outputs
 * stream-ordered on the given stream and never synchronises it, except where a
 * function says so.  bf16 tensors are raw 16-bit patterns.  Tensors are flat,
 * contiguous, row-major; a shape is only a product.
 *
 * Stream capture.  Every verification call sends a small descriptor table from
 * host memory that does not outlive the call, so none of them can be recorded
 * into a CUDA graph: a call on a stream that is being captured enqueues nothing
 * and returns RKV_ERR_UNSUPPORTED.  (rkv_gen_inputs* and rkv_screen_outputs pass
 * everything by value.)
 */
#ifndef RKV_H
#define RKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum rkv_status {
    RKV_OK = 0,
    RKV_ERR_INVALID_ARG = -1,  /* null pointer, K < 1, n < 1, bad enum, negative / non-finite tolerance */
    RKV_ERR_UNSUPPORTED = -2,  /* legal request outside this build's limits (see each function) */
    RKV_ERR_ALIGNMENT = -3,    /* a device pointer is not 16-byte aligned */
    RKV_ERR_WORKSPACE = -4,    /* workspace missing or smaller than rkv_workspace_bytes() */
    RKV_ERR_CUDA = -5,         /* a CUDA runtime call failed (no device, launch error, ...) */
    RKV_ERR_TIMEOUT = -6,      /* device side: a bounded wait on a bulk copy ran out */
    RKV_ERR_BOUNDS = -7        /* device side, debug build only: a range check failed (the access was skipped) */
} rkv_status;

/* Element storage types.  fp16 (IEEE binary16) and bf16 tensors are raw 16-bit patterns;
 * both are widened to fp32 exactly before anything is computed.  The generator produces
 * fp32 and bf16 only: a reference or input that is regenerated on the fly cannot be fp16. */
enum { RKV_F32 = 0, RKV_BF16 = 1, RKV_F16 = 2 };

/* Value distributions of the input generator. */
enum {
    RKV_DIST_NORMAL = 0,      /* N(0,1), Box-Muller                                   */
    RKV_DIST_UNIFORM_PM1 = 1, /* uniform on [-1, 1), multiples of 2^-23               */
    RKV_DIST_STUDENT_T2 = 2,  /* Student-t with 2 degrees of freedom (heavy-tailed)   */
    RKV_DIST_SPARSE90 = 3,    /* exact +0 with probability 0.9, else N(0,1)           */
    RKV_DIST_NORMAL_1E4 = 4   /* N(0,1) * 1e4 (large magnitude)                       */
};

/* Where a reference / input tensor comes from. */
enum {
    RKV_SRC_NONE = 0,      /* input only: no input tensor, copy-of-input flags stay clear */
    RKV_SRC_POINTER = 1,   /* read from device memory                                     */
    RKV_SRC_GENERATED = 2  /* regenerated on the fly from an rkv_gen_spec (fused path)    */
};

/* rkv_stats.verdict bits; a candidate passes iff verdict == 0. */
enum {
    RKV_FAIL_TOL = 1u << 0,            /* n_over_tol > 0                                        */
    RKV_FAIL_NAN = 1u << 1,            /* the candidate holds a NaN                             */
    RKV_FAIL_INF_MISMATCH = 1u << 2,   /* an infinity on one side not matched on the other      */
    RKV_FAIL_LOOPHOLE_CONST = 1u << 3, /* candidate constant, reference not, n > 1              */
    RKV_FAIL_LOOPHOLE_COPY = 1u << 4   /* candidate is a bit copy of the input, reference is not */
};

/* rkv_stats.flags bits. */
enum {
    RKV_FLAG_CAND_CONST = 1u << 0,         /* every candidate element bit-equal to element 0 */
    RKV_FLAG_CAND_COPY_OF_INPUT = 1u << 1, /* every candidate element bit-equal to input[i]  */
    RKV_FLAG_REF_CONST = 1u << 2,
    RKV_FLAG_REF_COPY_OF_INPUT = 1u << 3,
    RKV_FLAG_HAS_NAN = 1u << 4,
    RKV_FLAG_HAS_INF = 1u << 5
};

#define RKV_NO_INDEX UINT64_MAX

/*
 * Result for one candidate and one tensor (88 bytes, little-endian, 8-aligned).
 * With c the candidate and r the reference, both as fp32 (bf16 is upcast
 * exactly), an element is COMPARABLE when c and r are finite.  For comparable
 * elements e = |c - r| (one fp32 subtraction) and the element is over tolerance
 * when !(e <= atol + rtol*|r|), the product and the sum each rounded to fp32.
 * Equal infinities match and are not comparable; any other non-finite
 * involvement counts as over tolerance.  Indices are flat element offsets, the
 * first (smallest) index attaining the maximum; RKV_NO_INDEX when no element
 * qualifies.  max_rel_err ranges over comparable elements with r != 0.
 */
typedef struct rkv_stats {
    uint32_t verdict;
    uint32_t flags;
    uint64_t n_over_tol;
    uint64_t n_nan;           /* NaN elements of the candidate            */
    uint64_t n_inf;           /* infinite elements of the candidate       */
    uint64_t n_inf_mismatch;  /* non-comparable, not matching, an infinity on either side */
    uint64_t n_comparable;
    uint64_t argmax_abs_err;
    uint64_t argmax_rel_err;
    double sum_abs_err;       /* sum of e over comparable elements: fp32 within a tile of 14 KiB of
                                 the candidate, fp64 above; within 1e-6 of a sequential fp64 sum,
                                 and the same bits on every run (it is added in tile order)      */
    float max_abs_err;        /* 0 when nothing is comparable             */
    float max_rel_err;
    float mean_abs_err;       /* (float)(sum_abs_err / n_comparable), 0 if none */
    uint32_t reserved;
} rkv_stats;

/* A Philox stream: which (seed, stream_id, distribution) tensor to generate.
 * Element i is produced by word (i & 3) of Philox4x32-10 block (i >> 2) with
 * key = seed and counter = (block index, stream_id).  RKV_DIST_SPARSE90 also
 * consumes the stream stream_id + 1 (its zero mask). */
typedef struct rkv_gen_spec {
    uint64_t seed;
    uint64_t stream_id;
    int32_t dist;
    int32_t reserved;
} rkv_gen_spec;

/* One tensor of a verification case. */
typedef struct rkv_tensor_desc {
    uint64_t n;                /* elements; 1 <= n < 2^40                                      */
    const void *ref;           /* DEVICE, n elements of ref_dtype; used when ref_src == POINTER */
    const void *input;         /* DEVICE, n elements of cand_dtype; used when input_src == POINTER */
    const void *const *cands;  /* HOST array of K DEVICE pointers, n elements of cand_dtype each */
    rkv_gen_spec ref_gen;      /* used when ref_src == GENERATED   */
    rkv_gen_spec input_gen;    /* used when input_src == GENERATED */
    int32_t cand_dtype;        /* RKV_F32 | RKV_BF16 | RKV_F16 */
    int32_t ref_dtype;         /* RKV_F32 | RKV_BF16 | RKV_F16; a generated reference is rounded to it
                                  (RKV_F32 or RKV_BF16 then) */
    int32_t ref_src;           /* RKV_SRC_POINTER | RKV_SRC_GENERATED */
    int32_t input_src;         /* RKV_SRC_NONE | RKV_SRC_POINTER | RKV_SRC_GENERATED; the input
                                  has the candidates' dtype (a copy is a bit copy) */
    float atol;                /* finite, >= 0 */
    float rtol;                /* finite, >= 0 */
} rkv_tensor_desc;

/* Library version: major * 10000 + minor * 100 + patch. */
int rkv_version(void);

/* Static, NUL-terminated description of a status code. */
const char *rkv_status_string(int status);

/* Stream used by the two calls that take none (rkv_gen_inputs,
 * rkv_verify_batch).  cuda_stream is a cudaStream_t; NULL = default stream.
 * Process-wide; not synchronised against concurrent callers. */
int rkv_set_stream(void *cuda_stream);

/*
 * Input generator (Sec. 3: diverse initialisation states; App. "Kernel
 * Evaluation Environment": multiple random seeds).  Fills out with the tensor
 * (seed, stream 0, dist).
 *   shape  HOST array of ndim extents (>= 1 each); only the product is used
 *   dtype  RKV_F32 | RKV_BF16 (fp32 value rounded to nearest-even)
 *   out    DEVICE, product(shape) elements, 16-byte aligned
 * Runs on the stream set by rkv_set_stream.  Errors: INVALID_ARG, ALIGNMENT, CUDA.
 */
int rkv_gen_inputs(uint64_t seed, int dist, const int64_t *shape, int ndim, int dtype, void *out);

/*
 * Same generator with every knob: elements first_elem .. first_elem + n - 1 of
 * the tensor (seed, stream_id, dist) are written to out[0 .. n).  first_elem
 * must be a multiple of 4 (one Philox block serves four elements).
 */
int rkv_gen_inputs_ex(uint64_t seed, uint64_t stream_id, int dist, uint64_t n,
                      uint64_t first_elem, int dtype, void *out, void *cuda_stream);

/*
 * Verify K candidates against one reference (App. "Kernel Evaluation
 * Environment"; Sec. 5).  Both sides have dtype `dtype`; no input tensor, so the
 * copy-of-input flags stay clear.
 *   ref        DEVICE, n elements
 *   cands      HOST array of K DEVICE pointers, n elements each
 *   stats_out  DEVICE, K rkv_stats, written stream-ordered
 * Runs on the stream set by rkv_set_stream.  Uses a library-owned scratch
 * buffer that grows on demand (cudaMalloc on first use / growth: not safe
 * during stream capture; concurrent calls on different streams would share it,
 * so serialise them).  Errors: INVALID_ARG, UNSUPPORTED (also: the stream is
 * being captured), ALIGNMENT, CUDA.
 */
int rkv_verify_batch(const void *ref, const void *const *cands, int K, uint64_t n, int dtype,
                     float atol, float rtol, rkv_stats *stats_out);

/*
 * General form: T tensors per candidate, verified in one launch; candidate k
 * passes jointly iff it passes on every tensor (the paper's "passes all tests";
 * a backward candidate returns three gradients).
 *   tensors     HOST array of T descriptors (1 <= T <= 64); tensors[t].cands HOST array of K
 *   stats_out   DEVICE, K*T rkv_stats, entry [k*T + t]
 *   joint_pass  DEVICE, K uint32 (1 = pass on all T tensors), may be NULL
 *   workspace   DEVICE scratch, >= rkv_workspace_bytes(tensors, T, K) bytes, 256-byte
 *               aligned; contents are undefined afterwards; must not be shared by
 *               calls that overlap on the GPU
 * Nothing is allocated on the device.  The descriptors and pointer tables are
 * copied to the workspace with one cudaMemcpyAsync from pageable host memory and
 * the rest of the workspace is cleared with one cudaMemsetAsync.
 * Errors: INVALID_ARG, UNSUPPORTED (also: cuda_stream is being captured),
 * ALIGNMENT, WORKSPACE, CUDA.  A device-side timeout is reported by
 * rkv_device_status.
 */
int rkv_verify_multi(const rkv_tensor_desc *tensors, int T, int K, rkv_stats *stats_out,
                     uint32_t *joint_pass, void *workspace, size_t workspace_bytes,
                     void *cuda_stream);

/* Scratch bytes rkv_verify_multi needs for this case on the current device
 * (0 on an invalid argument).  Depends on n, the dtypes, T, K and the device's
 * SM count only: tables, 64 bytes per (tensor, candidate), 48 bytes * K per tensor and
 * resident thread block (per tile, for a tensor of fewer tiles than blocks), and one
 * double per (tile of 14 KiB of a candidate, candidate) for the error sums. */
size_t rkv_workspace_bytes(const rkv_tensor_desc *tensors, int T, int K);

/*
 * Config sweep (listing "Linear config": the single_ and multi_ lists of input, init and
 * shared settings; App. "Kernel Evaluation Environment": a kernel is correct iff it
 * passes for ALL input sizes x initialisation settings x seeds).  C test cases, each with
 * its own tensors (shapes, storage types, tolerances, stored or regenerated reference),
 * the same K candidate kernels in every case; one launch over the items of all cases.
 *   cases        HOST array of C case descriptors; cases[c].tensors is a HOST array of
 *                cases[c].T rkv_tensor_desc (each with its HOST array of K DEVICE pointers)
 *   C            1 <= C; the tensors of all cases together: at most 4096
 *   stats_out    DEVICE, K * (sum of T) rkv_stats: case c starts at K * (T of the cases
 *                before it); inside the case entry [k * T_c + t]
 *   case_pass    DEVICE, C*K uint32, entry [c*K + k] = candidate k passed on every tensor
 *                of case c; may be NULL
 *   all_pass     DEVICE, K uint32 = AND over the cases (the paper's verdict); may be NULL
 *   workspace    DEVICE, >= rkv_sweep_workspace_bytes(cases, C, K), 256-byte aligned
 * Errors as rkv_verify_multi; a device-side timeout is reported by rkv_device_status.
 */
typedef struct rkv_case_desc {
    const rkv_tensor_desc *tensors;   /* HOST */
    int32_t T;                        /* 1 <= T <= 64 */
    int32_t reserved;
} rkv_case_desc;

int rkv_verify_sweep(const rkv_case_desc *cases, int C, int K, rkv_stats *stats_out, uint32_t *case_pass,
                     uint32_t *all_pass, void *workspace, size_t workspace_bytes, void *cuda_stream);

size_t rkv_sweep_workspace_bytes(const rkv_case_desc *cases, int C, int K);

/* Synchronises cuda_stream and returns the device-side status word the last
 * rkv_verify_multi / rkv_verify_sweep on this workspace left (RKV_OK, RKV_ERR_TIMEOUT,
 * or RKV_ERR_BOUNDS from a debug build), or RKV_ERR_CUDA. */
int rkv_device_status(const void *workspace, void *cuda_stream);

/*
 * End-to-end form with HOST buffers (plumbing around rkv_verify_batch, no passage of its
 * own): copies the reference and the candidates to
 * the device in chunks (overlapped with verification on two streams), verifies,
 * copies the K results back and synchronises.  Pinned host buffers make the
 * copies asynchronous.  Allocates (and caches) device staging memory.
 *   ref_host     HOST, n elements of dtype
 *   cands_host   HOST array of K HOST pointers
 *   stats_host   HOST, K rkv_stats
 */
int rkv_verify_batch_host(const void *ref_host, const void *const *cands_host, int K, uint64_t n,
                          int dtype, float atol, float rtol, rkv_stats *stats_host);

/*
 * The general case with HOST buffers (plumbing around rkv_verify_multi, no passage of
 * its own): the descriptors of rkv_verify_multi, except that tensors[t].cands is a HOST
 * array of K HOST pointers and tensors[t].ref / tensors[t].input are HOST pointers
 * (when their source is RKV_SRC_POINTER; a generated reference or input is regenerated
 * on the device and nothing of it is copied).  References and inputs are copied once,
 * the candidates in chunks of a few candidates of every tensor, two chunks in flight,
 * each chunk verified while the next one travels; the results come back and the
 * stream set by rkv_set_stream is synchronised.  Host pointers need no alignment;
 * pinned buffers make the copies asynchronous.  Allocates (and caches) device staging
 * memory: not for callers that cannot allocate.
 *   stats_host  HOST, K*T rkv_stats, entry [k*T + t]
 *   joint_host  HOST, K uint32 (1 = pass on all T tensors), may be NULL
 * Errors: INVALID_ARG, UNSUPPORTED (T > 64, n >= 2^40, capturing stream), CUDA.
 */
int rkv_verify_multi_host(const rkv_tensor_desc *tensors, int T, int K, rkv_stats *stats_host,
                          uint32_t *joint_host);

/*
 * rkv_verify_batch with no allocation of any kind.  (The paper has no
 * counterpart: this form exists for the way the library gets embedded.)
 *
 * Who needs it: a caller that may not allocate device memory at the point of the
 * call -- a harness that has handed all of the GPU's memory to its own pool and
 * left the driver nothing to give out, a host thread that must not block on the
 * allocator's device-wide synchronisation, a process running under a memory
 * budget that counts every allocation it makes.  rkv_verify_batch grows a
 * library-owned buffer with cudaMalloc; rkv_verify_multi wants a workspace the
 * caller had to allocate at some point.  This form needs neither: its scratch
 * (per-block partial results, per-candidate state and the descriptor tables) is an 8 MiB array that is
 * part of the library's device image.  Every GPU that loads the library holds
 * those 8 MiB until the process exits, whether or not this function is called.
 *
 * Same arguments, same results and same comparison rule as rkv_verify_batch,
 * plus the stream to run on (a cudaStream_t; NULL = default stream).  ref, cands
 * and stats_out are the caller's; inputs are only read.
 *
 * Limits: K <= 256, and the scratch the case needs (rkv_workspace_bytes of the
 * single-tensor case: about 48 bytes * K * 2 * SM count plus 8 bytes * K per 14 KiB
 * of a candidate) must fit in 8 MiB; on a 148-SM part that is e.g. K = 64 candidates
 * of 2^24 fp32 elements, or K = 256 of 2^21.  A larger case is rejected with
 * RKV_ERR_UNSUPPORTED before anything is launched.  Other errors: INVALID_ARG,
 * ALIGNMENT, CUDA.
 *
 * First call on a device: looks up the array's device address once (with that
 * device current) and sets a kernel attribute.  Make that first call outside any
 * stream capture.  (Like every verification call it returns RKV_ERR_UNSUPPORTED
 * on a stream that is being captured: its table is sent from the host stack.)
 *
 * All calls on a device share the one array, and it keeps whatever the previous
 * call left there.  The library rewrites the status word and the tables and
 * clears the per-candidate state and the partial results at the start of every
 * call (stream-ordered), so a call never depends on old contents.  Two calls whose work overlaps
 * on the GPU (different streams, or several host threads) race on the array and
 * give undefined results: run them one after the other.
 *
 * Calls no cudaMalloc / cudaFree and no allocating library routine; the small
 * descriptor table is built on the host stack and sent with one cudaMemcpyAsync.
 */
int rkv_verify_batch_static(const void *ref, const void *const *cands, int K, uint64_t n, int dtype,
                            float atol, float rtol, rkv_stats *stats_out, void *cuda_stream);

/*
 * Host-only planning helper (no CUDA call; plumbing, no passage of its own): how the
 * work of one tensor is cut.
 * The tensor is cut into *n_tiles tiles of *tile_elems elements (a thread of the
 * verification kernel owns 64 bytes of each candidate tile: 3584 fp32 or 7168 16-bit
 * elements per tile).  One work item is
 * one tile against a part of the K candidates: a thread block keeps the tile's
 * reference values in registers and streams that tile of each candidate of the
 * part past them.  A tensor has up to three groups of items: the first *warm_tiles
 * tiles (the square root of the tile count, rounded down, at most 18), with the
 * candidates cut into *parts_warm parts (many small ones, so that every resident
 * block -- 2 per SM -- starts with one of these items), are verified first; the
 * running maxima and loophole flags they publish let the tiles after them, with
 * *parts_main parts of at most 64 candidates (more while these tiles are fewer than
 * the blocks), skip nearly all rare-path work; the last *tail_tiles tiles of a long
 * tensor, with *parts_tail parts of at most 16 candidates, come last and even out the
 * finishing times of the blocks.  A tensor whose tiles all fit the first wave of
 * blocks has one group: *warm_tiles == *n_tiles, *parts_main == 0, *tail_tiles == 0
 * and *parts_tail == 0 (in a call of several tensors, the tiles of all of them
 * count).  Part p of P covers candidates [p*K/P, (p+1)*K/P).
 *   cand_dtype  RKV_F32 | RKV_BF16 | RKV_F16 (storage type of the candidates)
 *   num_sms     SM count of the device
 * Errors: INVALID_ARG (n < 1, K < 1, num_sms < 1, bad dtype, null), UNSUPPORTED (n >= 2^40).
 */
int rkv_plan_items(uint64_t n, int cand_dtype, int K, int num_sms, uint32_t *tile_elems, uint32_t *n_tiles,
                   uint32_t *warm_tiles, uint32_t *parts_warm, uint32_t *parts_main, uint32_t *tail_tiles,
                   uint32_t *parts_tail);

/* Releases the library-owned scratch and staging buffers of all devices. */
int rkv_release_cached(void);

/* ------------------------------------------------------------------------------------
 * Task-soundness screens (App. A.1, the filtering criteria): is a task fit to be a
 * benchmark at all?  The paper excludes a task whose reference outputs (1) all lie
 * between -0.01 and 0.01, (2) have a standard deviation below 0.01 across model and input
 * seeds, (3) are uniform along their axes, or (4) vary by less than 0.01 across input
 * seeds.  One streaming pass over the reference outputs of S seeds computes the
 * statistics behind the four criteria; the limits are arguments (0.01 in the paper).
 * The readings taken, the paper giving the criteria in words only:
 *   (1) every finite value v of every seed has -range_lim <= v <= range_lim;
 *   (2) the population standard deviation of all finite values, pooled over the seeds,
 *       is below std_lim;
 *   (3) seen as rows x cols (row-major), every column (axis 0) or every row (axis 1) of
 *       every seed repeats its first element bit for bit;
 *   (4) the largest per-element spread max_s x_s[i] - min_s x_s[i] (one fp32 subtraction;
 *       elements that are not finite in some seed are left out) is below spread_lim.
 * ------------------------------------------------------------------------------------ */
enum rkv_screen_flag {
    RKV_SCREEN_NARROW_RANGE = 1u << 0,
    RKV_SCREEN_LOW_STD = 1u << 1,
    RKV_SCREEN_LOW_SEED_VARIATION = 1u << 2,
    RKV_SCREEN_UNIFORM_AXIS0 = 1u << 3,
    RKV_SCREEN_UNIFORM_AXIS1 = 1u << 4,
    RKV_SCREEN_NONFINITE = 1u << 5      /* informative: some value is NaN or infinite */
};

typedef struct rkv_screen_stats {
    uint32_t flags;               /* rkv_screen_flag bits; bits 0..4 each exclude the task */
    uint32_t reserved;
    uint64_t n_values;            /* S * rows * cols */
    uint64_t n_nonfinite;
    uint64_t argmax_seed_spread;  /* first element with the largest spread; RKV_NO_INDEX if none */
    double mean;                  /* of the finite values */
    double std;                   /* population standard deviation of the finite values */
    float vmin, vmax;             /* of the finite values (the sign of a zero is unspecified);
                                     +inf / -inf when there is none */
    float max_seed_spread;        /* -1 when S < 2 or no element is finite in every seed */
    uint32_t reserved2;
} rkv_screen_stats;               /* 64 bytes */

/* Bytes of device workspace rkv_screen_outputs needs on the current device (0 without one). */
size_t rkv_screen_workspace_bytes(void);

/*
 * Screens the reference outputs of one task.
 *   outs         HOST array of S DEVICE pointers, each to rows*cols elements of dtype,
 *                contiguous, row-major, 16-byte aligned; caller-owned, only read
 *   S            number of seeds, 1 <= S <= 16 (with S == 1 criterion (4) is not evaluated)
 *   rows, cols   the two-dimensional view the uniformity criterion is taken on (a tensor of
 *                more dimensions is passed as leading dimension x the rest, or any other
 *                split the caller cares about); rows*cols < 2^40
 *   dtype        RKV_F32 | RKV_BF16
 *   range_lim, std_lim, spread_lim   the limits of criteria (1), (2), (4), each >= 0
 *   stats_out    DEVICE pointer to one rkv_screen_stats, written by the call's last kernel
 *   workspace    DEVICE memory of at least rkv_screen_workspace_bytes(), 16-byte aligned;
 *                contents need not be preserved or cleared between calls
 *   cuda_stream  the stream (cudaStream_t) the two kernels are launched on; the call does
 *                not synchronise
 * mean and std are accumulated in fp64 in a fixed order (bit-reproducible on one device
 * model); everything else is exact.
 * Errors: INVALID_ARG (null, S < 1, rows or cols < 1, bad dtype, a negative or NaN limit),
 * UNSUPPORTED (S > 16, rows*cols >= 2^40), ALIGNMENT, WORKSPACE (null or too small), CUDA.
 */
int rkv_screen_outputs(const void *const *outs, int S, uint64_t rows, uint64_t cols, int dtype,
                       float range_lim, double std_lim, float spread_lim, rkv_screen_stats *stats_out,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ------------------------------------------------------------------------------------
 * Two loophole checks that need no reference (Sec. 3, the loophole list: "insufficient
 * output variation across different seeds", "hardcoding for specific input patterns";
 * App. A.1, criterion 4 read on a candidate's outputs instead of the task's).
 *
 * Cross-seed variation.  A candidate kernel is run on S input seeds; a kernel that
 * ignores its input (a hard-coded result) produces the same output every time.  With
 * x_s[i] the candidate's output for seed s, widened to fp32, the readings taken (the paper
 * gives no formula):
 *   IDENTICAL    every x_s has the storage bits of x_0;
 *   WITHIN_TOL   every x_s is within atol + rtol*|x_0| of x_0, element by element, by the
 *                comparison rule of rkv_stats with x_0 as the reference (NaN never close,
 *                equal infinities close);
 *   LOW_SPREAD   the largest per-element spread max_s x_s[i] - min_s x_s[i] (one fp32
 *                subtraction; elements not finite in some seed are left out) is below
 *                spread_lim (0.01 in the paper's filtering criteria);
 *   NONFINITE    informative: some element is NaN or infinite in some seed.
 * With S == 1 none of the first three is set and max_spread is -1.
 * ------------------------------------------------------------------------------------ */
enum rkv_cross_flag {
    RKV_CROSS_IDENTICAL = 1u << 0,
    RKV_CROSS_WITHIN_TOL = 1u << 1,
    RKV_CROSS_LOW_SPREAD = 1u << 2,
    RKV_CROSS_NONFINITE = 1u << 3
};

typedef struct rkv_cross_stats {
    uint32_t flags;             /* rkv_cross_flag bits */
    uint32_t reserved;
    uint64_t n_nonfinite;       /* elements with a non-finite value in some seed */
    uint64_t argmax_spread;     /* first element with the largest spread; RKV_NO_INDEX if none */
    float max_spread;           /* -1 when S < 2 or no element is finite in every seed */
    uint32_t reserved2;
} rkv_cross_stats;              /* 32 bytes */

/* Bytes of device workspace rkv_cross_seed needs on the current device (0 on a bad argument
 * or without a device). */
size_t rkv_cross_workspace_bytes(int K, int S);

/*
 * Cross-seed variation of K candidates in one launch; every output byte is read once.
 *   outs         HOST array of K*S DEVICE pointers, outs[k*S + s] = candidate k's output for
 *                input seed s: n elements of dtype, contiguous, 16-byte aligned, only read
 *   K, S         1 <= K <= 4096, 1 <= S <= 16
 *   dtype        RKV_F32 | RKV_BF16 | RKV_F16
 *   stats_out    DEVICE, K rkv_cross_stats
 *   workspace    DEVICE, >= rkv_cross_workspace_bytes(K, S), 16-byte aligned
 * Errors: INVALID_ARG, UNSUPPORTED (limits above, n >= 2^40, capturing stream), ALIGNMENT,
 * WORKSPACE, CUDA.
 */
int rkv_cross_seed(const void *const *outs, int K, int S, uint64_t n, int dtype, float atol, float rtol,
                   float spread_lim, rkv_cross_stats *stats_out, void *workspace, size_t workspace_bytes,
                   void *cuda_stream);

size_t rkv_copy_workspace_bytes(int K, int M);

/*
 * Copy of any input: a kernel receives several operands (activations, weights, the incoming
 * gradient); an output that is a bit copy of one of them passes a value check whenever
 * the reference happens to equal that operand, and is a pass-through either way.
 *   inputs         HOST array of M DEVICE pointers (1 <= M <= 8), n elements of dtype each
 *   cands          HOST array of K DEVICE pointers (1 <= K <= 4096), n elements of dtype each
 *   copy_mask_out  DEVICE, K uint32: bit m set iff candidate k has the storage bytes of
 *                  inputs[m] throughout (+0 and -0 differ)
 * A candidate is compared with an operand until a difference has been seen; only true
 * copies are read to the end.  Errors as rkv_cross_seed.
 */
int rkv_copy_of_inputs(const void *const *inputs, int M, const void *const *cands, int K, uint64_t n, int dtype,
                       uint32_t *copy_mask_out, void *workspace, size_t workspace_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RKV_H */
