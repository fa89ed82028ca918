/*
 * collage.h -- C ABI of the B200 (sm_100a) Collage bf16 multi-component-float AdamW library.
 *
 * The library implements the optimizer step of "Collage: Light-Weight Low-Precision Strategy
 * for LLM Training" (Algorithm 2) for the paper's precision options A (plain bfloat16),
 * B (Collage-light: theta held as a bfloat16 pair) and C (Collage-plus: theta and the second
 * moment held as pairs, beta2 as a pair), the error-free transforms it is built from
 * (Theorem 4.1, Algorithm 1, Appendix C), and the effective-descent-quality metric (Eq. 2-3).
 *
 * Arithmetic model (Section 3.1): every operator written in the paper takes bfloat16 operands
 * and rounds its exact result once, to nearest-even, to bfloat16.  Scalars are evaluated in
 * double on the host and cast to bfloat16 last (Section 4.2, Appendix D).
 *
 * Conventions for every entry point unless it says otherwise:
 *   - tensor pointers are DEVICE pointers to bfloat16 bit patterns (uint16_t), owned by the
 *     caller, on the current CUDA device; hyper-parameter structs, tensor lists and scalar
 *     outputs named "host" are HOST pointers;
 *   - state tensors are updated in place; `grad` is read only;
 *   - calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream); the library never synchronises the device and never allocates on the step path;
 *     collage_adamw_step, collage_adamw_step_multi and collage_adamw_step_fp32 only launch kernels,
 *     so once a call of the same kind has run on the device (it sets per-device kernel attributes
 *     the first time) they may be recorded by stream capture into a CUDA graph: the scalars of
 *     the step are kernel arguments and are recorded with it;
 *   - errors are detected on the host BEFORE anything is launched and reported as a status
 *     code; nothing is thrown across the boundary; there is no CPU fallback: a device that is
 *     not compute capability 10.x yields COLLAGE_ERR_ARCH;
 *   - pointers need not be 16-byte aligned and lengths need not be multiples of 8 (such
 *     tensors take a slower element-wise path with identical results);
 *   - n == 0 is a successful no-op;
 *   - NaN/Inf in tensor data is not an error: it propagates per IEEE 754;
 *   - threads: any entry point may be called from several host threads at once, on the same or on
 *     different devices and streams (the library's own first-call set-up is guarded), provided that
 *     calls in flight together share no tensor, no workspace, no plan being modified
 *     (collage_plan_set_replicas, collage_plan_destroy) and, for collage_adamw_step_host and
 *     collage_edq_static, no device: those two keep one context or scratch array per device;
 *   - the EDQ workspace (hyper->workspace) must hold zeros before its first use: clear it once with
 *     collage_workspace_init or cudaMemset.  Every call leaves it ready for the next one.
 */
#ifndef COLLAGE_H_
#define COLLAGE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    COLLAGE_OK = 0,
    COLLAGE_ERR_NULL = 1,       /* a required pointer is NULL                                   */
    COLLAGE_ERR_ARG = 2,        /* step == 0, unknown strategy/op/flag combination, hyper out of range */
    COLLAGE_ERR_ALIAS = 3,      /* two tensors of one call overlap, or one overlaps the workspace / EDQ record */
    COLLAGE_ERR_ARCH = 4,       /* current device is not sm_100                                 */
    COLLAGE_ERR_CUDA = 5,       /* a CUDA runtime call or launch failed                         */
    COLLAGE_ERR_WORKSPACE = 6,  /* workspace missing or smaller than collage_workspace_bytes()  */
    COLLAGE_ERR_LIMIT = 7       /* size beyond the fixed capacity of an entry point             */
} collage_status_t;

/* Precision options of Table 2. */
typedef enum {
    COLLAGE_BF16 = 0,   /* A: theta, m, v single bfloat16                    ( 8 B/param with grad) */
    COLLAGE_LIGHT = 1,  /* B: (theta, dtheta) pair                           (10 B/param)           */
    COLLAGE_PLUS = 2,   /* C: (theta, dtheta), (v, dv) pairs, beta2 as pair  (12 B/param)           */
    /* Comparator of the paper's experiments, not one of its options: BF16 AdamW with Kahan summation
     * at the parameter update (Appendix B): update' = update (+) c; theta' = theta (+) update';
     * c' = update' (-) (theta' (-) theta).  Same arrays as option B, x_lo holding c (10 B/param).
     * EDQ counts theta alone (Eq. 2 as printed). */
    COLLAGE_KAHAN = 3,
    /* A measuring stick outside the paper (its Algorithm 2 is strict bfloat16): option C's arrays and
     * traffic, but each step widens theta+dtheta and v+dv to float, runs AdamW in IEEE single
     * operations with float scalars, and splits the results back into normalised bfloat16 pairs
     * (hi = RN(x), lo = RN(x - hi)).  Quantifies what the strict arithmetic costs in accuracy. */
    COLLAGE_PLUS_FP32_REGISTERS = 4
} collage_strategy_t;

/* Algorithm 2 line 12 prints epsilon under the root; AdamW has it outside.  Default: outside. */
#define COLLAGE_FLAG_EPS_INSIDE_SQRT 1u
/* Variants of the parameter update (default: off).
 * TWOSUM_GROW: line 13's Grow uses TwoSum instead of Fast2Sum (Appendix C: same expansion with no
 *   ordering requirement), so the update is error-free also where |theta| < |update|.  B and C only.
 * DECAY_BY_GROW: the weight decay is not summed into the update (Appendix D: "either ... or") but
 *   applied first by an addition (Grow for B and C) of its own: d = (-a) (*) (lam (*) theta), then the
 *   Adam part (-a) (*) r.  A, B, C.  EDQ then measures against d + update. */
#define COLLAGE_FLAG_TWOSUM_GROW 2u
#define COLLAGE_FLAG_DECAY_BY_GROW 4u
/* Which kernel runs the step.  By default the size decides: a flat tensor of up to 2^21 parameters takes
 * a kernel without staging, one 8-parameter vector per thread straight from global memory (shortest
 * latency); above that, and for every multi-tensor plan, the bulk-copy pipeline streams at HBM bandwidth
 * in three stages of 4096-element tiles (6144 for COLLAGE_BF16); a COLLAGE_PLUS step over 2^27 parameters or
 * more uses two stages of 8192-element tiles (1-2 % faster there; in a plan only if chunk_elems is a
 * multiple of 8192, as the default is).  All of them compute the same bits.  These flags pin the choice
 * (tests and measurements): PIPELINE_KERNEL = the three-stage pipeline whatever the size, DIRECT_KERNEL =
 * the kernel without staging (flat entry points only), LARGE_TILES = the two-stage pipeline (COLLAGE_PLUS
 * without variant flags only).  More than one of them is ERR_ARG; where a flag does not apply it is ignored. */
#define COLLAGE_FLAG_PIPELINE_KERNEL 8u
#define COLLAGE_FLAG_DIRECT_KERNEL 16u
#define COLLAGE_FLAG_LARGE_TILES 32u

/* Hyper-parameters of one step (Algorithm 2 line 1).  HOST struct.
 * Valid ranges: lr, eps, weight_decay >= 0 and finite; 0 <= beta1, beta2 < 1. */
typedef struct collage_hyper {
    double lr, beta1, beta2, eps, weight_decay;
    uint32_t flags;          /* COLLAGE_FLAG_*                                                   */
    void* edq_out;           /* DEVICE collage_edq_t*, or NULL to skip the EDQ reduction          */
    void* workspace;         /* DEVICE scratch, >= collage_workspace_bytes(); needed iff edq_out  */
    size_t workspace_bytes;
} collage_hyper_t;

/* Result of the EDQ reduction (Eq. 3), written on the device by the call's last kernel.
 *   dot   = sum_i delta_i * eff_i        eff = (theta'+dtheta') - (theta+dtheta)   (Eq. 2)
 *   sumsq = sum_i delta_i^2              delta = the bfloat16 update of Algorithm 2 line 12
 *   edq   = dot / sqrt(sumsq), 0 if sumsq == 0
 *   lost  = #{i : delta_i != 0 and eff_i == 0}: parameters that an update was meant for and that did not
 *           move (Def. 3.2; "not updated", Figure 3 left).  For a pair the value theta + dtheta counts:
 *           a Grow that re-splits the same value over other components has not updated it.
 *   fault = 0, or the code of a bounded device-side wait that gave up during this call (see
 *           collage_pipeline_fault): the step was torn and the state arrays are then undefined.
 * Products and 8-element partial sums are formed in float, everything above in double, in a
 * fixed order: the result is reproducible for a given launch geometry. */
typedef struct collage_edq {
    double dot, sumsq, edq;
    uint64_t n;
    uint64_t lost;
    uint64_t fault;
} collage_edq_t;

/* One parameter tensor of a multi-tensor plan.  x_lo may be NULL for a plan used only with
 * COLLAGE_BF16; v_lo may be NULL unless the plan is used with COLLAGE_PLUS. */
typedef struct collage_tensor {
    void* x_hi;        /* theta          */
    void* x_lo;        /* delta-theta    */
    void* m;           /* first moment   */
    void* v_hi;        /* second moment  */
    void* v_lo;        /* delta-v        */
    const void* grad;
    uint64_t n;        /* elements       */
} collage_tensor_t;

typedef struct collage_plan collage_plan_t;   /* opaque; owns a small device table */

const char* collage_status_string(collage_status_t status);

/* Scalar preparation (Algorithm 2 line 1; Table 1; Appendix D "Scalar and Bias Correction").
 * HOST only, no CUDA call.  out_bf16[11] receives, as bfloat16 bit patterns,
 *   [0] RN(beta1) [1] RN(1-beta1) [2] RN(beta2) [3] RN(1-beta2)
 *   [4] beta2_hi = RN(beta2) [5] beta2_lo = RN(beta2 - beta2_hi)
 *   [6] RN(1-beta1^step) [7] RN(1-beta2^step) [8] RN(lr) [9] RN(weight_decay) [10] RN(eps)
 * every expression evaluated in double before the one rounding.
 * Errors: NULL -> ERR_NULL; step == 0 or hyper out of range -> ERR_ARG. */
collage_status_t collage_derive_scalars(const collage_hyper_t* hyper, uint64_t step, uint16_t out_bf16[11]);

/* Bytes of device scratch the EDQ reduction needs (independent of n; about 128 KiB). */
size_t collage_workspace_bytes(uint64_t n_total);

/* Clears an EDQ workspace (asynchronous memset on `stream`).  The step kernels end their EDQ
 * reduction (Eq. 3) inside the same launch: each thread block stores its partial sums in the
 * workspace and draws a ticket from a counter that lives there; the block that draws the last
 * ticket adds the partials in index order and writes the record.  The counter wraps back to zero
 * with the last ticket, so one clearing before the first use is enough.  A workspace serves one
 * call at a time: calls that may run concurrently need separate workspaces.
 * Errors: ERR_NULL, ERR_WORKSPACE (smaller than collage_workspace_bytes() or not 16-byte aligned),
 * ERR_CUDA. */
collage_status_t collage_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/* Combines EDQ records of disjoint parameter sets (tensors, slices, ranks) into the record of their
 * union, Eq. 3 on the summed partial sums: dot, sumsq, n and lost are added in array order, edq =
 * dot / sqrt(sumsq) (0 if sumsq == 0), fault = the first non-zero fault.  HOST arrays, no CUDA call.
 * `out` may be one of the parts.  Errors: ERR_NULL, ERR_ARG (count < 0). */
collage_status_t collage_edq_combine(const collage_edq_t* parts_host, int count, collage_edq_t* out_host);

/* "product" for the ordinary build; a measurement build of the same sources that compiles the
 * arithmetic out of the step kernel (to time the copy pipeline alone) answers "data-movement-only". */
const char* collage_build_flavor(void);

/* One AdamW step over one flat tensor (Algorithm 2 lines 8-13, all n parameters, step t >= 1).
 *   x_hi, m, v_hi, grad : required.   x_lo : required iff strategy != COLLAGE_BF16 (delta-theta, or
 *   the Kahan compensation for COLLAGE_KAHAN), else must
 *   be NULL.   v_lo : required iff strategy is COLLAGE_PLUS or COLLAGE_PLUS_FP32_REGISTERS, else
 *   must be NULL.
 * With hyper->edq_out set the record is written by the same launch (one kernel per step).
 * Errors: ERR_NULL, ERR_ARG (step 0, bad strategy, hyper range), ERR_ALIAS (overlapping
 * tensors; workspace or record overlapping a tensor or each other), ERR_WORKSPACE (edq_out set,
 * workspace missing, misaligned or too small), ERR_ARCH, ERR_CUDA. */
collage_status_t collage_adamw_step(void* x_hi, void* x_lo, void* m, void* v_hi, void* v_lo,
                                    const void* grad, uint64_t n, const collage_hyper_t* hyper,
                                    uint64_t step, collage_strategy_t strategy, void* stream);

/* Comparator of the paper's experiments: option D of Table 2 -- bfloat16 parameter and gradient,
 * float (fp32) optimizer states and float master weights, 16 B/param -- and, with master == NULL,
 * D^-MW of Section 5.1 (float optimizer states, no master weights, 12 B/param).  Standard
 * mixed-precision AdamW in the operation order of Algorithm 2; every operation is one IEEE
 * single-precision operation, scalars are evaluated in double and cast to float once.
 *   theta : DEVICE bfloat16[n], written (D: theta = RN_bf16(master); D^-MW: read and written)
 *   master: DEVICE float[n] or NULL;  m, v: DEVICE float[n];  grad: DEVICE bfloat16[n], read only
 * EDQ (hyper->edq_out / workspace as for collage_adamw_step) measures the float update against the
 * change of the stored parameter: the master weight for D, the bfloat16 parameter for D^-MW.
 * HBM traffic 28 B/param (D) or 22 B/param (D^-MW) against 22 B/param of Collage-plus.
 * Of the arithmetic flags only COLLAGE_FLAG_EPS_INSIDE_SQRT is accepted in hyper->flags.
 * Errors: ERR_NULL, ERR_ARG (step 0, hyper range, flags, float arrays not 4-byte aligned),
 * ERR_ALIAS, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA. */
collage_status_t collage_adamw_step_fp32(void* theta, void* master, void* m, void* v, const void* grad,
                                         uint64_t n, const collage_hyper_t* hyper, uint64_t step, void* stream);

/* The same step for state that lives in HOST memory (optimizer state kept off the device).
 * All six tensor pointers are HOST pointers (page-locked memory is needed for the copies to
 * overlap; pageable memory works, serialised by the runtime).  The arrays are streamed through
 * `staging_dev`, a DEVICE buffer of `staging_bytes` bytes (256-byte aligned, at least
 * collage_workspace_bytes() + 1 MiB; larger is faster up to a few hundred MiB), in slabs: while
 * slab i is computed, slab i+1 is copied in and slab i-1 copied out on two internal copy streams
 * that the library creates per device on the first call.  Work is ordered after earlier work on
 * `stream`, and `stream` waits for the last copy-out, so synchronising `stream` suffices.
 * hyper->edq_out, if set, is a HOST collage_edq_t* here (written by a copy enqueued on
 * `stream`); hyper->workspace is ignored.  Results are bit-identical to collage_adamw_step.
 * Calls on one device share the copy streams: issue them one at a time per device.
 * Errors: as collage_adamw_step, with ERR_WORKSPACE for a missing, misaligned or too small
 * staging buffer. */
collage_status_t collage_adamw_step_host(void* x_hi, void* x_lo, void* m, void* v_hi, void* v_lo,
                                         const void* grad, uint64_t n, const collage_hyper_t* hyper,
                                         uint64_t step, collage_strategy_t strategy, void* staging_dev,
                                         size_t staging_bytes, void* stream);

/* Multi-tensor step: all tensors of a plan in ONE launch over a chunk table.
 * collage_plan_create copies the HOST array `tensors[num]` and builds the device table
 * (this call allocates and synchronises; do it once, outside the step loop).  chunk_elems is
 * the work unit handed to a thread block, a multiple of 2048; 0 picks the default (24576;
 * multiples of 24576 keep every tile whole for every precision option and tile size).
 * Tensors with n == 0 are skipped.  The plan records which pointers were NULL; a step whose
 * strategy needs a missing component fails with ERR_NULL.  EDQ is over all tensors (Eq. 3
 * with theta the concatenation).
 * A plan belongs to the device that was current at creation; stepping it with another device
 * current is ERR_ARG.
 * Errors: ERR_NULL, ERR_ARG (num < 0, chunk_elems not a multiple of 2048, more than 2^32-1
 * chunks), ERR_ALIAS (any two arrays of the plan overlap), ERR_CUDA. */
collage_status_t collage_plan_create(const collage_tensor_t* tensors, int num, uint32_t chunk_elems,
                                     collage_plan_t** out_plan);
collage_status_t collage_adamw_step_multi(const collage_plan_t* plan, const collage_hyper_t* hyper,
                                          uint64_t step, collage_strategy_t strategy, void* stream);
collage_status_t collage_plan_destroy(collage_plan_t* plan);

/* Replicas of the parameter (sharded optimizer state: each GPU steps its own slice of the
 * parameters, every GPU needs all of theta for the next forward pass).  After this call every
 * step of the plan also writes the updated first component theta of tensor i to each replica,
 * tile by tile from inside the step kernel (the same bulk stores that write theta home), so the
 * gather costs no extra kernel and overlaps the step.  The paper describes no collective; this is
 * the one exchange its optimizer step would need (2 B/param per replica).
 *   replicas : HOST array of num_replicas * num DEVICE pointers, replica r of tensors[i] at
 *              replicas[r * num + i], `num` as given to collage_plan_create; each points to
 *              tensors[i].n bfloat16 values in this GPU's memory or in a peer GPU's memory mapped
 *              into this process (peer access enabled), and must have the same address modulo 16
 *              as tensors[i].x_hi.  Entries of empty tensors are ignored.  num_replicas <= 15;
 *              0 removes the replicas.
 * The call synchronises the device and allocates a small table: do it once, outside the step loop.
 * A replica holds the new theta once the step's kernel has finished; readers on other GPUs need
 * their own ordering with that (an event, a barrier).  Plain stores issued by each block for itself.
 * Errors: ERR_NULL, ERR_ARG (count, alignment, wrong device), ERR_ALIAS (a replica overlaps an
 * array of the plan or another replica), ERR_CUDA. */
collage_status_t collage_plan_set_replicas(collage_plan_t* plan, const void* const* replicas, int num_replicas);

/* Lets kernels of the CURRENT device store into memory of `peer_device` (a device ordinal of this
 * process), so that pointers into a peer's memory that the caller has mapped (CUDA IPC, virtual
 * memory management) can serve as replicas.  Host-side set-up, not on the step path; succeeds if the
 * access is already enabled.  The paper has no counterpart (its experiments do not shard the step).
 * Errors: ERR_ARG (same device, or the devices cannot reach each other), ERR_CUDA. */
collage_status_t collage_enable_peer_access(int peer_device);

/* The multi-tensor step with EDQ kept per tensor (Eq. 2-3 evaluated on each parameter tensor of the
 * plan separately; the lost-update count of Def. 3.2 per tensor gives the imprecision percentage of
 * Figure 3, left).  Same state update as collage_adamw_step_multi, bit for bit.
 *   per_tensor_out_dev : DEVICE collage_edq_t[num], num = the `num` given to collage_plan_create;
 *                        entry i belongs to tensors[i] (all zero for an empty tensor).
 *   chunk_workspace    : DEVICE scratch of at least collage_plan_workspace_bytes(plan) bytes, 16-byte
 *                        aligned (32 bytes per chunk of the plan).
 *   hyper->edq_out     : optional DEVICE collage_edq_t for the whole plan = the per-tensor sums added
 *                        in tensor order (association differs from collage_adamw_step_multi's, so
 *                        the last bits may differ); hyper->workspace is not used by this call.
 * Three launches (step, per-tensor sums, total) instead of one.  The variant flags (TWOSUM_GROW,
 * DECAY_BY_GROW) are not available through this entry point (ERR_ARG).
 * Errors: as collage_adamw_step_multi, plus ERR_ARG when num differs from the plan's and
 * ERR_WORKSPACE for the chunk workspace. */
size_t collage_plan_workspace_bytes(const collage_plan_t* plan);
collage_status_t collage_adamw_step_multi_per_tensor(const collage_plan_t* plan, const collage_hyper_t* hyper,
                                                     uint64_t step, collage_strategy_t strategy,
                                                     collage_edq_t* per_tensor_out_dev, int num,
                                                     void* chunk_workspace, size_t chunk_workspace_bytes,
                                                     void* stream);
/* Plan facts for callers that report or shard: total elements, number of chunks. */
uint64_t collage_plan_num_elements(const collage_plan_t* plan);
uint64_t collage_plan_num_chunks(const collage_plan_t* plan);

/* Batched MCF primitives, elementwise over n bfloat16 values.  Output arrays may be the input
 * arrays themselves (exact same pointer); partial overlap is ERR_ALIAS.
 *   fast_two_sum (Theorem 4.1): hi = a (+) b, lo = b (-) (hi (-) a); error-free if |a| >= |b|
 *   two_sum      (Algorithm TwoSum): same expansion, no ordering needed, 6 operations
 *   two_prod     (Algorithm TwoProdFMA): hi = a (*) b, lo = fma(a, b, -hi)
 *   grow         (Algorithm 1): (u, v) = Fast2Sum(x, a); (u, v) = Fast2Sum(u, y (+) v)
 *   scaling      (Algorithm Scaling): float v times expansion (a1, a2)
 *   mul          (Algorithm Mul): expansion (a1, a2) times expansion (b1, b2)
 *   renormalize  (named in the paper's listing keywords, not defined there): Fast2Sum(hi, lo) */
collage_status_t collage_fast_two_sum(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream);
collage_status_t collage_two_sum(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream);
collage_status_t collage_two_prod(const void* a, const void* b, void* hi, void* lo, uint64_t n, void* stream);
collage_status_t collage_grow(const void* x, const void* y, const void* a, void* u, void* v, uint64_t n, void* stream);
collage_status_t collage_scaling(const void* v, const void* a1, const void* a2, void* x, void* e, uint64_t n, void* stream);
collage_status_t collage_mul(const void* a1, const void* a2, const void* b1, const void* b2, void* x, void* e,
                             uint64_t n, void* stream);
collage_status_t collage_renormalize(const void* hi_in, const void* lo_in, void* hi, void* lo, uint64_t n, void* stream);

/* One rounded bfloat16 operation F^BF16(a op b) elementwise (Section 3.1), realised exactly as
 * inside the step kernel.  op: 0 add, 1 sub, 2 mul, 3 div, 4 sqrt(a), 5 fma(a,b,c).  b is
 * ignored for sqrt; c only used by fma (pass NULL otherwise). */
collage_status_t collage_rounded_op(int op, const void* a, const void* b, const void* c, void* out,
                                    uint64_t n, void* stream);

/* EDQ on stored arrays (Eq. 2-3): old and new parameter expansions and the intended update.
 * old_lo/new_lo both NULL = plain bfloat16 parameter.  out_dev: DEVICE collage_edq_t*.
 * Errors: ERR_NULL, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA. */
collage_status_t collage_edq(const void* old_hi, const void* old_lo, const void* new_hi,
                             const void* new_lo, const void* delta, uint64_t n, collage_edq_t* out_dev,
                             void* workspace, size_t workspace_bytes, void* stream);

/* EDQ for callers that cannot allocate device memory (the paper has no counterpart; this is an
 * interface convenience, the computation is collage_edq's).  Some callers own no allocator they
 * may call at this point: a training process that has handed every byte of the GPU to a memory
 * pool and forbids raw cudaMalloc inside the step (it can fail, and it synchronises the device),
 * a plugin running inside someone else's framework without access to its allocator, or code in a
 * latency-critical region.  For them the scratch that collage_edq takes as `workspace` is built
 * into the library: a fixed 64 KiB array in device memory (2048 partial sums), which every GPU
 * that loads the library holds until the process exits.  Arguments are those of collage_edq
 * without workspace; `out_dev` is still the caller's DEVICE collage_edq_t.
 *   - Capacity: the array has 2048 slots and a thread block reduces up to 2^21 elements, so
 *     n <= 2^32; a larger n is rejected with COLLAGE_ERR_LIMIT and nothing is launched.
 *   - The call itself allocates nothing and frees nothing.  The first call on each device looks up
 *     the array's device address (cudaGetSymbolAddress, with that device current); make that first
 *     call before any stream capture begins.
 *   - All calls on a device share the one array.  Each call overwrites every slot it later reads,
 *     so nothing needs clearing between calls; but two calls whose kernels overlap on the GPU
 *     (different streams, no ordering) race on it.  Order them, or use collage_edq with separate
 *     workspaces.
 *   - The sums are grouped per segment of ceil(n / 2048) elements (rounded up to a multiple of 8,
 *     at least 2048), a function of n alone and not of the launch geometry, so they can differ from
 *     collage_edq's in the last bits (same tolerance as against the CPU oracle).
 * Errors: ERR_NULL, ERR_LIMIT, ERR_ARCH, ERR_CUDA. */
collage_status_t collage_edq_static(const void* old_hi, const void* old_lo, const void* new_hi,
                                    const void* new_lo, const void* delta, uint64_t n,
                                    collage_edq_t* out_dev, void* stream);

/* The step kernel's copy pipeline waits on shared-memory barriers with a bound of two seconds of
 * the device's wall clock; a wait that runs out records a code in a device word and the block
 * leaves, so a fault can never hang the device.  The kernel still ends normally and the call has
 * long returned COLLAGE_OK, but the step was torn: the state arrays are undefined from then on.
 * A step that reduces EDQ copies the word into its record (collage_edq_t.fault), so a caller that
 * reads the record sees the fault at once.  This call copies the word to *out_host (0 = no fault
 * seen on the current device since the last read) and clears it.  It synchronises the device: call
 * it at checkpoints, not per step.  Errors: ERR_NULL, ERR_CUDA. */
collage_status_t collage_pipeline_fault(uint32_t* out_host);

/* Exercises the give-up path of those waits without any fault: launches one warp that waits on a
 * barrier nothing completes, bounded by `limit_ms` milliseconds (1..1000) of the device's wall
 * clock.  The wait runs out, the kernel returns normally, and the next
 * collage_pipeline_fault reports the code 100.  The device and the library stay usable.
 * Asynchronous on `stream`.  Errors: ERR_ARG (limit out of range), ERR_ARCH, ERR_CUDA. */
collage_status_t collage_wait_timeout_selftest(uint32_t limit_ms, void* stream);

/* Exhaustive self test of the arithmetic the kernels rely on, on the current device (Section 3.1's
 * model: one rounding to nearest-even per operation).  Compares, for EVERY pair of bfloat16 bit
 * patterns (2^32 pairs; 2^16 values for the root), the realisation used in the kernels with a
 * reference built from IEEE float/double arithmetic and one conversion to bfloat16:
 *   out_host[0] add  [1] sub  [2] mul            native packed bfloat16 instructions
 *   out_host[3] div  [4] sqrt                    reciprocal / root approximations vs div.rn, sqrt.rn,
 *                                                both in the form that answers every operand and in the
 *                                                branch-free form of the step kernel (whose unflagged
 *                                                lanes must be right on all operands it admits)
 *   out_host[5] division by a scalar through a host-rounded reciprocal (divisors in (0, 1])
 * Each entry is the number of results that differ (NaNs compared as a class); all must be 0.
 * HOST output; allocates a few bytes, synchronises `stream`; takes about a second.
 * Errors: ERR_NULL, ERR_ARCH, ERR_CUDA. */
collage_status_t collage_selftest(uint64_t out_host[6], void* stream);

#ifdef __cplusplus
}
#endif
#endif /* COLLAGE_H_ */
