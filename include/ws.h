/*
 * ws.h - C ABI of the sharded weight update for data-parallel training.
 *
 * The library implements the data path of cross-replica weight-update
 * sharding on one GPU: R logical replicas are R gradient buffers in device
 * memory; the summed gradient of shard r (reduce-scatter arithmetic) drives a
 * fused optimizer update of the r-th 1/R slice of weights and optimizer
 * slots, and the updated weights are written in the all-gather output layout
 * (paper Section 2.2, "Sharding with decomposed all-reduce").
 *
 * Conventions for every call
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work on it and
 *     return; they never synchronise and never allocate or free device memory.
 *   - "device pointer" arguments must be 16-byte aligned; "host array"
 *     arguments are read before the call returns and may be freed afterwards.
 *   - Nothing throws or aborts across this boundary; every failure is a
 *     ws_status.  Argument errors are found on the host before any launch.
 *   - The caller owns every buffer.  The library owns only ws_plan objects.
 *   - The pack, unpack and update kernels use programmatic dependent launch:
 *     a kernel may start while the preceding kernel of the stream drains, but
 *     before it waits for that kernel it reads nothing except the plan's
 *     tables and the tensor-pointer tables.  Those tables must therefore be
 *     complete before the kernel that precedes such a call on the stream is
 *     launched:
 *     upload them with ws_plan_upload / ws_tensor_table_upload (copies, which
 *     a later kernel never overtakes) and do not rewrite them from a kernel
 *     of your own directly in front of such a call.
 *   - Accuracy a caller may expect against the same update in exact
 *     arithmetic, per tensor, as max_i |x_i - ref_i| / max(|ref_i|, RMS(ref)):
 *     1e-6 for the fp32 outputs of WS_SGDM and WS_ADAM, 1e-5 for WS_LAMB,
 *     WS_LARS and WS_ADAFACTOR (their per-tensor norms are fp32 sums), one
 *     bf16 ulp (2^-8 relative) for bf16 outputs.  These hold for gradients of
 *     the scale of the state they update (the library's test recipe: standard
 *     deviation 1e-3, up to 1024 copies).  Single elements can reach 1e-5
 *     (2.4e-5 seen) under WS_ADAM when gradient copies ten times larger are
 *     summed (not averaged) over 8 or more replicas, the copies cancel and
 *     the element's second moment starts at (almost) zero: the fp32 sum then
 *     carries an error that is large against the cancelled total, and the
 *     step divides by its root.  That is a property of fp32 summation (a
 *     pairwise fp32 sum of the same copies gives the library's value bit for
 *     bit), not of the sharding.
 *   - dtype arguments say how 2- or 4-byte elements are interpreted.
 *
 * Layout vocabulary (Section 4.1 "Sharding representation", Section 5.2
 * "Batched communication operators"):
 *   tensor t has n_t elements (row-major, flattened - all dimensions combined);
 *   its piece size is p_t = A * ceil(ceil(n_t / R) / A); shard r of tensor t is
 *   elements [r p_t, (r+1) p_t), positions >= n_t being padding;
 *   one combined shard is piece r of every tensor back to back, tensor t at
 *   offset off_t, so the shard length is S = sum_t p_t and a packed buffer has
 *   G = R * S elements laid out shard-major [R][S] - the layout an all-gather
 *   of R equal contributions produces.
 */
#ifndef WS_H_
#define WS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WS_OK = 0,
    WS_ERR_INVALID_ARG = 1, /* null pointer, bad count, r out of range, bad enum        */
    WS_ERR_ALIGNMENT = 2,   /* a device pointer is not 16-byte aligned                  */
    WS_ERR_DTYPE = 3,       /* dtype combination not supported                          */
    WS_ERR_WORKSPACE = 4,   /* workspace missing or smaller than ws_workspace_bytes     */
    WS_ERR_NOT_UPLOADED = 5,/* plan tables are not on the device yet (ws_plan_upload)   */
    WS_ERR_CUDA = 6,        /* a CUDA runtime call or a launch failed                   */
    WS_ERR_TOO_LARGE = 7    /* size beyond a documented fixed limit                     */
} ws_status;

typedef enum { WS_F32 = 0, WS_BF16 = 1 } ws_dtype;
typedef enum { WS_SGDM = 0, WS_ADAM = 1, WS_LAMB = 2, WS_LARS = 3, WS_ADAFACTOR = 4 } ws_opt;

#define WS_MAX_DIMS 8
typedef struct {
    int32_t ndim;               /* 0..WS_MAX_DIMS; ndim == 0 is a scalar (1 element) */
    int64_t dims[WS_MAX_DIMS];  /* every dim >= 0; a zero dim makes an empty tensor   */
    uint32_t flags;             /* reserved, pass 0                                    */
} ws_tensor_desc;

/* One row of the segment table: tensor t inside a combined shard. */
typedef struct {
    int64_t numel;      /* n_t                                   */
    int64_t piece;      /* p_t, a multiple of the alignment A    */
    int64_t shard_off;  /* off_t, start of the piece in a shard  */
} ws_segment;

typedef struct ws_plan ws_plan;

/* ---------------------------------------------------------------- plan ---
 * Shard planner (Section 4.1: combine dimensions, pad so the shard count
 * divides, dynamic-slice by replica id; Section 5.2: a combined shard holds
 * one shard of every tensor).  Host only, no CUDA call.
 *   descs       host array of T tensor descriptors, in the caller's order
 *   R           shard count = replica count, >= 1
 *   align_elems A: power of two >= 8, every piece is a multiple of A elements
 *   tile_elems  work-tile length in elements used by the kernels; 0 = default
 *               (1024 ... 8192: the largest power of two that leaves at
 *               least 20000 tiles over all shards and 600 per shard);
 *               otherwise a multiple of 1024
 *   out         receives a new plan; release with ws_plan_destroy
 * Errors: WS_ERR_INVALID_ARG for null/empty input, bad R, A or tile size. */
ws_status ws_plan_create(const ws_tensor_desc* descs, int32_t T, int32_t R, int32_t align_elems,
                         int32_t tile_elems, ws_plan** out);
void ws_plan_destroy(ws_plan* plan);

/* Second layout policy (Section 5.2, "Batched communication operators": for a
 * combined all-reduce the input tensors are concatenated in their full shapes
 * and the internal shards are partitions of the concatenation, not bound to
 * any tensor's own sharding).  WS_LAYOUT_CONCAT lays the tensors back to back
 * (each start rounded up to A elements), cuts the concatenation of length C
 * into R shards of S = A ceil(ceil(C / R) / A) elements wherever the
 * boundaries fall, and so pads at most A-1 elements per tensor plus a tail
 * shorter than R A - against up to R A per tensor for the per-tensor layout,
 * which is what makes tiny shards expensive at large R.  A tensor may span
 * several shards or share a shard with many others; every call of this
 * library accepts plans of either layout.  In ws_plan_segments `piece` is 0
 * and `shard_off` is the tensor's start inside the concatenation;
 * ws_plan_num_tiles counts the tiles of all shards.  ws_plan_create is
 * ws_plan_create_layout with WS_LAYOUT_PER_TENSOR. */
typedef enum { WS_LAYOUT_PER_TENSOR = 0, WS_LAYOUT_CONCAT = 1 } ws_layout;
ws_status ws_plan_create_layout(const ws_tensor_desc* descs, int32_t T, int32_t R, int32_t align_elems,
                                int32_t tile_elems, ws_layout layout, ws_plan** out);
int32_t ws_plan_layout(const ws_plan* plan);

int32_t ws_plan_num_tensors(const ws_plan* plan); /* T */
int32_t ws_plan_num_shards(const ws_plan* plan);  /* R */
int32_t ws_plan_align(const ws_plan* plan);       /* A */
int64_t ws_plan_shard_elems(const ws_plan* plan); /* S */
int64_t ws_plan_valid_elems(const ws_plan* plan); /* N = sum n_t */
int64_t ws_plan_num_tiles(const ws_plan* plan);   /* work tiles per shard */
/* Host view of the segment table; plan-owned, valid until ws_plan_destroy. */
ws_status ws_plan_segments(const ws_plan* plan, const ws_segment** segs, int32_t* T);

/* The kernels read the plan from device memory.  The caller provides a buffer
 * of at least ws_plan_device_bytes(plan) bytes (16-byte aligned) that must
 * stay alive and unmodified while the plan is in use; ws_plan_upload copies
 * the tables into it with one cudaMemcpyAsync on `stream`.  Upload once per
 * plan; afterwards the plan is immutable and may be shared between threads. */
size_t ws_plan_device_bytes(const ws_plan* plan);
ws_status ws_plan_upload(ws_plan* plan, void* dev_buf, size_t bytes, void* stream);

/* One-launch schedule (optional).  The norm-based optimizers need every shard's partial norm sums
 * of a tensor before any shard can apply the step (Section 4.1), so their all-shard update is
 * phase 1, a combination step, phase 2.  As three launches, phase 2 reads the weight and the new
 * moments from DRAM again.  A plan whose schedule has been uploaded runs WS_LAMB's all-shard update
 * as ONE kernel instead: the two phases of every tensor are work items (runs of up to 8192 shard
 * positions) ordered so that a tensor's phase 2 follows its phase 1 at a short distance, while other
 * tensors' phase 1 streams from DRAM, and phase 2 finds part of its operands in L2 (toward the
 * update of Section 2.2, where every operand crosses HBM once).  Results: the same as the
 * three-launch form up to the order of the norm sums (the ratios agree to rounding; they are
 * bit-stable from run to run).
 *   ws_plan_schedule_bytes   device bytes of the schedule (0: this plan has none - more than
 *                            65535 shards or 2^30 work items)
 *   ws_plan_upload_schedule  builds the schedule on first use and copies it into the caller's
 *                            buffer (16-byte aligned, alive while the plan is in use) with
 *                            cudaMemcpyAsync on `stream`; call once, before the plan is shared
 *                            between threads
 * Afterwards ws_shard_update / ws_fused_update with r == -1 and WS_LAMB (and
 * ws_lamb_update_static_scratch) take the one-kernel route when there are 8 to 32 gradient copies -
 * where it measured faster on a B200; other cases, WS_LARS and the shard-by-shard calls run as
 * before.  The kernel's waits (a phase-2 item waits for its tensor's ratio) are bounded: if one
 * ever runs out, the kernel leaves the update incomplete and sets the 32-bit status word inside
 * the workspace (ws_workspace_sync_status gives its byte offset; 0 = completed) - a caller that
 * wants to detect this reads the word after synchronising the stream.
 * ws_plan_schedule_view / ws_plan_schedule_item expose the order for inspection (host only):
 * entry i of `order` is item index * 2 + phase (0: phase 1, 1: phase 2). */
size_t ws_plan_schedule_bytes(const ws_plan* plan);
ws_status ws_plan_upload_schedule(ws_plan* plan, void* dev_buf, size_t bytes, void* stream);
typedef struct {
    int32_t tensor, shard;
    int64_t pos;        /* start inside the shard                     */
    int64_t tensor_off; /* element index of the start in the tensor   */
    int32_t len;        /* elements of the item                       */
    int32_t nvalid;     /* how many of them exist in the tensor       */
} ws_sched_item;
ws_status ws_plan_schedule_view(ws_plan* plan, const uint32_t** order, int64_t* n_entries);
ws_status ws_plan_schedule_item(ws_plan* plan, int64_t item, ws_sched_item* out);
ws_status ws_workspace_sync_status(const ws_plan* plan, size_t* offset_bytes);

/* ------------------------------------------------------- pack / unpack ---
 * ws_pack: flat[r S + off_t + q] = X_t[r p_t + q] where that location exists,
 * +0 (all-zero bits) otherwise.  This is the "sharding program" for weights
 * and optimizer slots (Section 4.2, out-of-loop placement) and the formatting
 * step in front of the reduce-scatter for gradients (Section 5.1).  Padding
 * is produced in place; the tensors are never read beyond n_t.
 *   tensor_ptrs host array of T device pointers (tensor t has n_t elements of
 *               `dtype`, contiguous)
 *   flat        device buffer of G = R*S elements of `dtype`, fully overwritten
 * ws_unpack is the reverse formatting after the all-gather (the "unsharding
 * program"): X_t[i] = flat[(i div p_t) S + off_t + i mod p_t]; pads are not
 * read.  Both are bit copies. */
ws_status ws_pack(const ws_plan* plan, const void* const* tensor_ptrs, ws_dtype dtype, void* flat,
                  void* stream);
ws_status ws_unpack(const ws_plan* plan, const void* flat, ws_dtype dtype,
                    void* const* tensor_ptrs, void* stream);

/* ------------------------------------------------------ sharded update --- */

/* The R gradient copies (one per logical replica).
 *   slice_mode 0: ptrs[k] is replica k's packed buffer of G elements; the call
 *                 for shard r reads elements [r S, (r+1) S) of each.
 *   slice_mode 1: ptrs[k] is the S-element slice for the shard being updated
 *                 (what a reduce-scatter receive buffer holds); only valid with
 *                 a single shard r >= 0.
 * Gradient pads may hold anything: they are masked by location, never read
 * into the result (Section 4.1, "Non-elementwise operators").
 * The number of gradient copies is normally the plan's shard count, but any
 * count from 1 to 1024 is accepted: with partial sharding (Section 5.2) the
 * replicas form N groups that each shard the update M ways, so a plan with M
 * shards is fed N*M copies - the per-group reduce-scatter followed by the
 * cross-group all-reduce is the sum of all N*M slices of shard j.  The same
 * holds for the number of sets in ws_fused_update's gradient table. */
typedef struct {
    const void* const* ptrs; /* host array of R device pointers */
    int32_t R;               /* number of gradient copies, 1..1024 */
    ws_dtype dtype;          /* WS_F32 or WS_BF16 */
    int32_t slice_mode;
} ws_grads;

/* fp32 master weights and optimizer slots, kept sharded between steps
 * (Section 2.2: auxiliary variables stay sharded across iterations).
 * With r >= 0 each pointer is the S-element shard r.  With r == -1 each is
 * the shard-major [R][S] buffer of all shards.  Updated in place; pads are
 * written +0.  v is unused (may be NULL) for WS_SGDM and WS_LARS.
 * With WS_ADAFACTOR m is unused (may be NULL) and v is the factored second
 * moment of every tensor, ws_plan_factored_elems() floats laid out as
 * ws_plan_factored_layout() says; it is small and is not sharded. */
typedef struct {
    void* w;
    void* m;
    void* v;
} ws_state;

/* Hyper-parameters.  The paper cites the optimizers without printing them;
 * the library computes, per valid element, with g = grad_scale * sum_k g_k:
 *   WS_SGDM  m' = momentum m + g + weight_decay w;        w' = w - lr m'
 *   WS_ADAM  m' = beta1 m + (1-beta1) g;  v' = beta2 v + (1-beta2) g^2;
 *            w' = w - lr (m'/(1-beta1^step)) / (sqrt(v'/(1-beta2^step)) + eps)
 *   WS_LAMB  m', v' as Adam; u = Adam direction + weight_decay w;
 *            rho_t = ||w_t|| / ||u_t|| over tensor t (1 if either norm is 0);
 *            w' = w - lr rho_t u
 *   WS_LARS  (the optimizer of the paper's ResNet-50 runs, Table 1; formula of
 *            the LARS paper it cites) per tensor t the local rate
 *            lambda_t = trust_coeff ||w_t|| / (||g_t|| + weight_decay ||w_t||)
 *            (1 if either norm is 0); m' = momentum m + lr lambda_t (g +
 *            weight_decay w);  w' = w - m'
 *   WS_ADAFACTOR (the paper's other example of an optimizer with reduce
 *            operators, Section 4.1; formula of the Adafactor paper it cites:
 *            factored second moments, update clipping, relative step size,
 *            no momentum).  Tensor t is a rows x cols matrix, cols its last
 *            dimension and rows all leading ones together; with
 *            beta = 1 - step^-decay_exponent:
 *            Rv' = beta Rv + (1-beta) rowsum(g^2 + eps);
 *            Cv' = beta Cv + (1-beta) colsum(g^2 + eps);
 *            V = Rv' Cv'^T / sum(Rv');  U = g / sqrt(V);
 *            w' = w - max(eps2, RMS(w_t)) min(lr, 1/sqrt(step))
 *                     U / max(1, RMS(U_t) / clip_threshold).
 *            A tensor of fewer than two dimensions keeps the full
 *            v' = beta v + (1-beta)(g^2 + eps) and uses V = v'.
 *            weight_decay must be 0.
 * `step` is the 1-based index of the update being applied.  Derived constants
 * are formed in double on the host and narrowed to fp32 for the kernels. */
typedef struct {
    ws_opt opt;
    double lr, beta1, beta2, eps, weight_decay, momentum, grad_scale;
    int64_t step;
    double trust_coeff; /* WS_LARS only (eta) */
    double eps2, clip_threshold, decay_exponent; /* WS_ADAFACTOR only (1e-3, 1.0, 0.8 in its paper) */
} ws_hyper;

/* Where the updated weights go in the all-gather output layout (Section 2.2;
 * Section 4.2: the full weight is only needed in bfloat16 while the update
 * stays fp32).  `gathered` is the base of a G-element buffer of `dtype`; the
 * call for shard r overwrites slot [r S, (r+1) S) completely, pads with +0.
 * bf16 values are the fp32 results rounded to nearest-even.  gathered may be
 * NULL: then nothing extra is written (with r == -1 the fp32 [R][S] weight
 * state already is the gathered layout). */
typedef struct {
    void* gathered;
    ws_dtype dtype;
} ws_out;

/* Adafactor's view of the plan's tensors (Section 4.1 names it as an optimizer
 * whose reduces collapse some dimensions and pass others through).  Tensor t of
 * two or more dimensions holds rows_t + cols_t floats of factored state (row
 * accumulator, then column accumulator); a tensor of fewer dimensions holds
 * numel_t floats.  ws_plan_factored_elems is the total F;
 * ws_plan_factored_layout fills layout[3 t + 0..2] = {offset of tensor t's
 * state in floats, rows_t, cols_t} with rows_t = numel_t, cols_t = 0 for the
 * unfactored ones.  layout is a host array of 3 T entries.  Host only. */
int64_t ws_plan_factored_elems(const ws_plan* plan);
ws_status ws_plan_factored_layout(const ws_plan* plan, int64_t* layout);

/* Bytes of caller-provided scratch (device, 16-byte aligned) the update needs:
 * 0 for WS_SGDM / WS_ADAM.  For WS_LAMB it holds, in this order:
 *   float  rho[T]            trust ratios written by ws_lamb_finalize
 *   (padding to 16 bytes)
 *   double norms[T][2]       squared norms (sum w^2, sum u^2) per tensor
 *   float  partials[R][tiles][2]   per-tile partial sums from phase 1
 *                                  ([tiles][2] for the concatenated layout)
 *   (scratch of the one-launch route: per-item partial sums, per-tensor
 *    counters and flags, a ticket counter and the status word)
 * so a caller can read rho and the norms back for logging.  WS_LARS uses the
 * same arrays (rho holds the local rates, norms sum w^2 and sum g^2)
 * followed, at the next 256-byte boundary, by
 *   float  ghat[R][S]        the summed gradients kept from phase 1 for phase 2
 * WS_ADAFACTOR uses all four (rho holds the applied step size alpha_t / max(1,
 * RMS(U_t)/d), norms sum w^2 and sum U^2) followed by
 *   float  acc[F']           this step's row / column sums of g^2 + eps
 *   double rsum[T]           sum of the new row accumulators per tensor
 *   float  fac[F']           1/sqrt factors of V for the two elementwise passes
 *   float  alpha[T]          max(eps2, RMS(w_t)) min(lr, 1/sqrt(step))
 * where F' is F = ws_plan_factored_elems() with every tensor's row part and
 * column part padded to a multiple of 8 floats.  The WS_ADAFACTOR workspace
 * must be 32-byte aligned (its second pass reads ghat with 256-bit loads);
 * a workspace that is only 16-byte aligned is refused with WS_ERR_ALIGNMENT. */
size_t ws_workspace_bytes(const ws_plan* plan, ws_opt opt);

/* Where the per-tile partial sums live inside the workspace: byte offset of
 * partials[0] and the bytes of one shard's row (per-tensor layout: tiles * 8).
 * A multi-GPU caller that runs ws_lamb_partial for its own shard r on every
 * rank exchanges row r with the other ranks (an all-gather of rows, or an
 * all-reduce over rows that are zero elsewhere: the combination of per-replica
 * reduce results of Section 4.1) before every rank calls ws_lamb_finalize.
 * Host only.  WS_ERR_INVALID_ARG for the concatenated layout, whose shards own
 * different numbers of tiles. */
ws_status ws_workspace_partials(const ws_plan* plan, size_t* offset_bytes, size_t* row_bytes);

/* Fused reduce + optimizer update + gathered-layout write for shard r
 * (0 <= r < R), or for all R shards in one launch when r == -1.
 * Reads the r-th slice of each of the R gradient buffers exactly once, w/m/v
 * once, writes w/m/v (and the gathered slot) once (Section 2.2: the update is
 * memory bound - read gradient, weight, auxiliaries; write weight,
 * auxiliaries).  With opt == WS_LAMB or WS_LARS only r == -1 is accepted here
 * (phase 1 over all shards, finalize, phase 2 over all shards): the per-tensor
 * ratio needs every shard's partial norms before any shard can apply
 * (Section 4.1).
 * WS_ADAFACTOR (r == -1 only) runs three passes: (1) reduce the gradients, keep
 * the sum, and add every tile's partial row sums and column sums of g^2 + eps
 * (pads masked by location) into acc - the sharding cuts rows and columns, so
 * this stands where the paper combines the shards' partial reduce results with
 * an all-reduce (Section 4.1, "Non-elementwise operators"); a finalize step
 * forms Rv', Cv' and the step size; (2) sum U^2 per tensor; a second finalize
 * forms the clipping; (3) apply.  The row and column sums use floating-point
 * atomic adds, so Rv', Cv' and everything after them can differ in the last
 * bits between runs. */
ws_status ws_shard_update(const ws_plan* plan, int32_t r, const ws_grads* grads,
                          const ws_state* state, const ws_hyper* hyper, const ws_out* out,
                          void* workspace, size_t workspace_bytes, void* stream);

/* LAMB shard by shard (what one replica would run).  Phase 1 for shard r:
 * reduce, moments m'/v' written, per-tile partial sums of w^2 and u^2 over
 * valid locations stored to workspace (pads masked with the identity by
 * comparing locations with n_t).  ws_lamb_finalize sums every shard's
 * partials in a fixed order in double and writes rho[T]; it stands where the
 * paper has the combined scalar all-reduce (Section 5.2), so call it after
 * phase 1 of ALL shards.  Phase 2 for shard r recomputes u from w, m', v' and
 * applies w' = w - lr rho u, writing the gathered slot.  hyper->opt must be
 * WS_LAMB.
 * The shard-by-shard form gives bit for bit the result of the all-shard call
 * when every shard slice handed in is 32-byte aligned (S * element size a
 * multiple of 32: any A for fp32, A >= 16 for bf16 gradient slices);
 * otherwise the kernels fall back to 128-bit accesses for that shard, the
 * partial sums are formed in another order and the ratios agree to rounding. */
ws_status ws_lamb_partial(const ws_plan* plan, int32_t r, const ws_grads* grads,
                          const ws_state* state, const ws_hyper* hyper, void* workspace,
                          size_t workspace_bytes, void* stream);
ws_status ws_lamb_finalize(const ws_plan* plan, void* workspace, size_t workspace_bytes,
                           void* stream);
ws_status ws_lamb_apply(const ws_plan* plan, int32_t r, const ws_state* state,
                        const ws_hyper* hyper, const ws_out* out, void* workspace,
                        size_t workspace_bytes, void* stream);

/* LARS shard by shard, the same three steps (the paper ran ResNet-50 with LARS
 * on real replicas, Table 1): phase 1 for shard r reduces the gradients, keeps
 * the sum in ghat slot r of the workspace and leaves per-tile partial sums of
 * w^2 and g^2; ws_lars_finalize (after phase 1 of ALL shards, with every
 * shard's partial rows present in the workspace - ws_workspace_partials) forms
 * the local rates lambda_t from hyper->trust_coeff and hyper->weight_decay;
 * phase 2 for shard r applies the momentum step and writes the gathered slot.
 * The workspace has ws_workspace_bytes(plan, WS_LARS) bytes.  hyper->opt must
 * be WS_LARS. */
ws_status ws_lars_partial(const ws_plan* plan, int32_t r, const ws_grads* grads,
                          const ws_state* state, const ws_hyper* hyper, void* workspace,
                          size_t workspace_bytes, void* stream);
ws_status ws_lars_finalize(const ws_plan* plan, const ws_hyper* hyper, void* workspace,
                           size_t workspace_bytes, void* stream);
ws_status ws_lars_apply(const ws_plan* plan, int32_t r, const ws_state* state,
                        const ws_hyper* hyper, const ws_out* out, void* workspace,
                        size_t workspace_bytes, void* stream);

/* Adafactor stage by stage, for one shard r >= 0 or all shards (r == -1): what
 * ws_shard_update(WS_ADAFACTOR) runs in this order.  On real replicas each
 * runs the per-shard stages for its own shard and exchanges the reduce results
 * between them - the case of Section 4.1 where "sharding affects the collapsed
 * dimensions": every replica reduces what its shard holds, then the replicas
 * combine their results with an all-reduce.
 *   WS_AF_BEGIN    clears this step's row / column sums (no shard argument)
 *   WS_AF_SUMS     shard r: reduce the gradients, keep the sum (ghat slot r),
 *                  add the shard's partial row / column sums of g^2 + eps into
 *                  the sums, leave per-tile sums of w^2
 *                  -> exchange: all-reduce (sum) the float region
 *                     ws_workspace_adafactor_sums() names; share the partial
 *                     rows (ws_workspace_partials)
 *   WS_AF_MOMENTS  Rv', Cv' (state->v, the same on every replica) and the
 *                  1/sqrt factors
 *   WS_AF_SUMSQ    shard r: per-tile sums of U^2
 *                  -> exchange: share the partial rows again
 *   WS_AF_CLIP     step sizes alpha_t / max(1, RMS(U_t)/d) for every tensor
 *   WS_AF_APPLY    shard r: w' = w - step size * U, gathered slot r
 * Arguments a stage does not use may be NULL (grads outside WS_AF_SUMS, out
 * outside WS_AF_APPLY, state in WS_AF_BEGIN / SUMSQ / CLIP).  The workspace has
 * ws_workspace_bytes(plan, WS_ADAFACTOR) bytes and persists through the stages. */
typedef enum {
    WS_AF_BEGIN = 0, WS_AF_SUMS = 1, WS_AF_MOMENTS = 2, WS_AF_SUMSQ = 3, WS_AF_CLIP = 4, WS_AF_APPLY = 5
} ws_af_stage;
ws_status ws_adafactor_stage(const ws_plan* plan, ws_af_stage stage, int32_t r, const ws_grads* grads,
                             const ws_state* state, const ws_hyper* hyper, const ws_out* out,
                             void* workspace, size_t workspace_bytes, void* stream);
/* Byte offset and size of the float array of row / column sums inside the
 * Adafactor workspace (the all-reduce operand between WS_AF_SUMS and
 * WS_AF_MOMENTS).  Host only. */
ws_status ws_workspace_adafactor_sums(const ws_plan* plan, size_t* offset_bytes, size_t* bytes);

/* ------------------------------------- formatting fused into the update ---
 * Section 5.1: padding the gradient before the reduce-scatter costs every
 * replica a read and a write of the full data, so the paper fuses the
 * formatting into the reduce-scatter and the all-gather and pads in place.
 * ws_fused_update is that fusion on one GPU: the kernel reads the R replicas'
 * gradients straight from their tensor lists (element r p_t + q of tensor t
 * for shard position off_t + q; positions past n_t are never read), updates
 * the sharded fp32 state exactly as ws_shard_update does, and writes the
 * updated weights straight into the weight tensors (fp32, or bf16 rounded to
 * nearest-even, Section 4.2).  No packed gradient buffer and no gathered
 * buffer exist; results are bit-identical to ws_pack of every gradient list,
 * ws_shard_update, ws_unpack.
 *
 * Tensor pointers reach the kernel through a device-resident table that is
 * uploaded once (the tensors of a training job stay where they are):
 *   ws_tensor_table_upload copies `nsets` lists of T device pointers (host
 *   array, set-major: ptrs[k*T + t]) into the caller's device buffer of at
 *   least ws_tensor_table_bytes(plan, nsets) bytes with one cudaMemcpyAsync and
 *   fills *out, which the caller passes to ws_fused_update and keeps alive,
 *   together with the device buffer, while it is in use.  Every tensor pointer
 *   must be 16-byte aligned; 32-byte alignment of all of them lets the kernels
 *   use 256-bit accesses.
 * The tensors may live in any memory the device can address, pinned host
 * memory included: the kernel then pulls the gradients over PCIe itself and
 * writes the weights back the same way, with no staging copy (the table
 * itself must be in device memory).
 * ws_fused_update arguments: `grads` is a table of R sets (the R replicas'
 * gradient lists), `weights` a table of one set (the weight tensors that
 * receive the result), `state` as for ws_shard_update (r >= 0: one shard;
 * r == -1: all shards, the only form accepted for WS_LAMB, WS_LARS and
 * WS_ADAFACTOR), `workspace` as for ws_shard_update.
 * With WS_SGDM and WS_ADAM `weights` may hold up to grads->nsets sets: the
 * kernel then writes the updated weights into every set.  This is the form
 * for real replicas whose tensors are mapped into one another's address space
 * (CUDA IPC or symmetric memory; the caller fills the tables with the peers'
 * addresses): replica r calls ws_fused_update(plan, r, ...) with the R
 * replicas' gradient lists and the R replicas' weight lists, so the one kernel
 * pulls its slice of every peer's gradients (the reduce-scatter), updates its
 * shard, and stores the new weights into every peer's tensors (the
 * all-gather) - Section 5.1's fusion of the formatting into both collectives,
 * with plain peer loads and stores.  The caller orders the kernels of
 * different replicas (gradients complete before, weights read after). */
typedef struct {
    void* dev;        /* device table, layout [T][nsets] */
    int32_t nsets;
    int32_t T;
    ws_dtype dtype;   /* element type of the tensors the table points to */
    int32_t min_align;/* largest power of two (<= 256) dividing every pointer */
} ws_tensor_table;

size_t ws_tensor_table_bytes(const ws_plan* plan, int32_t nsets);
ws_status ws_tensor_table_upload(const ws_plan* plan, const void* const* ptrs, int32_t nsets,
                                 ws_dtype dtype, void* dev_buf, size_t bytes, void* stream,
                                 ws_tensor_table* out);
/* ws_pack of every set of a tensor table in ONE launch: set k goes to flats[k] (host array of
 * table->nsets device pointers, G elements of the table's dtype each).  Same result as nsets calls
 * of ws_pack; meant for the R gradient lists of a step on the separate-kernel route. */
ws_status ws_pack_sets(const ws_plan* plan, const ws_tensor_table* table, void* const* flats,
                       void* stream);
ws_status ws_fused_update(const ws_plan* plan, int32_t r, const ws_tensor_table* grads,
                          const ws_state* state, const ws_hyper* hyper,
                          const ws_tensor_table* weights, void* workspace, size_t workspace_bytes,
                          void* stream);

/* ------------------------------------------------- host-buffer step ---
 * One whole step for callers whose gradients and weights live in HOST memory
 * (the end-to-end form of the path of Section 2.2: local gradients in, full
 * updated weights out).  A "tensor arena" is the model's tensors back to back
 * in the caller's order, each tensor's start rounded up to a multiple of 8
 * elements; ws_plan_arena_elems gives its length and ws_plan_arena_offsets the
 * start of every tensor (plan-owned array of T offsets, in elements).
 *
 * ws_step_host enqueues on `stream`, for k = 0..R-1: copy host_grads[k]
 * (arena of grad_dtype) to dev_grad_arena, pack it into dev_packed_grads[k];
 * then the fused update of all shards (as ws_shard_update with r == -1 on
 * `state`, writing `out` if out->gathered is set); then unpack the updated
 * weights (from out->gathered if set, else from state->w) into
 * dev_weight_arena and copy that to host_weights.  Copies are
 * cudaMemcpyAsync: with pinned host memory the call returns before the work
 * is done, and host_weights is valid after the stream is synchronised.
 * Nothing is allocated; all device buffers are the caller's:
 *   dev_grad_arena    arena_elems elements of grad_dtype (staging, reused)
 *   dev_packed_grads  host array of R device pointers, G elements each
 *   dev_weight_arena  arena_elems elements of the weight dtype
 * The weight dtype is out->dtype when out->gathered is set, else WS_F32. */
int64_t ws_plan_arena_elems(const ws_plan* plan);
ws_status ws_plan_arena_offsets(const ws_plan* plan, const int64_t** offsets, int32_t* T);

typedef struct {
    const void* const* host_grads; /* host array of R HOST pointers */
    ws_dtype grad_dtype;
    void* dev_grad_arena;
    void* const* dev_packed_grads;
    void* dev_weight_arena;
    void* host_weights;            /* HOST arena, arena_elems elements */
} ws_host_io;

ws_status ws_step_host(const ws_plan* plan, const ws_host_io* io, const ws_state* state,
                       const ws_hyper* hyper, const ws_out* out, void* workspace,
                       size_t workspace_bytes, void* stream);

/* ------------------------------------- LAMB without a caller workspace ---
 * (No counterpart in the paper: this entry point exists for deployment
 * reasons only.)
 *
 * ws_lamb_update_static_scratch does exactly what ws_shard_update does for
 * opt == WS_LAMB and r == -1 (phase 1 over all shards, finalize, phase 2 over
 * all shards; same arguments, same results), but needs no `workspace`: the
 * trust ratios, norms and per-tile partial sums go to an array of
 * WS_STATIC_SCRATCH_BYTES that is built into the library.  It is meant for
 * callers that cannot get device memory when the update runs - an optimizer
 * plug-in inside a framework whose allocator already owns the whole GPU, a step
 * loop that must stay out of the CUDA allocator because cudaMalloc can stall
 * the device, a binding layer that can forward buffers but not create them.
 * The call performs no device allocation or free of any kind.
 *
 * Limits and rules:
 *   - ws_workspace_bytes(plan, WS_LAMB) must not exceed WS_STATIC_SCRATCH_BYTES
 *     (4 MiB; enough for BERT-large at R = 16 with the default tile size),
 *     otherwise WS_ERR_TOO_LARGE is returned and nothing is launched.
 *   - Every GPU that loads the library carries the array until the process
 *     exits, whether or not this entry point is ever called.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call outside any
 *     stream capture.  Later calls on the same device skip the lookup.  The
 *     cached address belongs to the device's primary context: do not reset
 *     the device (cudaDeviceReset) while the library stays loaded, the next
 *     call would hand the kernels the old context's address.
 *   - All calls on one device share the one array, and it keeps whatever the
 *     previous call left in it.  Nothing in it needs clearing (each call
 *     overwrites every entry it later reads), but two calls whose kernels can
 *     run at the same time on one GPU - different streams, different threads -
 *     would overwrite each other's partial sums: serialise them.
 *   - The caller still owns and passes gradients, state and the gathered
 *     output exactly as for ws_shard_update. */
#define WS_STATIC_SCRATCH_BYTES (4u * 1024u * 1024u)
size_t ws_static_scratch_bytes(void); /* == WS_STATIC_SCRATCH_BYTES of the loaded library */
ws_status ws_lamb_update_static_scratch(const ws_plan* plan, const ws_grads* grads,
                                        const ws_state* state, const ws_hyper* hyper,
                                        const ws_out* out, void* stream);

/* ---------------------------------------------- bounds-checking debug build ---
 * (Test infrastructure of the library, no counterpart in the paper.)  A copy of the library
 * compiled with -DWS_DEBUG_BOUNDS (`python -m paper_2004_13336_b200.build --debug` builds it as
 * libws_debug.so; the Python binding loads it when the environment variable WS_DEBUG_BOUNDS is 1)
 * makes every kernel compare the range of each work item with the extents of the buffers it was
 * given before it touches them.  A range outside them ORs a bit into a status word and the item is
 * skipped; nothing traps or asserts.
 *   ws_debug_bounds_enabled   1 in the debug build, 0 in the regular one
 *   ws_debug_bounds_read      synchronises the device, returns the bits (1: w / m / v, 2: a packed
 *                             gradient buffer, 4: the gathered buffer or the stored gradient sum,
 *                             8: the flat buffer of ws_pack / ws_unpack, 0x40000000: the self-test)
 *                             and clears them when `clear` is non-zero; WS_ERR_INVALID_ARG in the
 *                             regular build
 *   ws_debug_bounds_selftest  runs the check on an index outside its extent (no memory is
 *                             accessed), so a test can see the bit arrive */
int32_t ws_debug_bounds_enabled(void);
ws_status ws_debug_bounds_read(uint32_t* bits, int32_t clear);
ws_status ws_debug_bounds_selftest(void* stream);

/* Static, never NULL. */
const char* ws_status_string(ws_status s);
/* Text of the last CUDA error seen by the calling thread inside this library
 * ("" if none).  Static storage per thread. */
const char* ws_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* WS_H_ */
