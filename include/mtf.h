/*
 * mtf.h - C ABI of the B200 library for layout-lowered named-dimension einsum (Mesh-TensorFlow,
 * arXiv 1811.02084) and the Transformer blocks built from it.
 *
 * Model of the paper that this boundary follows
 *   - A mesh is an n-dimensional array of (here: virtual) processors with named dimensions
 *     (Section 2, Section 4).
 *   - Tensors have named dimensions; a computation layout maps tensor-dimension names to
 *     mesh-dimension names (Section 4).  A tensor's layout is the restriction of that map to its
 *     own dimensions; it must be injective and sizes must divide (Section 5).
 *   - Processor p keeps, along every mapped dimension, the contiguous block selected by its mesh
 *     coordinate (Section 5).  Processor ranks unrank row-major over the mesh dimensions, last
 *     mesh dimension fastest.
 *   - An einsum is a local einsum on every processor's slices followed by a sum over the group of
 *     processors that differ only along the mesh dimensions of reduced-out split dimensions
 *     (Section 6, "Einstein Summation").  On one GPU that sum is an on-device reduction.
 *
 * General conventions
 *   - Every tensor is stored ONCE, globally, dense and row-major in the order of its `dims`
 *     (last dimension contiguous).  A processor's slice is a box view of it; replicas are logical.
 *   - `data` pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     The library never allocates tensor memory; scratch space is passed in as `workspace`.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Launches are
 *     asynchronous; no call synchronises the device unless stated.
 *   - All validation happens before any launch.  Every call returns an mtf_status; nothing throws
 *     or aborts across this boundary.  mtf_last_error() gives thread-local detail text.
 *   - Handles are immutable after creation, may be shared between threads, and are destroyed by
 *     the caller.  Strings are copied at creation.
 */
#ifndef MTF_H_
#define MTF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MTF_OK = 0,
  MTF_ERR_INVALID_ARG = 1,      /* NULL pointer, bad count, bad dtype, duplicate layout rule ...        */
  MTF_ERR_DUPLICATE_DIM = 2,    /* a tensor or mesh carries one dimension name twice (Section 4)        */
  MTF_ERR_UNKNOWN_DIM = 3,      /* a name that is not there: mesh dim of a rule, output dim of einsum   */
  MTF_ERR_SIZE_MISMATCH = 4,    /* one dimension name with two sizes in one operation                   */
  MTF_ERR_ILLEGAL_LAYOUT = 5,   /* two dims of a tensor / of an operation on one mesh dim (Section 8.5) */
  MTF_ERR_NOT_DIVISIBLE = 6,    /* split dimension size not divisible by the mesh-dim size (Section 5)  */
  MTF_ERR_UNSUPPORTED = 7,      /* legal in the paper's language, not implemented on the GPU path       */
  MTF_ERR_WORKSPACE_TOO_SMALL = 8,
  MTF_ERR_CUDA = 9,             /* a CUDA runtime/driver call failed; text in mtf_last_error()          */
  MTF_ERR_TIMEOUT = 10          /* a bounded device-side wait gave up (see mtf_device_status)           */
} mtf_status;

typedef enum { MTF_F32 = 0, MTF_BF16 = 1 } mtf_dtype;

/* Opaque handles.  (The layout handle type carries a _t because mtf_layout is the call that makes one.) */
typedef struct mtf_mesh_s mtf_mesh_t;
typedef struct mtf_layout_s mtf_layout_t;
typedef struct mtf_plan_s mtf_plan_t;

/* A named dimension (Section 4): name + static size.  Sizes are at least 1: a tensor with an empty
 * dimension has no slices to lay out and every call that sees one returns MTF_ERR_INVALID_ARG. */
typedef struct { const char* name; int64_t size; } mtf_dim;

/* A named tensor: non-owning view.  `data` is a device pointer (ignored where stated). */
typedef struct { void* data; mtf_dtype dtype; int32_t ndim; const mtf_dim* dims; } mtf_tensor;

/* Component-wise work fused into an einsum's output (Section 6 "Component-wise Operations",
 * Section 7 implicit broadcasting), applied in this order to the fp32 accumulator:
 *     t = scale * acc;  t += bias (broadcast);  if relu: t = max(t, 0);
 *     if relu_mask: t = (relu_mask > 0) ? t : 0;   t += residual;   out = cast(t)
 * bias      : dims must be a subset of the output dims (any order);  f32 or bf16.
 * relu_mask : same dims, same order and dtype class as the output (bf16 or f32).
 * residual  : same dims and order as the output (bf16 or f32).
 * reduce_sum_out : optional second output (Section 6 "Reduction" fused into the einsum): an f32
 *             tensor whose dims are a subset of the output dims; it receives the sum of t (taken
 *             after the relu_mask stage, before the residual and the cast) over the other output
 *             dims.  The library zeroes it on the stream before the launch and accumulates with
 *             fp32 atomics (order not fixed).  Used for dbias = sum over tokens of dhp.
 * NULL pointers / relu = 0 / scale = 1 switch a stage off.  The struct is read during planning
 * only for which stages are on and their descriptors; data pointers are read at exec time. */
typedef struct {
  float scale;
  int32_t relu;
  const mtf_tensor* bias;
  const mtf_tensor* relu_mask;
  const mtf_tensor* residual;
  const mtf_tensor* reduce_sum_out;
} mtf_epilogue;

/* Which kernel family a plan runs (informational; chosen by the planner). */
typedef enum { MTF_KERNEL_SIMT = 0, MTF_KERNEL_TCGEN05 = 1 } mtf_kernel_kind;
/* How the sum over a reduce group is realised (Section 6: the Allreduce after the local einsum).
 *   CHAINED   : the CTA that owns an output tile runs the K loops of the group's slices back to
 *               back, in ascending processor order, into one accumulator (no extra HBM traffic).
 *   WORKSPACE : every (slice, tile) writes an fp32 partial to the workspace; the CTA that arrives
 *               last for a tile sums the partials in ascending processor order and finishes it. */
typedef enum { MTF_REDUCE_NONE = 0, MTF_REDUCE_CHAINED = 1, MTF_REDUCE_WORKSPACE = 2 } mtf_reduce_mode;

/* ---- mesh (Section 2, Section 4) ------------------------------------------------------------ */
/* mesh_dims: host array of ndim (name, size) pairs, 1 <= ndim <= 4, sizes >= 1, names distinct. */
mtf_status mtf_mesh_create(int32_t ndim, const mtf_dim* mesh_dims, mtf_mesh_t** out);
mtf_status mtf_mesh_destroy(mtf_mesh_t* mesh);
/* Number of processors P and, for processor p, its coordinates (host array of the mesh's ndim). */
mtf_status mtf_mesh_size(const mtf_mesh_t* mesh, int64_t* n_processors);
mtf_status mtf_mesh_coords(const mtf_mesh_t* mesh, int64_t processor, int64_t* coords);

/* ---- computation layout (Section 4; examples in Section 8.1-8.5, Section 9) ------------------ */
/* nrules pairs tensor_dim[i] -> mesh_dim[i] (host strings).  A tensor dimension may appear once
 * (it is a map); several tensor dimensions may map to one mesh dimension; the mesh dimension
 * must exist (MTF_ERR_UNKNOWN_DIM).  nrules = 0 is the legal empty layout (Section 8.4).
 * The layout keeps a reference to nothing: the mesh may be destroyed afterwards. */
mtf_status mtf_layout(const mtf_mesh_t* mesh, int32_t nrules, const char* const* tensor_dim,
                      const char* const* mesh_dim, mtf_layout_t** out);
mtf_status mtf_layout_destroy(mtf_layout_t* layout);
/* Legality of one tensor under the layout (Section 5, Section 8.5): MTF_ERR_DUPLICATE_DIM,
 * MTF_ERR_ILLEGAL_LAYOUT or MTF_ERR_NOT_DIVISIBLE, else MTF_OK. */
mtf_status mtf_layout_check_tensor(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* dims);
/* Slice box of `processor` (Section 5): host outputs offsets[ndim], sizes[ndim]; the local index l
 * maps to the global flat index sum_i (offsets[i] + l_i) * prod_{i' > i} dims[i'].size. */
mtf_status mtf_slice_map(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* dims, int64_t processor,
                         int64_t* offsets, int64_t* sizes);
/* Device copy of one processor's slice of `global` into the dense row-major buffer `out_slice`
 * (device, same dtype, prod(sizes) elements).  One kernel launch on `stream`. */
mtf_status mtf_slice_gather(const mtf_layout_t* layout, const mtf_tensor* global, int64_t processor,
                            void* out_slice, void* stream);

/* ---- one mesh dimension across several GPUs (Section 2: a mesh is a naming abstraction over the
 * physical processors; Section 3, Algorithm 1 line 2: the gradient Allreduce; Section 8.1 / 8.2 /
 * Table 1 "Comm." column: which einsums need an Allreduce under which layout) ----------------------
 * One process per GPU.  mtf_layout_bind_ranks maps mesh dimension `mesh_dim` (size m, divisible by
 * `world`) onto `world` ranks: rank r owns the virtual processors whose coordinate on that mesh
 * dimension lies in [r m / world, (r + 1) m / world).  The returned handle is a layout over THIS
 * RANK'S part of the mesh (that mesh dimension has m / world processors in it), and every tensor
 * handed to a call under it is the rank's box of the global tensor: a dimension that the layout
 * splits over `mesh_dim` has its global size / world here (mtf_rank_box gives the box), everything
 * else is whole (replicated across ranks).  All calls work as on one GPU; in addition
 *   - an einsum (or reduction) that sums out a dimension split over `mesh_dim` leaves, on every
 *     rank, a partial result that the ranks must add up: mtf_plan_needs_rank_sum says so, and when
 *     collective hooks were given the library calls `start(user, data, count, dtype, stream)` right
 *     behind the launch that produced the partial result (the hook enqueues a sum over all ranks, in
 *     place, that begins when `stream` reaches this point, and returns without blocking);
 *   - `wait(user, stream)` makes `stream` wait for every sum started so far.  The block calls
 *     (mtf_ffn_*, mtf_attention_*, mtf_decoder_layer_*, mtf_layernorm_backward) call it before a
 *     launch that reads a summed tensor and before they return; after a bare mtf_einsum call
 *     mtf_rank_wait when the result is needed;
 *   - component-wise stages that are not linear (bias, relu, relu_mask, a fused reduce_sum of such
 *     values, a row softmax) cannot ride in a launch whose result is only a partial sum:
 *     MTF_ERR_UNSUPPORTED.  A residual can: rank 0 adds it, the others do not.
 * The hooks are the only place where ranks meet; the library itself links no communication library
 * (the Python binding provides hooks over torch.distributed: NCCL on GPUs, gloo in CPU tests).
 * Hooks may be NULL (both or neither): the caller then sums the flagged outputs itself.
 * world = 1 is legal and changes nothing. */
typedef mtf_status (*mtf_rank_allreduce_fn)(void* user, void* data, int64_t count, mtf_dtype dtype, void* stream);
typedef mtf_status (*mtf_rank_wait_fn)(void* user, void* stream);
mtf_status mtf_layout_bind_ranks(const mtf_layout_t* layout, const char* mesh_dim, int32_t world, int32_t rank,
                                 mtf_rank_allreduce_fn start, mtf_rank_wait_fn wait, void* user, mtf_layout_t** out);
/* This rank's box of a GLOBAL tensor under a rank-bound layout: host outputs offsets[ndim], sizes[ndim]. */
mtf_status mtf_rank_box(const mtf_layout_t* bound_layout, int32_t ndim, const mtf_dim* global_dims, int64_t* offsets, int64_t* sizes);
/* 1 when the plan's result is a partial sum the ranks still have to add up (bit 0: the output, bit 1:
 * the fused reduce_sum output), else 0.  Always 0 under a layout that is not rank-bound. */
mtf_status mtf_plan_needs_rank_sum(const mtf_plan_t* plan, int32_t* flags);
mtf_status mtf_rank_wait(const mtf_layout_t* bound_layout, void* stream);

/* ---- einsum (Section 6 "Einstein Summation"; Section 8 code fragment) ------------------------- */
/* Plan  out[out dims] = sum over dims not in out of  in[0] * in[1]  under `layout`.
 * The equation is carried by the dimension names, as in mtf.einsum(x, w, output_shape=[...]).
 * n_in must be 2 (MTF_ERR_UNSUPPORTED otherwise).  `data` of the descriptors is ignored here.
 * Errors: duplicate names, size mismatch, output dim in no input (MTF_ERR_UNKNOWN_DIM), illegal
 * layout for any operand or for the whole iteration space, non-divisible split sizes, and
 * MTF_ERR_UNSUPPORTED for a dimension that only one input has and the output lacks.
 * A bf16 x bf16 einsum that the tensor-core kernel cannot take (strides that are not 16-byte aligned,
 * an N slice that is not a multiple of 8, a reduced dimension that only one operand has, more than
 * three batch dimensions) runs on the generic one-thread-per-element kernel only up to 2^30
 * multiply-adds; above that the plan is refused with MTF_ERR_UNSUPPORTED and the reason in
 * mtf_last_error(), unless mtf_plan_force(MTF_KERNEL_SIMT, ..) asked for the generic kernel. */
mtf_status mtf_einsum_plan(const mtf_layout_t* layout, int32_t n_in, const mtf_tensor* in_desc,
                           const mtf_tensor* out_desc, const mtf_epilogue* epilogue, mtf_plan_t** out);
mtf_status mtf_plan_destroy(mtf_plan_t* plan);
/* Scratch bytes mtf_einsum_exec needs (0 unless the reduce mode is WORKSPACE). */
mtf_status mtf_plan_workspace_bytes(const mtf_plan_t* plan, size_t* bytes);
/* Per-processor cost counts (Table 1; Appendix B): multiply-adds of the local einsum, values
 * entering the Allreduce (one output slice when a split dimension is reduced out, else 0), local
 * elements of inputs plus output, and how many mesh dimensions are reduced over. */
mtf_status mtf_plan_cost(const mtf_plan_t* plan, int64_t* macs_per_proc, int64_t* allreduce_values_per_proc,
                         int64_t* slice_elems_per_proc, int32_t* n_reduce_mesh_dims);
/* What the planner decided: kernel family, reduce mode, number of distinct slices computed
 * (replicas are computed once, Section 8.4), reduce-group size, and the reduced mesh dims as a bit mask. */
mtf_status mtf_plan_info(const mtf_plan_t* plan, int32_t* kernel_kind, int32_t* reduce_mode,
                         int64_t* n_slices, int64_t* group_size, uint32_t* reduce_mesh_dim_mask);
/* Run a plan.  in[0..1] and out carry device pointers; dims must equal the planned ones.
 * epilogue may be NULL only if the plan was made without one.  One kernel launch (plus one memset
 * of the tile counters in WORKSPACE mode) on `stream`. */
mtf_status mtf_einsum_exec(const mtf_plan_t* plan, const mtf_tensor* in, mtf_tensor* out,
                           const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes, void* stream);
/* One-shot form: plan (cached inside the layout handle by shapes, dtypes and epilogue stages) and
 * run.  `equation` is optional sugar, e.g. "batch io, io hidden -> batch hidden"; when given it
 * must agree with the descriptors' names (MTF_ERR_INVALID_ARG otherwise); NULL = names only. */
mtf_status mtf_einsum(const mtf_layout_t* layout, const char* equation, int32_t n_in, const mtf_tensor* in,
                      mtf_tensor* out, const mtf_epilogue* epilogue, void* workspace, size_t workspace_bytes,
                      void* stream);
mtf_status mtf_einsum_workspace_bytes(const mtf_layout_t* layout, int32_t n_in, const mtf_tensor* in,
                                      const mtf_tensor* out, const mtf_epilogue* epilogue, size_t* bytes);
/* mtf_einsum for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a property of the library, not of the method.)  Who needs it: code that runs where a device
 * allocation is not allowed or not possible - a host that hands the library tensors but owns the
 * allocator and will not lend it, a loop that must never trigger the implicit device-wide
 * synchronisation an allocation or a free can cause, a region that is being replayed and may not
 * create memory.  Such a caller has nowhere to get the `workspace` that mtf_einsum wants when the
 * planner realises the group sum through partial tiles (MTF_REDUCE_WORKSPACE).  This call takes no
 * workspace: the partial tiles and tile counters live in a fixed 32 MiB array inside the library
 * image, which every GPU that loads the library holds until the process exits.
 *   - Same arguments and results as mtf_einsum, minus the workspace.  The call itself allocates no
 *     device memory and calls no allocating routine; it launches one memset of the tile counters
 *     and one kernel on `stream`.
 *   - An einsum whose plan needs more than 32 MiB of scratch is refused with
 *     MTF_ERR_WORKSPACE_TOO_SMALL before anything is launched (use mtf_einsum and bring your own).
 *     Plans that need no scratch run exactly as through mtf_einsum.
 *   - The first call on each device looks up the array's device address (a one-time query of the
 *     runtime with that device current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left; the
 *     counters are zeroed on the stream before each launch and partial tiles are written before
 *     they are read, so calls that follow each other on one stream are fine.  Calls that may
 *     overlap on the GPU (different streams, different threads) race on it: serialise them. */
mtf_status mtf_einsum_builtin_scratch(const mtf_layout_t* layout, const char* equation, int32_t n_in,
                                      const mtf_tensor* in, mtf_tensor* out, const mtf_epilogue* epilogue,
                                      void* stream);
/* Testing hook: force the kernel family / reduce mode of plans created afterwards by this thread
 * (-1 = planner's choice; kernel_kind 2 = tensor cores with one CTA per tile, i.e. without the
 * two-CTA pairs the planner prefers on tall slices; kernel_kind 3 / 4 = tensor cores with the
 * 256 x 512 pair tiles wherever the shape allows them (pairs, plain epilogue, N slice a multiple of
 * 512) / never, instead of the launcher's count of waves; reduce_mode 3 = keep the planner's reduce mode
 * but, where the output tiles leave a partly filled last wave, give every worker an equal range of
 * (tile, k-block) units and assemble cut tiles from fragments in the workspace).  A forced choice
 * the shape cannot run gives MTF_ERR_UNSUPPORTED. */
mtf_status mtf_plan_force(int32_t kernel_kind, int32_t reduce_mode);
/* A promise about the next contraction this thread launches (mtf_einsum, mtf_einsum_exec): it reads nothing
 * that the launch before it on the same stream writes, and writes nothing that launch reads or writes.  A
 * tensor-core contraction then does not wait for that launch before it starts: its tiles begin on the SMs the
 * earlier launch's last round of tiles leaves idle, its workers take their tiles from a counter as they become
 * free, and it waits for the earlier launch before it ends, so whatever follows on the stream still sees both
 * complete.  Hinted launches that follow one another may all overlap each other and the launch before the first
 * of them, so the promise must hold against all of those; everything launched before that launch is complete
 * when they start.  The
 * promise is used up by the next contraction whether or not it can honour it (launches with a workspace
 * reduction or a fused reduce_sum, and the generic kernel, run in stream order as always; so does every
 * fourth hinted launch in a row).  The Transformer blocks use it between their own independent launches
 * (Algorithm 1 leaves the order of independent operations open).  Results do not depend on it. */
mtf_status mtf_hint_independent(void);

/* ---- feed-forward block (Section 8: y = Relu(x w + bias) v) ------------------------------------- */
/* x [*tokens, d_in], w [d_in, hidden], bias [hidden] or NULL, v [hidden, d_in]; outputs h_saved
 * [*tokens, hidden] (kept for the backward pass) and y [*tokens, d_in].  Two einsums; bias add and
 * relu are fused into the first. */
mtf_status mtf_ffn_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w,
                           const mtf_tensor* bias, const mtf_tensor* v, mtf_tensor* h_saved, mtf_tensor* y,
                           void* workspace, size_t workspace_bytes, void* stream);
/* Backward (Section 8.1: parameter gradients are einsums that reduce out the token dims; Section
 * 8.2: the gradient on x reduces out hidden):
 *   dhp = (dy . v^T) * [h_saved > 0];  dv = h^T . dy;  dw = x^T . dhp;  dbias = sum_tokens dhp;
 *   dx = dhp . w^T.   dbias may be NULL.  dhp lives in the workspace. */
mtf_status mtf_ffn_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w,
                            const mtf_tensor* v, const mtf_tensor* h_saved, const mtf_tensor* dy,
                            mtf_tensor* dx, mtf_tensor* dw, mtf_tensor* dbias, mtf_tensor* dv,
                            void* workspace, size_t workspace_bytes, void* stream);
/* Scratch bytes for the larger of forward and backward with these shapes. */
mtf_status mtf_ffn_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* w,
                                   size_t* bytes);

/* ---- softmax, layer normalisation, attention, decoder layer ------------------------------------------
 * Section 9 gives the layout of the Transformer (batch, heads, d_ff split; no tensor carries two of
 * them) and defers its mathematics to Vaswani et al.; the formulas below are that model's, written
 * as named-dim einsums (Section 6) plus the "Reduction" lowering for the row statistics.
 * Activations bf16; logits and their gradient f32 scratch; parameters of layer norm f32. */

/* weights = softmax over the LAST dimension of logits (f32 in, bf16 out, same dims).  causal != 0
 * excludes entries whose last index exceeds the second-to-last index (their weight is exactly 0). */
mtf_status mtf_softmax_forward(const mtf_layout_t* layout, const mtf_tensor* logits, int32_t causal,
                               mtf_tensor* weights, void* stream);
/* dlogits = weights * (dweights - sum over the last dim of dweights * weights); dweights f32. */
mtf_status mtf_softmax_backward(const mtf_layout_t* layout, const mtf_tensor* weights, const mtf_tensor* dweights,
                                mtf_tensor* dlogits, void* stream);
/* Einsum and softmax in one launch: weights = softmax over the LAST dimension of scale * einsum(a, b)
 * (the attention logits of Section 9's Transformer; bf16 operands, bf16 weights, device pointers).
 * The f32 logits stay in the tensor cores' accumulator memory and never reach HBM.  Only for
 * contractions whose whole output row fits one tile: the last output dimension is not split by the
 * layout and has at most 256 entries (512 when the second-to-last dimension has more than 128);
 * anything else, and any plan the tensor-core kernel cannot run, returns MTF_ERR_UNSUPPORTED and
 * leaves `weights` untouched (call mtf_einsum + mtf_softmax_forward instead).  causal as in
 * mtf_softmax_forward (the two last output dimensions are the query and memory positions).
 * workspace: unused today (pass what mtf_einsum would get); stream: CUDA stream or NULL. */
mtf_status mtf_einsum_softmax(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b, float scale,
                              int32_t causal, mtf_tensor* weights, void* workspace, size_t workspace_bytes, void* stream);
/* Its backward, also one launch: dlogits = weights * (dw - sum over the last dim of dw * weights)
 * with dw = einsum(a, b) (a = gradient of the attention output, b = values).  `weights` has the dims
 * of dlogits (bf16).  Same shape conditions, and in addition the two last output dimensions must be
 * multiples of 32 and 64 inside every slice; otherwise MTF_ERR_UNSUPPORTED. */
mtf_status mtf_einsum_softmax_backward(const mtf_layout_t* layout, const mtf_tensor* a, const mtf_tensor* b,
                                       const mtf_tensor* weights, mtf_tensor* dlogits, void* workspace,
                                       size_t workspace_bytes, void* stream);
/* y = gamma * (x - mean) * (var + eps)^-1/2 + beta over the LAST dimension (biased variance).
 * stats: f32 tensor with two values per row (mean, reciprocal standard deviation), kept for backward. */
mtf_status mtf_layernorm_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* gamma,
                                 const mtf_tensor* beta, float eps, mtf_tensor* y, mtf_tensor* stats, void* stream);
/* dx = rstd * (g - mean(g) - xh * mean(g * xh)) + residual, g = dy * gamma, xh = (x - mean) * rstd;
 * dgamma = sum over rows of dy * xh, dbeta = sum over rows of dy (both or neither; under a batch split
 * these sums are the gradient Allreduce of Algorithm 1).  residual may be NULL.
 * workspace (device, 16-byte aligned; may be NULL): with at least mtf_layernorm_workspace_bytes(row
 * length) bytes the two column sums are added up in a fixed order (per-block partial sums, then one
 * pass in block order) and repeat bit for bit from run to run; with less, or for row lengths that
 * report 0 bytes, they are accumulated with fp32 atomics into the zeroed outputs (order not fixed). */
mtf_status mtf_layernorm_backward(const mtf_layout_t* layout, const mtf_tensor* dy, const mtf_tensor* x, const mtf_tensor* stats, const mtf_tensor* gamma,
                                  const mtf_tensor* residual, mtf_tensor* dx, mtf_tensor* dgamma, mtf_tensor* dbeta, void* workspace,
                                  size_t workspace_bytes, void* stream);
mtf_status mtf_layernorm_workspace_bytes(int64_t row_length, size_t* bytes);

/* Multi-head attention.  x [batch, length, d_model]; wq, wk [d_model, heads, d_k]; wv [d_model, heads,
 * d_v]; wo [heads, d_v, d_model] (names are taken from the descriptors; the key/value side uses the
 * dimension name "memory_length" for a renamed copy of `length`).
 *   q[b,l,h,k] = sum_d x wq;  kk[b,m,h,k] = sum_d x wk;  vv[b,m,h,v] = sum_d x wv;
 *   logits[b,h,l,m] = d_k^-1/2 sum_k q kk;  weights = softmax over m (causal: m <= l);
 *   o[b,l,h,v] = sum_m weights vv;  y[b,l,d] = sum_{h,v} o wo  (+ residual, NULL or y's dims).
 * q, kk, vv, weights [batch, heads, length, memory_length], o are outputs kept for the backward pass. */
mtf_status mtf_attention_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq,
                                 const mtf_tensor* wk, const mtf_tensor* wv, const mtf_tensor* wo, int32_t causal,
                                 const mtf_tensor* residual, mtf_tensor* q, mtf_tensor* kk, mtf_tensor* vv,
                                 mtf_tensor* weights, mtf_tensor* o, mtf_tensor* y, void* workspace,
                                 size_t workspace_bytes, void* stream);
/* Gradients of the above for upstream dy [batch, length, d_model]: dwq, dwk, dwv, dwo (reduce out the
 * token dims) and dx (reduces out heads; dx_residual, NULL or dx's dims, is added).
 * causal: a hint, never needed for the result (causal weights hold exact zeros where m > l and those
 * zeros give zero gradients): non-zero promises that `weights` came from a causal forward call, and the
 * one-launch backward core then skips the key blocks that lie wholly right of the diagonal.  A non-zero
 * hint on weights that are not causal gives wrong gradients. */
mtf_status mtf_attention_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq,
                                  const mtf_tensor* wk, const mtf_tensor* wv, const mtf_tensor* wo, int32_t causal,
                                  const mtf_tensor* q,
                                  const mtf_tensor* kk, const mtf_tensor* vv, const mtf_tensor* weights,
                                  const mtf_tensor* o, const mtf_tensor* dy, const mtf_tensor* dx_residual,
                                  mtf_tensor* dx, mtf_tensor* dwq, mtf_tensor* dwk, mtf_tensor* dwv, mtf_tensor* dwo,
                                  void* workspace, size_t workspace_bytes, void* stream);
mtf_status mtf_attention_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_tensor* wq,
                                         const mtf_tensor* wv, size_t* bytes);

/* Decoder layer (post-layer-norm residual blocks):  a = LN1(x + Attention(x));  out = LN2(a + FFN(a)). */
typedef struct {
  const mtf_tensor *wq, *wk, *wv, *wo, *ln1_gamma, *ln1_beta, *w, *bias /* may be NULL */, *v, *ln2_gamma, *ln2_beta;
} mtf_decoder_params;
/* Caller-allocated activations the forward pass fills and the backward pass reads:
 * q, kk, vv, weights, o as in attention; s1 = x + Attention(x); stats1; a; h [*, d_ff]; s2 = a + FFN(a); stats2. */
typedef struct {
  mtf_tensor *q, *kk, *vv, *weights, *o, *s1, *stats1, *a, *h, *s2, *stats2;
} mtf_decoder_saved;
typedef struct {
  mtf_tensor *dwq, *dwk, *dwv, *dwo, *dln1_gamma, *dln1_beta, *dw, *dbias /* may be NULL */, *dv, *dln2_gamma, *dln2_beta;
} mtf_decoder_grads;
mtf_status mtf_decoder_layer_forward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_decoder_params* params,
                                     int32_t causal, float eps, const mtf_decoder_saved* saved, mtf_tensor* out,
                                     void* workspace, size_t workspace_bytes, void* stream);
/* (causal: the hint of mtf_attention_backward; pass what the forward call was given, or 0) */
mtf_status mtf_decoder_layer_backward(const mtf_layout_t* layout, const mtf_tensor* x, const mtf_decoder_params* params,
                                      int32_t causal, const mtf_decoder_saved* saved, const mtf_tensor* dout, mtf_tensor* dx,
                                      const mtf_decoder_grads* grads, void* workspace, size_t workspace_bytes, void* stream);
mtf_status mtf_decoder_layer_workspace_bytes(const mtf_layout_t* layout, const mtf_tensor* x,
                                             const mtf_decoder_params* params, size_t* bytes);

/* ---- parameter update (Section 3, Algorithm 1 line 3: W(t+1) = Update(W(t), gradient)) -----------
 * The paper leaves Update open.  This library's reading: stochastic gradient descent with optional
 * momentum and decoupled weight decay on an f32 master copy, refreshing the bf16 working copy the
 * contractions read, all in one memory-bound pass:
 *     m <- momentum * m + g  (momentum tensor NULL: m = g);  W <- W - lr * (m + weight_decay * W);  Wb <- bf16(W)
 * grad f32 or bf16; master f32 (updated in place); momentum f32 or NULL (updated in place; must be
 * given when hp->momentum != 0); param bf16 or NULL.  All tensors have master's dims, are 16-byte
 * aligned, device memory.  The update is component-wise (Section 6), hence local under every layout:
 * each processor updates its own slice, which on one GPU is one pass over the stored tensor.  Under
 * a rank-bound layout every rank updates its box after the gradients were summed across ranks. */
typedef struct { float lr, momentum, weight_decay; } mtf_update_params;
mtf_status mtf_update(const mtf_layout_t* layout, const mtf_tensor* grad, mtf_tensor* master, mtf_tensor* momentum, mtf_tensor* param,
                      const mtf_update_params* hp, void* stream);

/* ---- reshape and storage order (Section 6.1 "Reshape") ------------------------------------------------
 * A reshape that keeps the sizes and changes dimension names changes the layout.  Per mesh dimension
 * the paper names the communication it needs: a tensor dimension split over it before but none after
 * = Allgather; none before, one after = local slicing; different tensor dimensions before and after
 * = Alltoall.  On one GPU a tensor is stored once and slices are views, so such a reshape is a change
 * of descriptor and moves no data; mtf_reshape_plan reports, for mesh dimension j, pattern[j] and the
 * number of elements one processor would receive (host arrays of the mesh's ndim; all gathers are
 * counted before any slicing, ascending mesh dimension).  Errors as mtf_layout_check_tensor, for the
 * input and for the output dims. */
typedef enum { MTF_RESHAPE_NONE = 0, MTF_RESHAPE_ALLGATHER = 1, MTF_RESHAPE_SLICE = 2, MTF_RESHAPE_ALLTOALL = 3 } mtf_reshape_pattern;
mtf_status mtf_reshape_plan(const mtf_layout_t* layout, int32_t ndim, const mtf_dim* in_dims, const char* const* out_names, int32_t* pattern,
                            int64_t* received_per_proc);
/* What does move data on one GPU: a change of storage order.  out's dims are a permutation (by name)
 * of in's; same dtype; device pointers; one launch, bound by HBM (each element read once, written
 * once).  E.g. [batch, length, heads, d_k] -> [batch, heads, length, d_k], the block transpose an
 * Alltoall between a batch split and a heads split performs. */
mtf_status mtf_transpose(const mtf_layout_t* layout, const mtf_tensor* in, mtf_tensor* out, void* stream);
/* Inverse of mtf_slice_gather: the dense row-major slice of `processor` (device, global's dtype) is
 * written into its box of `global`.  (What an Allgather does with every processor's slice.) */
mtf_status mtf_slice_scatter(const mtf_layout_t* layout, const void* slice, int64_t processor, mtf_tensor* global, void* stream);
/* Layout search (Section 11 names it as future work; the cost model is Table 1's): over every
 * assignment of the n_names candidate tensor dimensions to a mesh dimension or to none, legal for all
 * n_einsums einsums in0[e] . in1[e] -> out[e] (descriptors; data ignored), minimise
 *     sum_e  multiply-adds per processor + comm_weight * values entering an Allreduce per processor,
 * ties going to the smaller sum of slice elements, then to the first assignment in enumeration order
 * (first name slowest; unsplit, then mesh dimension 0, 1, ...).  chosen_mesh_dim[i] = index of the
 * mesh dimension names[i] is split over, or -1.  MTF_ERR_ILLEGAL_LAYOUT when nothing is legal. Host only. */
mtf_status mtf_layout_search(const mtf_mesh_t* mesh, int32_t n_einsums, const mtf_tensor* in0, const mtf_tensor* in1, const mtf_tensor* out,
                             int32_t n_names, const char* const* names, double comm_weight, int32_t* chosen_mesh_dim, double* cost,
                             int64_t* footprint);

/* ---- the vocab dimension (Section 9: vocab, d_ff and heads are the split dimensions) ------------------
 * Token ids and targets are device arrays of int32, one per token, values in [0, vocab); a value
 * outside is skipped (zero row / zero loss) and reported by mtf_device_status as MTF_ERR_INVALID_ARG.
 *   mtf_embedding_forward : x[t, :] = table[ids[t], :]   - the einsum onehot(ids) . table, which reduces
 *       `vocab`; under a vocab split exactly one slice holds the row, and the table being stored once,
 *       the group sum is a row lookup.  table [vocab, d], x [*tokens, d], same dtype (bf16 or f32).
 *   mtf_embedding_backward: dtable[v, :] = sum over tokens with ids[t] = v of dx[t, :]  (f32, zeroed by
 *       the call, fp32 atomics: order not fixed); summed across ranks when a token dim is split over them.
 *   mtf_xent_forward      : logits[t, v] = sum_d h[t, d] wout[d, v] (bf16, through mtf_einsum under the
 *       layout); per token lse = log sum_v exp(logits) - taken over the logits as stored, maximum
 *       subtracted, the local reduction of every part of a row and the combine over the parts
 *       (Section 6 "Reduction") - and loss = lse - logits[t, target[t]].  lse, loss: f32, one per token.
 *       With a 256-byte aligned workspace of at least tokens * 16 * ceil(vocab / 256) bytes per vocab
 *       slice layout (tokens x column parts x 8 bytes) the contraction takes the local reductions in its
 *       own epilogue and the logits are not read back; otherwise a second pass over the logits does both.
 *   mtf_xent_backward     : dlogits = (exp(logits - lse) - onehot(target)) * dloss[t], written over
 *       `logits`; dh = dlogits . wout^T (reduces vocab: the group sum of a vocab split);
 *       dwout = h^T . dlogits (reduces the token dims).  dloss f32, one per token.
 * A vocab dimension split across RANKS is refused (MTF_ERR_UNSUPPORTED): the row statistics would need
 * a max / sum combine across ranks.  workspace: as for mtf_einsum (plus the above for mtf_xent_forward). */
mtf_status mtf_embedding_forward(const mtf_layout_t* layout, const int32_t* ids, const mtf_tensor* table, mtf_tensor* x, void* stream);
mtf_status mtf_embedding_backward(const mtf_layout_t* layout, const int32_t* ids, const mtf_tensor* dx, mtf_tensor* dtable, void* stream);
mtf_status mtf_xent_forward(const mtf_layout_t* layout, const mtf_tensor* h, const mtf_tensor* wout, const int32_t* targets, mtf_tensor* logits,
                            mtf_tensor* lse, mtf_tensor* loss, void* workspace, size_t workspace_bytes, void* stream);
/* The row parts of the two calls around this comment on their own, on logits that are already stored
 * (bf16 [*tokens, vocab], vocab a multiple of 8): lse and loss per token; dlogits written over the logits. */
mtf_status mtf_softmax_xent_forward(const mtf_layout_t* layout, const mtf_tensor* logits, const int32_t* targets, mtf_tensor* lse, mtf_tensor* loss,
                                    void* stream);
mtf_status mtf_softmax_xent_backward(const mtf_layout_t* layout, mtf_tensor* logits, const int32_t* targets, const mtf_tensor* lse,
                                     const mtf_tensor* dloss, void* stream);
mtf_status mtf_xent_backward(const mtf_layout_t* layout, const mtf_tensor* h, const mtf_tensor* wout, const int32_t* targets, mtf_tensor* logits,
                             const mtf_tensor* lse, const mtf_tensor* dloss, mtf_tensor* dh, mtf_tensor* dwout, void* workspace, size_t workspace_bytes,
                             void* stream);

/* ---- reductions (Section 6 "Reduction") --------------------------------------------------------- */
/* out[out dims] = sum over the other dims of in (out dims a subset of in's).  Local reduction per
 * slice, then the group sum across the mesh dims of reduced-out split dims, in one launch. */
mtf_status mtf_reduce_sum(const mtf_layout_t* layout, const mtf_tensor* in, mtf_tensor* out, void* stream);

/* ---- stage tap (verification aid) ----------------------------------------------------------------
 * The block calls keep some results of their einsums only in scratch memory (the feed-forward
 * block's dhp; the attention block's do, dlogits, dq, dkk, dvv; the decoder layer's gradient streams
 * ds2, da, ds1), and reuse that scratch.  While a tap is open on the calling thread, every block call
 * of that thread copies each such intermediate, right behind the launch that produced it and on the
 * same stream, into `device_buffer` (device memory, 256-byte aligned, caller-owned), one after the
 * other at 256-byte aligned offsets.  A checker can then hold every launch of a block to the
 * single-einsum tolerance: the inputs the launch read and the output it wrote are all available.
 *   mtf_stage_tap_begin : opens the tap (forgets the previous one's entries).
 *   mtf_stage_tap_end   : closes it, returns the number of entries; MTF_ERR_WORKSPACE_TOO_SMALL when
 *                         the buffer was too small (entries that did not fit were not copied).
 *   mtf_stage_tap_entry : name (valid until the next begin on this thread), byte offset and size of
 *                         entry `index`, in the order the intermediates were produced.
 * With no tap open the block calls do no extra work.  (The paper has no counterpart.) */
mtf_status mtf_stage_tap_begin(void* device_buffer, size_t bytes);
mtf_status mtf_stage_tap_end(int32_t* n_entries);
mtf_status mtf_stage_tap_entry(int32_t index, const char** name, size_t* offset, size_t* bytes);

/* ---- status ------------------------------------------------------------------------------------- */
const char* mtf_status_string(mtf_status s);
const char* mtf_last_error(void);
/* Synchronises the current device and reads the sticky device status word: 0 = no kernel of this
 * library gave up on a bounded wait since the last call; non-zero = a code naming the wait.
 * Resets the word.  Returns MTF_ERR_TIMEOUT when it was non-zero, else MTF_ERR_INVALID_ARG when a
 * token id or target outside [0, vocab) was seen by the vocab kernels since the last call. */
mtf_status mtf_device_status(int32_t* code);
/* Testing hook for the failure path of the bounded device-side waits.  limit_cycles > 0 sets how many SM
 * cycles a wait may take before it gives up (<= 0 restores the default of about two seconds);
 * withhold_one_signal != 0 makes every tensor-core launch leave out the "accumulator complete" signal
 * of its first tile, so that the wait for it runs out: the kernel records a code, all its roles
 * leave through the common teardown (copies and MMAs in flight are given time to land, tensor memory
 * is freed), the launch ends normally, its output is unspecified, and the next mtf_device_status
 * returns MTF_ERR_TIMEOUT.  Nothing traps or faults and the context stays usable.  Affects the current
 * device until changed back; not for production use. */
mtf_status mtf_debug_wait_test(int64_t limit_cycles, int32_t withhold_one_signal);
/* Number of kernels this library has launched from this process (all threads). */
int64_t mtf_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* MTF_H_ */
