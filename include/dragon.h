/*
 * dragon.h -- C ABI of the B200 graph virtual machine (libdragon.so).
 *
 * The library evaluates a compiled function  f = function(inputs, outputs)  (Sec. 2.1 of
 * "Dragon: A Computation Graph Virtual Machine Based Deep Learning Framework",
 * arXiv 1707.08265) over large tensors on one GPU: the forward pass and the generated
 * gradient pass of a tensor-as-node DAG, after the forward prune (Sec. 2.2, Algorithm 1)
 * and the backward prune (Sec. 2.3, Algorithm 2).
 *
 * Conventions that hold for every entry point
 *   - Tensor ids and operator ids are dense non-negative ints in creation order; this is
 *     the "creating order" of Sec. 3.2.  A negative return value is an error code.
 *   - All host pointers are read during the call only; nothing is retained.
 *   - All device memory (feeds, fetches, workspace) belongs to the caller.  The library
 *     allocates device memory only for its own immutable instruction streams, on the first
 *     dragon_run() of a function, and frees it in dragon_function_destroy().
 *   - Tensors are row-major and contiguous, rank 0..2.  Device pointers must be 16-byte
 *     aligned.
 *   - Every entry point returns an error code (or NULL) instead of launching on bad
 *     arguments; dragon_last_error() gives the message.  No call synchronises the device
 *     except dragon_function_status().
 */
#ifndef DRAGON_H_
#define DRAGON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dragon_graph dragon_graph_t;       /* host-only graph under construction   */
typedef struct dragon_function dragon_function_t; /* pruned + compiled function           */
typedef struct dragon_workspace dragon_workspace_t; /* named tensors in device memory (Sec. 3.1) */
typedef int32_t dragon_id;

enum {
  DRAGON_OK = 0,
  DRAGON_ERR_INVALID_ARG = -1,
  DRAGON_ERR_SHAPE = -2,         /* declared output shape differs from the inferred one, or operands do not broadcast */
  DRAGON_ERR_DTYPE = -3,
  DRAGON_ERR_NOT_SSA = -4,       /* output already has a producer, or an operator reads its own output */
  DRAGON_ERR_MISSING_INPUT = -5, /* a marked source tensor is not among the function's inputs */
  DRAGON_ERR_NO_PATH = -6,       /* gradient requested but no chain objective -> derivative target */
  DRAGON_ERR_UNSUPPORTED = -7,
  DRAGON_ERR_WORKSPACE = -8,     /* workspace missing, misaligned or too small */
  DRAGON_ERR_CUDA = -9,
  DRAGON_ERR_TIMEOUT = -10       /* a bounded device-side wait ran out (reported by dragon_function_status) */
};

enum { DRAGON_F32 = 0, DRAGON_BF16 = 1, DRAGON_I32 = 2 };

/* Operator types.  The paper names Sigmoid, Tanh, ReLU (Sec. 2.4) and uses mul, add, sin in
 * its example (Sec. 2.2); the remaining semantics are this library's:
 *   ADD, SUB, MUL          a+b, a-b, a*b with right-aligned broadcasting among [], [C], [R,C]
 *   DIV                    a / (1 + |b|)
 *   EXP                    exp(min(max(x, -10), 10))
 *   SQRT, RECIPROCAL       sqrt(x), 1/x (the RMSProp and Adam updaters of Sec. 3.2 divide by a root);
 *                          approximate instructions of at most one unit in the last place, arguments
 *                          below 2^-126 in magnitude count as zero
 *   SUM, MEAN              over the last axis, result broadcast back to the operand's shape
 *   INNER_PRODUCT(X, W)    Y[m,n] = sum_k X[m,k] * W[n,k]; operands are consumed as bf16,
 *                          accumulation is fp32
 *   BIAS_ADD(Y, b)         Y[m,n] + b[n]
 *   SOFTMAX_CROSS_ENTROPY(Z, labels)  scalar -(1/M) sum_m log softmax(Z[m,:])[labels[m]],
 *                          labels int32 in [0, N); an out-of-range label contributes 0 and
 *                          sets the function status to DRAGON_ERR_INVALID_ARG (no fault)
 *   OPAQUE                 an operator the library knows only as an edge set: any number of inputs
 *                          and of outputs (Sec. 2.2: an edge from every input to every output), output
 *                          shapes as declared.  Both prunes treat it like any other operator; a
 *                          function that keeps one compiles (marks, kept operators and masks can
 *                          be read) but cannot run: dragon_run returns DRAGON_ERR_UNSUPPORTED.
 */
enum {
  DRAGON_OP_ADD = 0, DRAGON_OP_SUB = 1, DRAGON_OP_MUL = 2, DRAGON_OP_DIV = 3,
  DRAGON_OP_SIN = 4, DRAGON_OP_EXP = 5, DRAGON_OP_TANH = 6, DRAGON_OP_SIGMOID = 7,
  DRAGON_OP_RELU = 8, DRAGON_OP_SUM = 9, DRAGON_OP_MEAN = 10,
  DRAGON_OP_INNER_PRODUCT = 11, DRAGON_OP_BIAS_ADD = 12, DRAGON_OP_SOFTMAX_CROSS_ENTROPY = 13,
  DRAGON_OP_SQRT = 14, DRAGON_OP_RECIPROCAL = 15, DRAGON_OP_OPAQUE = 16,
  DRAGON_OP_COUNT_ = 17
};

/* ---- graph capture (Sec. 2.1: tensors are nodes; an operator connects each of its inputs
 *      to each of its outputs, Sec. 2.2) -------------------------------------------------- */

dragon_graph_t* dragon_graph_create(void);
void dragon_graph_destroy(dragon_graph_t* g); /* NULL is allowed */

/* Declares a tensor.  name: unique, NUL-terminated (Sec. 3.1: each tensor has a unique name).
 * rank 0..2, shape[rank] > 0 (host pointer, may be NULL for rank 0).  Returns the new id. */
dragon_id dragon_add_tensor(dragon_graph_t* g, const char* name, int dtype, int rank, const int64_t* shape);

/* Appends an operator.  in/out: host arrays of tensor ids declared earlier.  Every output must
 * have no producer yet, must not be among the inputs and must not have been read already; its
 * declared shape must equal the inferred one (Sec. 4.3: a mistaken shape is caught before
 * executing).  Every executable operator type has exactly one output; DRAGON_OP_OPAQUE takes
 * n_out >= 1.  attrs is reserved (pass NULL, 0).  Returns the operator id. */
dragon_id dragon_add_op(dragon_graph_t* g, int op_type, const dragon_id* in, int n_in,
                        const dragon_id* out, int n_out, const double* attrs, int n_attrs);

/* theano.tensor.grad analogue (Sec. 4.1): attaches one gradient stage for the derivative pairs
 * objs x wrts (Sec. 2.3).  The stage computes the gradient of the sum of all elements of all
 * objs.  For each wrts[j] a new f32 tensor of the same shape is declared and its id written to
 * out_grad_tensor_ids[j] (host array of n_wrt ids).  DRAGON_ERR_NO_PATH if some wrts[j] has no
 * chain to any objective.  Gradient tensors can be fetched but not consumed by operators. */
int dragon_add_grad(dragon_graph_t* g, const dragon_id* objs, int n_obj, const dragon_id* wrts, int n_wrt,
                    dragon_id* out_grad_tensor_ids);

int dragon_graph_num_tensors(const dragon_graph_t* g);
int dragon_graph_num_ops(const dragon_graph_t* g);

/* ---- compile: prune + instruction streams (Sec. 2.2, 2.3, 3.2) -------------------------- */

/* Builds f = function(inputs, outputs).  An input that the targets do not need is legal, is
 * reported as pruned, and its feed pointer is never read (the redundant b of Sec. 2.2).  An input
 * may also be a tensor that an operator produces (Sec. 3.1: any tensor can be fed): in this
 * function it is given, the operator that would have produced it is not its parent, both prunes
 * run on the graph without the edges into it, and a chain objective -> derivative target counts
 * only if it avoids those edges; fetching a gradient whose derivative target has no chain left
 * fails with DRAGON_ERR_NO_PATH.  Gradient tensors cannot be fed.  Works without a GPU.  The
 * graph is not changed and may be destroyed afterwards.  Returns NULL on error. */
dragon_function_t* dragon_function(dragon_graph_t* g, const dragon_id* inputs, int n_in,
                                   const dragon_id* outputs, int n_out);
void dragon_function_destroy(dragon_function_t* f); /* NULL is allowed */

/* Marked flags M of Algorithm 1 run over the two-stage DAG from the fetched targets: one byte
 * per tensor id (n_tensors must equal the graph's tensor count at compile time). */
int dragon_function_marked(const dragon_function_t* f, uint8_t* flag_per_tensor, int n_tensors);

/* Kept operators.  fwd_ops: kept forward operator ids in creation order.  grad_ops: for every
 * kept gradient operator the id of its forward operator, stage by stage, inverse creation
 * order inside a stage (Sec. 3.2); grad_input_mask (may be NULL): bit p set iff the gradient
 * with respect to operand position p is produced (first occurrence of a repeated operand).
 * The counts are always written; the arrays are filled up to their capacities. */
int dragon_function_kept_ops(const dragon_function_t* f, dragon_id* fwd_ops, int cap_f, int* n_f,
                             dragon_id* grad_ops, uint32_t* grad_input_mask, int cap_g, int* n_g);

/* In-place structures of the pruned graph (Sec. 2.4, Algorithm 3): ancestor[t] is the tensor whose
 * memory tensor t may share - the first node, in creation order, of the path of nodes with exactly
 * one child that leads to t (t itself when it starts a path), or -1 if t is not marked.  Marked
 * tensors and kept forward operators take part (the paper renames after the prunes). */
int dragon_function_rename_dictionary(const dragon_function_t* f, dragon_id* ancestor, int n_tensors);

/* The tensors that cross kernels inside the caller's workspace, after memory sharing: up to cap
 * quintuples {byte offset, bytes, first plan step that touches it, last one, 1 if it was placed over an
 * input of its producing step (in place)}.  Returns their number.  Two tensors whose step ranges
 * overlap never share bytes, except an in-place output and the input it replaces. */
int dragon_function_workspace_tensors(const dragon_function_t* f, int64_t* out, int cap);

/* In-place use.  The updater graphs of Sec. 3.2 overwrite their state (W, momentum, second moment), and
 * Sec. 2.4 is about operators that write over their input.  Returns 1 if fetch position `output` may be
 * given the very same device pointer as feed position `input` in dragon_run(), 0 if not, a negative
 * code for bad positions.  It is 1 exactly when the function is a single elementwise launch over a
 * flat domain, both tensors have the domain's shape and the same type, and the program reads the
 * input for the last time before it first writes the output: every thread then overwrites only
 * elements it has already read (the copy of a tile that is fetched ahead of time is never a tile that
 * has been written).  The state of an update then stays in the caller's device memory from step to
 * step.  Any other overlap between feeds and fetches is undefined. */
int dragon_function_can_alias(const dragon_function_t* f, int input, int output);

/* One byte per listed input: 1 if the pruned function reads it. */
int dragon_function_used_inputs(const dragon_function_t* f, uint8_t* flag_per_input, int n_in);

/* Number of kernel launches one dragon_run() issues, and a short human-readable plan
 * (NUL-terminated, truncated to cap). */
int dragon_function_num_launches(const dragon_function_t* f);
int dragon_function_describe(const dragon_function_t* f, char* buf, int cap);

/* Introspection of one graph-VM step of the plan (step index = line of dragon_function_describe),
 * for tools and tests that check the emitted instruction stream without a GPU.  info[0..9] =
 * {number of code words, row mode (0/1), cols, number of operands, spill slots, shared-memory
 * slots, rows or elements (low 32 bits), rows or elements (high 32 bits), number of reduced
 * outputs, register slots of the kernel build the program is for (3 dense, 7 wide)}; code (may be NULL)
 * receives up to cap_code words (encoding: csrc/vm_isa.h); operands (may be NULL) receives up to
 * cap_operands quadruples {where (0 feed, 1 fetch, 2 workspace), position or workspace offset / 256,
 * kind (0 full, 1 row, 2 scalar), dtype}; reduced (may be NULL) receives up to cap_reduced triples
 * {0 column sums / 1 scalar sum, accumulator index, fetch position (or -1 for a workspace tensor)}.
 * Returns DRAGON_ERR_INVALID_ARG if the step is not a graph-VM step. */
int dragon_function_vm_step(const dragon_function_t* f, int step, int64_t* info, uint32_t* code, int cap_code,
                            int64_t* operands, int cap_operands, int64_t* reduced, int cap_reduced);

/* Execution tier of the graph-VM programs of f.  By default (mode 1) every program is turned, at the
 * function's first run, into a kernel of its own: the leaves of its instructions in program order as
 * straight-line PTX with every decoded field a constant, assembled by the driver (a fraction of a second
 * per program).  It computes what the interpreter computes, bit for bit (every leaf uses explicitly
 * rounded operations), without fetch, decode and dispatch.  The paper has one kernel per operator
 * (Sec. 3.3); this is the other end: one kernel per pruned function segment.  mode 0 holds f to the
 * interpreter kernel; mode 2 specialises now and returns the number of programs specialised, or
 * DRAGON_ERR_CUDA (with the assembler's message in dragon_last_error()) if that is not possible.  In
 * mode 1 a program whose kernel cannot be made stays interpreted and dragon_function_describe() says so.
 * dragon_function_num_specialized(): programs of f that currently run as specialised kernels.  The
 * environment variable DRAGON_VM_TIER=0 makes mode 0 the default of functions created afterwards. */
int dragon_function_specialize(dragon_function_t* f, int mode);
int dragon_function_num_specialized(const dragon_function_t* f);

/* The PTX text of the specialised kernel of a graph-VM step (step index as for dragon_function_vm_step),
 * for tools and tests; works without a GPU.  Copies up to cap - 1 characters and a NUL into buf (buf may be
 * NULL if cap is 0) and returns the full length, or a negative code. */
int dragon_function_vm_ptx(const dragon_function_t* f, int step, char* buf, int cap);

/* Static check of a graph-VM instruction stream (encoding: csrc/vm_isa.h): every case id exists in the
 * kernel build with register_slots slots (3 or 7), every register slot, shared-memory slot, uniform,
 * memory operand, spill slot and accumulator an instruction names lies inside the given limits, row sums
 * occur only in row programs, and the stream is loop_begin ... body from loop_start ... one loop end ...
 * end.  A program is immutable once compiled, so this check on the host stands for a range check in every
 * leaf of the kernel; the compiler runs it on each program it emits (a failure there is
 * DRAGON_ERR_UNSUPPORTED at dragon_function) and this entry point exposes it to tools and tests.
 * code: host array of n_code words.  Returns DRAGON_OK or DRAGON_ERR_INVALID_ARG (dragon_last_error()
 * names the word and the index).  The paper has no counterpart: its operators are separate kernels. */
int dragon_verify_vm_program(const uint32_t* code, int n_code, int loop_start, int register_slots, int n_operands,
                             int n_smem_slots, int n_spill_slots, int n_column_accs, int n_scalar_accs, int row_mode);

/* Scratch memory (partial sums, tensors that cross kernels, spilled values, a status word).
 * dev_ptr: device memory, 256-byte aligned, at least dragon_function_workspace_bytes() long,
 * owned by the caller and not touched by anyone else while a run is in flight. */
size_t dragon_function_workspace_bytes(const dragon_function_t* f);
int dragon_function_set_workspace(dragon_function_t* f, void* dev_ptr, size_t bytes);

/* ---- run (Sec. 2.1: push inputs, get outputs) ------------------------------------------ */

/* feeds: host array of n_in device pointers in the order of inputs (entries of pruned inputs
 * may be NULL); fetches: host array of n_out device pointers; cuda_stream: a cudaStream_t.
 * Asynchronous; launches nothing on error.  Each needed input is read and each fetched output
 * written by the kernels of the plan; a fetch that is itself an input is copied. */
int dragon_run(dragon_function_t* f, const void* const* feeds, void* const* fetches, void* cuda_stream);

/* The same with HOST buffers: copies every needed input from host_feeds[j] to the staging area,
 * runs, and copies every fetched output to host_fetches[j], all asynchronously on cuda_stream
 * (the caller synchronises the stream before reading the results; pinned host memory makes the
 * copies truly asynchronous).  staging_dev: caller-owned device memory, 256-byte aligned, at
 * least dragon_function_staging_bytes() long.  Entries of pruned inputs may be NULL.
 * A function that is a single elementwise launch over a large flat domain is run in chunks of
 * the element range, with the copies of neighbouring chunks on two streams of the function's own
 * so that copy-in, kernel and copy-out overlap; cuda_stream still orders the call as a whole (it
 * waits for the last copy-out), so the caller sees the same behaviour. */
size_t dragon_function_staging_bytes(const dragon_function_t* f);
int dragon_run_host(dragon_function_t* f, const void* const* host_feeds, void* const* host_fetches,
                    void* staging_dev, size_t staging_bytes, void* cuda_stream);

/* ---- workspace (Sec. 3.1: the workspace owns every tensor; any of them can be fed or fetched by
 *      name; Sec. 3.2: the state of an updater lives there between runs) ------------------------ */

/* A workspace owns device memory for named tensors and for the scratch areas of the functions run
 * against it.  It is used from one host thread and with one stream at a time; destroying it frees
 * everything it allocated (no run that uses it may still be in flight). */
dragon_workspace_t* dragon_workspace_create(void);
void dragon_workspace_destroy(dragon_workspace_t* w); /* NULL is allowed */

/* Feed by name.  The first feed of a name creates the tensor (type, rank 0..2 and shape as given,
 * contents zero); later feeds must repeat type and shape (DRAGON_ERR_DTYPE / DRAGON_ERR_SHAPE).
 * src: host or device memory holding the tensor contiguously, or NULL to create without copying;
 * the copy is asynchronous on cuda_stream (pageable host memory makes it synchronous). */
int dragon_workspace_feed(dragon_workspace_t* w, const char* name, int dtype, int rank, const int64_t* shape,
                          const void* src, void* cuda_stream);

/* Fetch by name: copies the tensor's bytes to dst (host or device memory, caller-owned) asynchronously
 * on cuda_stream.  bytes must equal the tensor's size.  DRAGON_ERR_MISSING_INPUT for an unknown name. */
int dragon_workspace_fetch(dragon_workspace_t* w, const char* name, void* dst, size_t bytes, void* cuda_stream);

/* Device address of a named tensor as of now (a later run that rebinds the name may change it), with its
 * type, rank and shape (each may be NULL; shape receives rank extents).  NULL for an unknown name. */
void* dragon_workspace_tensor(dragon_workspace_t* w, const char* name, int* dtype, int* rank, int64_t* shape);

/* Bytes of device memory the workspace holds. */
size_t dragon_workspace_bytes(const dragon_workspace_t* w);

/* Runs f against the workspace: every input that the pruned function reads is the workspace tensor with
 * the input's graph name (DRAGON_ERR_MISSING_INPUT if it was never fed, DRAGON_ERR_DTYPE /
 * DRAGON_ERR_SHAPE if it does not fit: Sec. 4.3, a mistaken shape is caught before executing); output j
 * is written to the tensor named output_names[j], or, where output_names or its entry is NULL, to the one
 * named like the output in the graph; missing tensors are created.  An output may be bound to the name
 * of an input (W' -> W in the updater of Sec. 3.2): it overwrites the input in place where
 * dragon_function_can_alias() allows, otherwise it is written to a second buffer that the name points
 * to once the run is enqueued (the old buffer is kept for the next such run), so a later run or fetch on
 * the same stream sees the new contents.  If f has no scratch area yet, the workspace allocates one.
 * Asynchronous on cuda_stream; errors as for dragon_run(). */
int dragon_workspace_run(dragon_workspace_t* w, dragon_function_t* f, const char* const* output_names,
                         void* cuda_stream);

/* Device-side timing of one launch step of the plan (step index as listed by
 * dragon_function_describe, one line per step; for a graph-VM step the VM kernel alone is
 * bracketed, not its finishing reduction).  dragon_function_profile() arms a ring of
 * `capacity` CUDA event pairs recorded around that step by every following dragon_run()
 * (step < 0 disarms); dragon_function_profile_read() synchronises the recorded events and
 * returns the summed kernel time and the number of runs since arming, then re-arms. */
int dragon_function_profile(dragon_function_t* f, int step, int capacity);
int dragon_function_profile_read(dragon_function_t* f, double* total_ms, int* runs);

/* Synchronises the stream of the last run and returns the device status word of that run: DRAGON_OK,
 * DRAGON_ERR_TIMEOUT (a bounded wait gave up) or DRAGON_ERR_INVALID_ARG (bad label). */
int dragon_function_status(dragon_function_t* f);

/* Mean softmax cross-entropy loss without any allocation.  The paper has no counterpart: this is
 * a convenience of this library for callers that cannot give it a workspace.
 *
 * Who needs it: code that runs where device memory cannot be requested -- a plug-in inside a host
 * application whose own pool already owns the whole GPU (a cudaMalloc from the plug-in would fail,
 * or take memory the pool counts on), or a latency-bound loop that cannot afford the device-wide
 * synchronisation an allocation or a free may imply.  Such a caller cannot use dragon_run(), which
 * wants a caller-provided workspace and uploads instruction streams on first use.
 *
 * Computes  loss_out[0] = -(1/rows) * sum_m log softmax(logits[m,:])[labels[m]]  exactly like the
 * SOFTMAX_CROSS_ENTROPY operator (same kernels).  logits: device, row-major [rows, cols], dtype
 * DRAGON_F32 or DRAGON_BF16; labels: device int32[rows]; loss_out: device float[1]; all owned by
 * the caller.  The per-row partial losses live in a fixed array inside the library image
 * (257 KiB per GPU, held from library load to process exit), which limits rows to 65536:
 * larger inputs are rejected with DRAGON_ERR_WORKSPACE.  The call allocates and frees nothing
 * and is asynchronous on cuda_stream.
 *
 * The first call on each device looks up the array's device address (a one-time set-up under
 * the current device); make that first call outside any stream capture.  All calls on a device
 * share the one array: it keeps the previous call's contents (the function clears what has to
 * start at zero), and two calls that overlap on the GPU -- different streams, no ordering --
 * race on it and give wrong results.  An out-of-range label contributes 0 to the sum as in the
 * operator, but is not reported: this entry point has no function whose status could be read, so
 * validate labels beforehand if they can be wrong.  logits must be 16-byte aligned, labels and
 * loss_out 4-byte aligned (DRAGON_ERR_INVALID_ARG otherwise).  The array's address is looked up
 * once per device and kept; after a cudaDeviceReset() in the same process it is stale and this
 * entry point must not be used any more. */
int dragon_softmax_ce_loss_static(const void* logits, int dtype, const int32_t* labels, int rows, int cols,
                                  float* loss_out, void* cuda_stream);

/* Host instantiation of the VM's elementary functions (fn: DRAGON_OP_SIN, _EXP, _TANH,
 * _SIGMOID, _SQRT, _RECIPROCAL; DRAGON_OP_DIV evaluates 1/(1+|x|); 100 + DRAGON_OP_SIN evaluates the cosine),
 * for accuracy sweeps on machines without a GPU.  x, y: host arrays of n floats. */
int dragon_host_math(int fn, const float* x, float* y, int n);

/* Thread-local message of the last failing call on this thread. */
const char* dragon_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DRAGON_H_ */
