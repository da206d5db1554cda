/*
 * randes.h -- C ABI of the B200 RanDeS library.
 *
 * RanDeS (Randomized Delta Superposition) stores T models fine-tuned from one
 * base W_0 as W_0 plus ONE superposed delta
 *
 *        M = sum_i T_i (W_i - W_0)                       (Section 4, first display)
 *
 * where every T_i is a random orthogonal transform fixed by a seed, and brings
 * one model back on demand as
 *
 *        What_t = W_0 + lambda * T_t^-1 (M)              (Section 4, second display)
 *
 * T_i is a shuffle of same-shape layers (Section 4.3), a per-column +-1 sign
 * flip (Section 4.4), or both.  Models are added to and removed from M without
 * recomputation (Section 5.7).
 *
 * General conventions
 * -------------------
 * - A model is a list of n_layers row-major tensors [rows, cols]; a 1-D
 *   parameter is [1, cols].  "Column" = the second, contiguous index.
 * - Layers with the same `group` id must have the same shape; a group is the
 *   set of "layers of the same type" that may be shuffled among each other.
 *   Group members are ordered by layer index.
 * - Pointer arrays (`base`, `tasks`, `out`) are HOST arrays of DEVICE
 *   pointers, one per layer, in layer order.  The library copies them; the
 *   caller may free or reuse the arrays as soon as the call returns.
 * - All tensor data, M and the workspace are DEVICE memory owned by the
 *   caller.  The library allocates no device memory and frees nothing it is
 *   handed.  Weight tensors must be aligned to their element size; 16-byte
 *   aligned tensors with cols % 4 == 0 take the vectorised path.
 * - M is one arena of randes_superposition_bytes() bytes, 256-byte aligned;
 *   slot l starts at byte randes_layer_offset(plan, l) (the first slot a little
 *   way in, not at 0: ask, do not assume).  Its element type is
 *   the plan's m_dtype: fp32 by default whatever the storage type of the
 *   weights, or bf16 (half the footprint; a smaller superposition is what
 *   the paper's conclusion leaves to future work).  Sums always run in fp32: with a bf16 M,
 *   compress rounds each element once at the end (nearest even), add / remove
 *   widen the stored element, add in fp32 and round again, retrieve widens.
 * - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   Calls enqueue work and return; results are ordered on `stream`.  All calls
 *   on one plan must be issued on one stream or otherwise ordered by the
 *   caller: they share the plan's device workspace.
 * - Every entry point returns 0 (RANDES_OK) or a negative randes_status_t;
 *   randes_last_error() then describes the failure.  Arguments are validated
 *   before anything is launched; nothing crosses the ABI as an exception.
 * - Results are deterministic: every output element is written by exactly one
 *   thread, tasks are summed in plan order, each fp32 operation is rounded
 *   once (W_i - W_0, then the accumulation; retrieval is one fused
 *   multiply-add), bf16 conversion is round-to-nearest-even.
 * - Not thread-safe per plan; distinct plans may be used from distinct threads.
 */
#ifndef RANDES_H
#define RANDES_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct randes_plan_s randes_plan_t; /* opaque, host memory, library-owned */

typedef enum { RANDES_F32 = 0, RANDES_BF16 = 1 } randes_dtype_t;

/* per-group transform flags.
 *   RANDES_SHUFFLE  random permutation of the group's members per task (Section 4.3)
 *   RANDES_FLIP     per-column +-1 sign flip (Section 4.4)
 *   RANDES_SHIFT    deterministic alternative to SHUFFLE (appendix on the dynamics between
 *                   shuffling and sign flips): the participating members are rotated
 *                   towards higher index, task t by 1 + (t mod (n - 1)) of n positions.
 *                   Mutually exclusive with RANDES_SHUFFLE.
 *   RANDES_SKIP(k)  skip rate of the same appendix: only the members with index 0, k,
 *                   2k, ... of the group (in layer order) are shuffled / shifted and
 *                   flipped; k = 0 or 1 means all.  1 <= k <= 255.
 *   RANDES_GAUSS    the "RD" context matrix of the ablation in Section 5.5 instead of the +-1 one:
 *                   a diagonal of (nearly) standard normal entries, one per (task, slot, column).
 *                   Not orthogonal: compress multiplies by it, retrieve divides (the paper shows
 *                   that it interferes more; it is here for that comparison).  Entry = sum of
 *                   twelve uniforms minus six, drawn from the task's Philox stream in exactly
 *                   rounded fp32 steps.  Mutually exclusive with RANDES_FLIP; needs an fp32
 *                   superposition.  A plan with such a group runs compress, add, remove and
 *                   retrieve through kernels of their own, which read the entries from a table
 *                   kept in the plan's workspace (size it with randes_plan_workspace_bytes_groups;
 *                   one extra kernel launch whenever tasks are registered or removed), and does not offer
 *                   randes_retrieve_batch, randes_retrieve_static, randes_delta_gram or randes_linear. */
enum { RANDES_SHUFFLE = 1, RANDES_FLIP = 2, RANDES_SHIFT = 4, RANDES_GAUSS = 1 << 16 };
#define RANDES_SKIP(k) (((uint32_t)(k) & 0xFFu) << 8)

typedef struct { uint32_t rows, cols, group; } randes_layer_t;
typedef struct { uint32_t flags; } randes_group_t;

typedef enum {
    RANDES_OK = 0,
    RANDES_INVALID_ARGUMENT = -1,
    RANDES_SHAPE_MISMATCH = -2,   /* members of one group differ in shape */
    RANDES_UNKNOWN_TASK = -3,
    RANDES_DUPLICATE_TASK = -4,
    RANDES_WORKSPACE_TOO_SMALL = -5,
    RANDES_UNSUPPORTED_DTYPE = -6,
    RANDES_MISALIGNED = -7,       /* pointer not aligned to its element size */
    RANDES_CAPACITY = -8,         /* plan already holds max_tasks tasks */
    RANDES_CUDA_ERROR = -9,
    RANDES_OUT_OF_MEMORY = -10    /* host allocation failed */
} randes_status_t;

/*
 * Bytes of device workspace a plan over these layers needs for up to max_tasks
 * registered tasks.  Returns 0 on invalid arguments.  Host-only.
 */
size_t randes_plan_workspace_bytes(const randes_layer_t* layers, uint32_t n_layers,
                                   uint32_t max_tasks);

/*
 * The same for a plan with these groups.  Equal to randes_plan_workspace_bytes unless a group
 * carries RANDES_GAUSS (the diagonal context of Section 5.5): such a plan also keeps, in its
 * workspace, a table of the context's factors -- 4 bytes per registered task and column of every
 * layer, written when a task is registered -- and randes_plan answers WORKSPACE_TOO_SMALL to less.
 * Returns 0 on invalid arguments.  Host-only.
 */
size_t randes_plan_workspace_bytes_groups(const randes_layer_t* layers, uint32_t n_layers,
                                          const randes_group_t* groups, uint32_t n_groups,
                                          uint32_t max_tasks);

/*
 * Build a plan (Sections 4.2-4.4; seeds as in the appendix on the default
 * experimental setup: one seed per model drives both its shuffle and its sign
 * matrices).
 *
 *   layers[n_layers], groups[n_groups]  host arrays, copied.
 *   storage_dtype   element type of every W_0 / W_i tensor.
 *   m_dtype         element type of the superposition arena M (RANDES_F32 or RANDES_BF16).
 *   task_ids/seeds[n_tasks]  the initially registered models, in the order in
 *                   which compress sums them.  Ids must be distinct.
 *   max_tasks       capacity of the registry (>= n_tasks, >= 1).
 *   dev_workspace   device memory, 256-byte aligned, at least
 *                   randes_plan_workspace_bytes_groups() bytes; used by the plan until
 *                   randes_plan_destroy.  The layer, tile and permutation
 *                   tables are copied into it on `stream`.
 *   out_plan        receives the plan; free with randes_plan_destroy.
 *
 * For every registered task and every group with RANDES_SHUFFLE and >= 2
 * members a permutation sigma is drawn from the task's seed (Fisher-Yates on a
 * Philox4x32-10 stream); slot k of the shuffled delta holds member sigma(k).
 * Errors: INVALID_ARGUMENT, SHAPE_MISMATCH, DUPLICATE_TASK,
 * WORKSPACE_TOO_SMALL, UNSUPPORTED_DTYPE, MISALIGNED, CUDA_ERROR.
 */
int randes_plan(const randes_layer_t* layers, uint32_t n_layers,
                const randes_group_t* groups, uint32_t n_groups,
                randes_dtype_t storage_dtype, randes_dtype_t m_dtype,
                const uint32_t* task_ids, const uint64_t* seeds, uint32_t n_tasks,
                uint32_t max_tasks,
                void* dev_workspace, size_t dev_workspace_bytes, void* stream,
                randes_plan_t** out_plan);

void randes_plan_destroy(randes_plan_t* plan); /* NULL is allowed; frees host memory only */

/* Size of the arena M: 1 KiB of lead-in, then rows*cols elements of m_dtype per layer, each slot padded to
 * 256 bytes.  Independent of the number of tasks (Section 4.1: a seed per added model). */
size_t randes_superposition_bytes(const randes_plan_t* plan);

/* Byte offset of slot `layer` inside M; (size_t)-1 if out of range. */
size_t randes_layer_offset(const randes_plan_t* plan, uint32_t layer);

uint32_t randes_num_layers(const randes_plan_t* plan);
uint32_t randes_num_tasks(const randes_plan_t* plan);

/* Copies the registered ids / seeds, in summation order, into host arrays of
 * randes_num_tasks() entries (either may be NULL). */
int randes_task_list(const randes_plan_t* plan, uint32_t* task_ids, uint64_t* seeds);

/*
 * Self-check of a plan, on the host (a debugging aid: no compute call needs it).  Verifies what the
 * kernels take for granted: every task's sigma is a bijection that stays inside its group and
 * sigma^-1 inverts it (Section 4.3: layers are shuffled among layers of the same type only); the slots
 * of M are aligned, ordered and disjoint; and each of the plan's tile lists covers every
 * (row, column block) of every layer exactly once and never leaves a layer -- so every element of M or
 * of a retrieved model is written by exactly one thread block.  Returns RANDES_OK, or
 * INVALID_ARGUMENT with randes_last_error() naming the first violation.
 */
int randes_plan_validate(const randes_plan_t* plan);

/*
 * Checked build (a debugging aid: the library compiled with -DRANDES_CHECKED, see the build script).  In that
 * build the streaming kernels (retrieve, compress / add / remove, their group and batched forms) compare, before a
 * thread block touches a tile, every index the tile's addresses are derived from -- the tile's layer, the layers and
 * slots it reaches through sigma / sigma^-1 (Section 4.3), its rows -- with the plan's bounds; a tile that fails is
 * skipped instead of read or written, and the first failure is kept in a device word.  This call synchronises with
 * the current device and returns that word: 0 = none; else bit 63 set, bits 48-55 the kernel (1 retrieve,
 * 2 compress / add / remove, 3 add / remove for bf16 weights, 4 group compress, 5 batched retrieve, 6 batched group
 * retrieve), bits 40-47 what failed (1 the tile's layer, 2 a permuted layer or slot, 3 the rows), bits 0-31 the tile.
 * *checked_build (may be NULL) tells whether this library is a checked build; the ordinary build always reports 0.
 * What such a word means in practice: the plan's device workspace was overwritten, or the plan does not belong to
 * these tensors.  Errors: INVALID_ARGUMENT, CUDA_ERROR.
 */
int randes_debug_violation(uint64_t* word, int* checked_build);

/*
 * Persistence.  What RanDeS keeps per model is a seed (Section 4.1), so a plan
 * is fully described by its layer shapes, group flags, element types and the
 * registered (id, seed) pairs in summation order; M itself is the caller's
 * buffer to save.  serialize writes that description as a self-contained blob
 * (host memory; pass buffer = NULL to get the size) and returns the number of
 * bytes, 0 on error.  deserialize rebuilds an equivalent plan from a blob; the
 * workspace arguments are those of randes_plan (NULL workspace = host-only),
 * and max_tasks is raised to the number of stored tasks if it is smaller.
 * Errors: INVALID_ARGUMENT (not a blob, truncated), plus those of randes_plan.
 */
size_t randes_plan_serialize(const randes_plan_t* plan, void* buffer, size_t buffer_bytes);
/*
 * Bytes of device workspace a plan equal to this one needs (same layers, groups, element types and
 * max_tasks): the figure randes_plan checks, at most randes_plan_workspace_bytes_groups().  Also
 * answered by a host-only plan -- to size the workspace of a plan kept as a blob, deserialize it
 * without a workspace, ask, and deserialize again with the memory.  0 for a NULL plan.
 */
size_t randes_plan_workspace_needed(const randes_plan_t* plan);
int randes_plan_deserialize(const void* buffer, size_t buffer_bytes, uint32_t max_tasks,
                            void* dev_workspace, size_t dev_workspace_bytes, void* stream,
                            randes_plan_t** out_plan);

/*
 * Host copies of one task's layer tables (n_layers entries each, either may be
 * NULL):  src_of_slot[l] = layer whose delta lands on slot l (sigma);
 * slot_of_pos[p] = slot holding layer p's delta (sigma^-1).   (Section 4.3)
 * Errors: UNKNOWN_TASK.
 */
int randes_task_tables(const randes_plan_t* plan, uint32_t task_id,
                       uint32_t* src_of_slot, uint32_t* slot_of_pos);

/*
 * compress (Section 4, first display; Section 4.4, first display):
 *   M[l][r,c] = sum over registered tasks i, in plan order, of
 *               s_i(l,c) * ( W_i[sigma_i(l)][r,c] - W_0[sigma_i(l)][r,c] )
 * starting from +0.  M is overwritten.
 *   base[n_layers]             W_0, or NULL: `tasks` then hold the deltas
 *                              themselves (adapter deltas, Section 5.8).
 *   tasks[n_tasks * n_layers]  tasks[i*n_layers + l] = layer l of the i-th
 *                              registered task.
 * With a bf16 superposition at most 32 tasks can be summed in one call
 * (CAPACITY otherwise): further models are added with randes_add_model.
 * One kernel launch, or two when some groups are shuffled (those groups go through a kernel that stages
 * the base tiles of a whole group in shared memory, the remaining tensors through the per-layer kernel).
 * Errors: INVALID_ARGUMENT, MISALIGNED, CAPACITY, CUDA_ERROR.
 */
int randes_compress(randes_plan_t* plan, const void* const* base, const void* const* tasks,
                    void* M, void* stream);

/*
 * Model hot swapping (Section 5.7).
 *   add:     registers (task_id, seed) at the end of the summation order and
 *            performs  M <- M + T_j(W_j - W_0)  in place.
 *   remove:  performs  M <- M - T_j(W_j - W_0)  in place and drops the task.
 *            The library keeps no deltas: the caller passes the same weights
 *            that were added.  Exact up to one fp32 rounding per element.
 * base may be NULL (task holds the delta).  One kernel launch each.
 * Errors: DUPLICATE_TASK, CAPACITY (add); UNKNOWN_TASK (remove);
 * INVALID_ARGUMENT, MISALIGNED, CUDA_ERROR.
 */
int randes_add_model(randes_plan_t* plan, uint32_t task_id, uint64_t seed,
                     const void* const* base, const void* const* task, void* M, void* stream);
int randes_remove_model(randes_plan_t* plan, uint32_t task_id,
                        const void* const* base, const void* const* task, void* M, void* stream);

/*
 * Several models added in one pass over M (Section 5.7 applied to a set):
 *   M <- M + T_a(W_a - W_0) + T_b(W_b - W_0) + ...      in the order given,
 * each term rounded once in fp32, starting from M's values; the tasks are
 * registered at the end of the summation order, in that order.  With an fp32
 * superposition the result equals, bit for bit, n_tasks calls of
 * randes_add_model, but M is read and written once instead of n_tasks times.
 * A bf16 superposition is widened once and rounded once, at the end (so the
 * result may differ in the last bit from separate adds, which round each time);
 * it takes at most 32 models per call.
 *   task_ids[n_tasks], seeds[n_tasks]   new, distinct ids; n_tasks may be 0 (nothing happens)
 *   base[n_layers] or NULL; tasks[n_tasks * n_layers] as for randes_compress
 * Either every model is added or, on error, none.  One kernel launch.
 * Errors: DUPLICATE_TASK, CAPACITY, INVALID_ARGUMENT, MISALIGNED, CUDA_ERROR.
 */
int randes_add_models(randes_plan_t* plan, const uint32_t* task_ids, const uint64_t* seeds, uint32_t n_tasks,
                      const void* const* base, const void* const* tasks, void* M, void* stream);

/*
 * retrieve (Section 4, second display; Section 4.4, second display):
 *   out[p][r,c] = fma(lambda, s_t(l,c) * M[l][r,c], W_0[p][r,c]),  l = sigma_t^-1(p)
 * written as out_dtype (fp32, or bf16 rounded to nearest even).
 *   base[n_layers], out[n_layers]; out must not alias base or M.
 * One kernel launch.  Errors: UNKNOWN_TASK, UNSUPPORTED_DTYPE,
 * INVALID_ARGUMENT, MISALIGNED, CUDA_ERROR.
 */
int randes_retrieve(randes_plan_t* plan, uint32_t task_id, float lambda,
                    randes_dtype_t out_dtype, const void* const* base, const void* M,
                    void* const* out, void* stream);

/*
 * A linear layer on the retrieved weight of one layer, without writing that
 * weight to memory (Section 4, second display, inside y = x What^T; the serving
 * case of the paper's introduction):
 *   y[b][r] = sum_c x[b][c] * ( W_0[p][r,c] + lambda * s_t(l,c) * M[l][r,c] ),  l = sigma_t^-1(p)
 * computed as x W_0[p]^T + lambda * (x D_t) M[l]^T: the inverse sign flip acts on the
 * activations' columns, the inverse shuffle is the choice of the slot l.  Two bf16
 * products on the tensor cores with fp32 accumulation; lambda is applied once per
 * output in fp32.  Needs a plan with bf16 weights AND a bf16 superposition.
 *   layer                 position p; its shape [rows, cols] must have cols % 8 == 0
 *   x                     device, [n_tokens, cols] bf16 row-major, 16-byte aligned
 *   base[n_layers]        host array of device pointers (only base[layer] is used, 16-byte aligned)
 *   M                     device, the superposition arena
 *   y, y_dtype            device, [n_tokens, rows] row-major, fp32 or bf16 (the fp32 result rounded to nearest
 *                         even, once); must not alias the inputs
 *   n_tokens              at most 8388480 (65535 blocks of 128 tokens)
 * Needs no workspace (the plan may have been built without one).  One or two kernel launches
 * (the first tokens in blocks of 256, the rest in blocks of 128, split where that takes the fewest
 * waves over the SMs); asynchronous on `stream`.  The result equals the fp64 definition within
 * 2 * cols * 2^-24 * sum_c |x| (|W_0| + |lambda M|) per output (fp32 accumulation of 2 * cols
 * exact products in any order).  Errors: UNSUPPORTED_DTYPE, UNKNOWN_TASK, INVALID_ARGUMENT,
 * MISALIGNED, CUDA_ERROR.
 */
int randes_linear(const randes_plan_t* plan, uint32_t task_id, float lambda, uint32_t layer, const void* x,
                  uint32_t n_tokens, const void* const* base, const void* M, void* y, randes_dtype_t y_dtype, void* stream);

/*
 * randes_linear behind a gate (same computation: Section 4, second display, inside y = x What^T).
 * Every thread block first waits until the 32-bit word *gate in device memory is non-zero --
 * written, for instance, by the kernel on another stream that produces x -- and only then reads
 * its operands.  The wait, like every other wait inside the kernel, ends after wait_ns nanoseconds
 * of the block's life (0 = the default of one second, at most 60 s): a block whose wait runs out
 * issues no copy and no product, writes nothing to y, frees what it holds, returns, and is counted
 * by randes_linear_giveups; the call itself still returns RANDES_OK (it only enqueues), so a caller
 * that uses a gate reads the counter afterwards.  The context stays usable.
 *   gate      device, 4-byte aligned, not NULL; whoever writes it must make x visible first
 *             (a release store or a fence before the store)
 * Errors: those of randes_linear, plus INVALID_ARGUMENT (gate NULL, wait_ns beyond 60 s).
 */
int randes_linear_gated(const randes_plan_t* plan, uint32_t task_id, float lambda, uint32_t layer, const void* x,
                        uint32_t n_tokens, const void* const* base, const void* M, void* y, randes_dtype_t y_dtype,
                        const uint32_t* gate, uint64_t wait_ns, void* stream);

/*
 * Every wait inside the randes_linear kernel is bounded; a thread block whose wait runs out
 * skips its tile and counts itself here.  *count = number of such blocks since the library was
 * loaded on the current device (0 in a healthy run).  Synchronises with the device.
 */
int randes_linear_giveups(unsigned int* count);

/*
 * Batched retrieve: rebuild n_tasks models in one pass (Section 4, second
 * display, for several tasks at once; the multi-model serving case of the
 * paper's introduction).  Equivalent, bit for bit, to n_tasks calls of
 * randes_retrieve, but W_0 is read once instead of n_tasks times.
 *   task_ids[n_tasks]           distinct registered ids, 1 <= n_tasks <= 32 and <= max_tasks
 *   out[n_tasks * n_layers]     out[b*n_layers + l] = layer l of the b-th requested model
 * One kernel launch, or two when some groups are shuffled (fp32 weights and superposition).
 * Errors: as randes_retrieve, plus DUPLICATE_TASK, CAPACITY.
 */
int randes_retrieve_batch(randes_plan_t* plan, const uint32_t* task_ids, uint32_t n_tasks, float lambda,
                          randes_dtype_t out_dtype, const void* const* base, const void* M,
                          void* const* out, void* stream);

/*
 * Interference diagnostics (Section 3, the equation for the norm of the
 * interference; the paper's figures on pairwise cosine similarity among the
 * interfering deltas during retrieval).  Computes, for the registered tasks in
 * plan order, the Gram matrix of the transformed deltas
 *     gram[i*n + j] = < T_i (W_i - W_0) , T_j (W_j - W_0) >     (fp64, n = number of tasks)
 * summed over every parameter.  Because every T is orthogonal, the deltas that
 * interfere when task t is retrieved, T_t^-1 T_j d_j (j != t), have exactly these
 * inner products: cos(j, l) = gram[j][l] / sqrt(gram[j][j] gram[l][l]) and
 * || lambda sum_{j != t} T_t^-1 T_j d_j || = lambda sqrt( sum_{j,l != t} gram[j][l] ).
 *   base / tasks     as for randes_compress (base may be NULL: tasks hold deltas)
 *   gram             DEVICE array of n*n doubles, written on `stream`
 *   scratch          device memory of at least randes_delta_gram_scratch_bytes(plan) bytes
 * Products are exact in fp64 and summed in a fixed order (fp64 tensor-core
 * products over blocks of 8 x 8 tasks, upper triangle, mirrored): the result is
 * symmetric and reproducible bit for bit.  At most 32 tasks.  One pass over the
 * weights, two kernel launches.
 * Errors: INVALID_ARGUMENT, CAPACITY, MISALIGNED, WORKSPACE_TOO_SMALL, CUDA_ERROR.
 */
size_t randes_delta_gram_scratch_bytes(const randes_plan_t* plan);
int randes_delta_gram(randes_plan_t* plan, const void* const* base, const void* const* tasks,
                      double* gram, void* scratch, size_t scratch_bytes, void* stream);

/*
 * What the Gram matrix says about one retrieval (Section 3, the equation for the norm of
 * the interference; Section 4, second display: What_t - W_0 - lambda d_t is exactly the
 * interference term).  For the task in row/column t of `gram`,
 *     *norm = lambda * sqrt( sum_{j != t} sum_{l != t} gram[j*n + l] )
 *           = || lambda * sum_{j != t} T_t^-1 T_j d_j ||_2 ,
 * the rows added in index order, each row in index order, in fp64; a sum that rounding
 * pushed below zero counts as zero.
 *   gram   HOST array of n*n doubles (randes_delta_gram's result copied back), n >= 1
 * Host-only; nothing is launched.  Errors: INVALID_ARGUMENT (NULL, t >= n).
 */
int randes_interference_norm(const double* gram, uint32_t n, uint32_t t, double lambda, double* norm);

/*
 * Pairwise cosine similarity among the deltas that interfere in a retrieval (the paper's
 * figures on cosine similarity among interfering deltas, main text and appendix):
 *     cos(j, l) = gram[j*n + l] / sqrt(gram[j*n + j] * gram[l*n + l])
 * (the same for T_j d_j, T_l d_l and for T_t^-1 T_j d_j, T_t^-1 T_l d_l: T_t is orthogonal).
 *   gram      HOST array of n*n doubles
 *   exclude   index of the retrieved task, left out of the mean; negative = none
 *   cosines   HOST array of n*n doubles or NULL; receives every cos(j, l) (1 on the
 *             diagonal; 0 where a delta has zero norm)
 *   mean      or NULL; receives the mean over the pairs j < l with j, l != exclude,
 *             summed in index order (0 when there is no such pair)
 * Host-only; nothing is launched.  Errors: INVALID_ARGUMENT (NULL gram, n == 0, exclude >= n).
 */
int randes_pairwise_cosines(const double* gram, uint32_t n, int32_t exclude, double* cosines, double* mean);

/*
 * retrieve for callers that cannot provide a device workspace.  (The paper has
 * no counterpart: this entry point exists for deployment, not for the method.)
 *
 * Who needs it: code that is handed the weight tensors and a stream but does
 * not own a device allocator -- a plug-in inside a serving process whose memory
 * pool belongs to the host framework, or a request handler that swaps models in
 * a latency-critical loop, where cudaMalloc / cudaFree would stall the device
 * and are therefore forbidden.  Such a caller builds its plan with
 * dev_workspace == NULL (host-only) and calls this instead of randes_retrieve.
 *
 * Same arguments, results and errors as randes_retrieve (bit-identical output);
 * `plan` may be host-only.  The tables the kernel reads are copied, in
 * one transfer on `stream`, into a fixed array of RANDES_STATIC_SCRATCH_BYTES that lives inside
 * the library on every GPU that loads it, for the life of the process.  The
 * call allocates no device memory and frees none.
 *   - Limit: 52 bytes per layer plus 16 bytes per tile of 16 rows x 1024 fp32
 *     (2048 bf16) columns, each of the five tables rounded up to 256 bytes,
 *     must fit the array (models up to roughly a billion parameters); larger
 *     plans fail with RANDES_CAPACITY before anything is launched.
 *   - The first call on each device looks up the array's device address and
 *     sizes the grid; make that first call outside any stream capture.
 *   - All calls on one device share the array.  Calls on one stream are ordered
 *     and safe; calls whose work may overlap on the GPU (different streams,
 *     different plans or threads) race on the tables and must be serialised by
 *     the caller.  Nothing in the array needs clearing between calls: each call
 *     rewrites every entry it reads.
 */
#define RANDES_STATIC_SCRATCH_BYTES (1u << 20)
int randes_retrieve_static(const randes_plan_t* plan, uint32_t task_id, float lambda,
                           randes_dtype_t out_dtype, const void* const* base, const void* M,
                           void* const* out, void* stream);

/* Number of kernels this library has launched in this process (all plans). */
uint64_t randes_launch_count(void);

/* Description of the calling thread's most recent failure; never NULL. */
const char* randes_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* RANDES_H */
