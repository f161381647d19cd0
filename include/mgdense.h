/*
 * mgdense — DENSE multi-hop neighbourhood sampling, GraphSage forward over DENSE and
 * DistMult link scoring on one NVIDIA B200 (sm_100a), behind a plain C ABI.
 *
 * The operations are those of MariusGNN (EuroSys '23): Algorithm 1 (multi-hop sampling
 * into the DENSE arrays), Section 4.1 (oneHopSample / computeNextDelta over the in-memory
 * subgraph), Section 4.2 (repr_map, layer evaluation, Algorithm 2's update, Algorithm 3's
 * aggregation) and the partition buffer of Section 3.
 *
 * Conventions
 *  - Every call returns an int32 status: MG_OK (0) or a negative MG_ERR_* code; nothing
 *    throws, aborts or traps.  mg_last_error(ctx) gives a message owned by the context.
 *  - "host" / "device" is stated per pointer.  Input arrays are caller-owned and only read
 *    during the call unless a parameter says the library keeps (borrows) the pointer.
 *  - Opaque handles are created and destroyed by the library.  A context is bound to one
 *    device and one stream (the stream handed to mg_create; 0 = the default stream); all
 *    kernels run on it.  Partition swaps run on a library-owned side stream.
 *  - Node ids are int32.  CSR row offsets are int32 or int64 on input.
 *  - A context is not thread-safe; use one per host thread.
 */
#ifndef MGDENSE_H
#define MGDENSE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MG_OK 0
#define MG_ERR_ARG (-1)         /* null pointer, negative size, k <= 0, fanout <= 0, id out of range */
#define MG_ERR_STATE (-2)       /* call made before the data it needs was loaded */
#define MG_ERR_NONRESIDENT (-3) /* a target lies in a partition that is not in the buffer */
#define MG_ERR_DUPLICATE (-4)   /* a batch lists the same target twice (Algorithm 1 wants unique ids) */
#define MG_ERR_CAPACITY (-5)    /* a caller-set capacity was exceeded; nothing was written out of bounds */
#define MG_ERR_OOM (-6)         /* a device or host allocation failed */
#define MG_ERR_TIMEOUT (-7)     /* a bounded wait on the side stream ran out */
#define MG_ERR_CUDA (-8)        /* a CUDA runtime call failed; see mg_last_error */

#define MG_DTYPE_F32 0
#define MG_DTYPE_F16 1

#define MG_BACKING_HBM 0  /* the whole feature table lives in device memory */
#define MG_BACKING_HOST 1 /* the table stays in (preferably pinned) host memory; only the
                             buffer's partitions are copied into device slots */

#define MG_GEMM_TF32 0 /* tcgen05 kind::tf32, operands rounded to nearest TF32, fp32 accumulate */
#define MG_GEMM_FP32 1 /* CUDA-core fp32 FMA; slow, for isolating tensor-core rounding */

#define MG_CORRUPT_DST 1
#define MG_CORRUPT_SRC 2
#define MG_CORRUPT_BOTH 3

#define MG_MAX_HOPS 8
#define MG_MAX_FANOUT 1024
#define MG_MAX_BATCHES 4096
#define MG_MAX_PARTS 256

typedef struct mg_ctx mg_ctx;
typedef struct mg_dense mg_dense;
typedef struct mg_model mg_model;
typedef struct mg_lp_batch mg_lp_batch;

/* Capacities of one mg_sample_many call.  A zero field selects the worst-case bound
 * computed from the targets and fanouts, clamped to the graph's size. */
typedef struct mg_sample_caps {
    int64_t max_nodes_total;     /* sum over batches of |node_ids| */
    int64_t max_entries_total;   /* sum over batches of |nbrs| */
    int32_t max_nodes_per_batch; /* |node_ids| of one batch; sizes the per-batch id table */
    int32_t max_inner_nodes_per_batch; /* nodes of one batch WITHOUT its farthest delta (targets and the deltas that are
                                          sampled from).  When the last hop is deduplicated in shared memory only these
                                          go through the id tables in global memory, so a bound here makes the tables
                                          several times smaller (L2-resident at the bench's sizes).  0 = as large as
                                          max_nodes_per_batch. */
} mg_sample_caps;

/* One batch's DENSE in the paper's layout (Section 4.1): node_ids = [Delta_0 .. Delta_k],
 * nbrs = [nbrs(Delta_1) .. nbrs(Delta_k)].  All pointers are DEVICE pointers into a buffer
 * owned by the mg_dense, valid until the next mg_dense_view / mg_sample* on it or its free.
 * node_id_offsets has k+2 entries (last = n_nodes); nbr_offsets has n_sampled+1 entries
 * (last = n_entries) — the terminal entries Algorithm 2 reads on the last layer. */
typedef struct mg_dense_arrays {
    int32_t k;
    int32_t n_nodes;   /* |node_ids| */
    int32_t n_sampled; /* nodes that carry neighbours = n_nodes - |Delta_0| */
    int32_t n_entries; /* |nbrs| */
    const int32_t* node_ids;
    const int32_t* node_id_offsets;
    const int32_t* nbrs;
    const int32_t* nbr_offsets;
    const int32_t* repr_map;
} mg_dense_arrays;

/* ---- context ---------------------------------------------------------------------- */

/* Create a context on `device`, issuing work on `stream` (a cudaStream_t; NULL = default
 * stream).  *out receives the handle. */
int mg_create(mg_ctx** out, int device, void* stream);
/* Free everything the context owns (graph copy, buffer slots, workspaces).  Handles made
 * from it (mg_dense, mg_model, mg_lp_batch) must be freed first. */
int mg_destroy(mg_ctx* ctx);
/* Message of the last failed call on this context ("" if none).  Owned by the context. */
const char* mg_last_error(const mg_ctx* ctx);

/* ---- graph store and partition buffer (Section 3) ------------------------------------- */

/* Load the sampling adjacency as CSR: row v lists the nodes v aggregates from (Figure 1:
 * the incoming neighbourhood), each row sorted by neighbour id.  row_offsets has
 * n_nodes+1 entries of int32 (offsets_are_i64 = 0) or int64; nbrs has n_edges int32
 * entries.  Both pointers are host (ptrs_are_device = 0) or device pointers; the library
 * copies them.  Resets partitioning to one resident partition.  Errors: MG_ERR_ARG on
 * null/negative/non-monotone sizes (offsets[0] != 0 or offsets[n] != n_edges), MG_ERR_OOM. */
int mg_load_graph(mg_ctx* ctx, int64_t n_nodes, int64_t n_edges, const void* row_offsets,
                  int offsets_are_i64, const int32_t* nbrs, int ptrs_are_device);

/* Load the second edge list of Section 4.1 as CSR over the same nodes: row v lists the
 * destinations of v's outgoing edges, each row sorted by neighbour id; same array
 * conventions as mg_load_graph, which must have been called before (a new mg_load_graph
 * drops this list).  Needed by mg_set_sample_direction(MG_SAMPLE_INOUT).  The in-buffer
 * filter applies to it as to the first list.  Errors: MG_ERR_STATE without a graph,
 * MG_ERR_ARG on a malformed CSR, MG_ERR_OOM. */
int mg_load_out_graph(mg_ctx* ctx, int64_t n_edges, const void* row_offsets, int offsets_are_i64,
                      const int32_t* nbrs, int ptrs_are_device);

/* Which edges one-hop sampling draws from (Section 4.1, Section 7.1): MG_SAMPLE_IN (default) =
 * the rows given to mg_load_graph; MG_SAMPLE_INOUT = per node up to f of those followed by
 * up to f rows of mg_load_out_graph (f = the hop's fanout, applied per direction; the
 * outgoing draws are keyed by slots 65536 + t).  Errors: MG_ERR_ARG on an unknown value,
 * MG_ERR_STATE for MG_SAMPLE_INOUT without an outgoing list. */
#define MG_SAMPLE_IN 0
#define MG_SAMPLE_INOUT 1
int mg_set_sample_direction(mg_ctx* ctx, int direction);

/* Split the nodes into n_parts physical partitions (Section 3).  part_of_node = NULL: ceil(n_nodes / n_parts)
 * contiguous ids each (the last one short) -- the sequential lookup table cut into pieces.  part_of_node != NULL: a
 * HOST array of n_nodes partition ids (< n_parts), copied -- the partition-id array of the graph store; Section 5.2's
 * policy (training nodes in the first partitions, the others assigned at random) is expressed this way.  A node's place
 * inside its partition is its rank among the partition's nodes in ascending id.  With MG_BACKING_HOST the host table
 * (or the blocks named by mg_set_partition_source) is then partition-major: partition 0's rows in that order, then
 * partition 1's, ...; with MG_BACKING_HBM the table stays in node order.  Buffer slots hold the largest partition.
 * Negatives of mg_lp_prepare count resident nodes partition after partition, ascending id inside a partition.
 * All partitions start non-resident except when n_parts == 1.  Drops any loaded feature table.
 * Errors: MG_ERR_ARG (n_parts outside [1, MG_MAX_PARTS], an id >= n_parts), MG_ERR_STATE, MG_ERR_OOM. */
int mg_set_partitioning(mg_ctx* ctx, int32_t n_parts, const uint8_t* part_of_node);

/* Attach the table of base representations (Section 2): n_nodes rows of `dim` values of
 * `dtype`, row-major.  dim * sizeof(dtype) must be a multiple of 16 bytes.
 *  - MG_BACKING_HBM: every row is kept in device memory.  A device `table`
 *    (table_is_device = 1) is BORROWED — it must outlive the context's use of it; a host
 *    table is copied.  buffer_capacity_parts only bounds how many partitions may be
 *    resident for sampling.
 *  - MG_BACKING_HOST: `table` is a host pointer the caller keeps valid (pinned memory makes
 *    the swaps asynchronous).  The library allocates buffer_capacity_parts + 1 device slots
 *    of one partition each (the spare slot lets a one-partition swap load while the old
 *    set is still in use) and copies partitions in as mg_set_resident asks. */
int mg_load_features(mg_ctx* ctx, const void* table, int table_is_device, int dtype, int32_t dim,
                     int32_t buffer_capacity_parts, int backing);

/* MG_BACKING_HOST only: partition `part`'s rows (its ceil(n_nodes / n_parts) rows, the last partition fewer) are
 * at host_block instead of at their place in the table -- for tables that do not fit host memory as a whole (config
 * 4: 187 GB): the caller keeps a few pinned staging blocks, fills one with a partition (from disk, or regenerated),
 * names it here, and asks for the partition with mg_set_resident.  mg_load_features may then be given table = NULL.
 * The block must stay valid and unchanged until the mg_commit_resident that brings the partition in has returned
 * MG_OK (and, if the partition's rows are updated in the buffer, until it has been evicted: the write-back goes to the
 * same block).  NULL removes the override.  Errors: MG_ERR_ARG, MG_ERR_STATE (no host-backed buffer, or a set pending). */
int mg_set_partition_source(mg_ctx* ctx, int32_t part, const void* host_block);

/* Ask for the set of resident partitions (the S_i of Section 3).  The difference to the
 * current set is computed; partitions to be added are copied host->device on the side
 * stream (MG_BACKING_HOST).  Sampling and forward calls keep using the current set until
 * mg_commit_resident.  async = 0 commits before returning.  Errors: MG_ERR_ARG (id out of
 * range, duplicates), MG_ERR_CAPACITY (n > buffer capacity), MG_ERR_STATE. */
int mg_set_resident(mg_ctx* ctx, const int32_t* part_ids /*host*/, int32_t n, int async);

/* Wait at most timeout_ms for the pending copies (polling, never an unbounded wait), then
 * switch the slot map to the pending set and rebuild the in-buffer view of the graph: the
 * rows of resident nodes restricted to resident neighbours (sampling sees only in-memory
 * nodes and edges, Section 3).  timeout_ms <= 0 polls once.  MG_ERR_TIMEOUT leaves the pending set
 * pending and the committed one in use: sampling and forward calls go on under the old set, and a
 * later mg_commit_resident picks the pending set up.  A sample drawn under the old set stays usable
 * after the commit only if every partition that was resident when it was drawn kept its slot (the
 * new set contains the old one); otherwise calls that read feature rows through it (mg_forward,
 * mg_backward, mg_gather_h0, mg_gat_forward, mg_apply_embedding_sgd ...) refuse it with
 * MG_ERR_STATE -- run them before the commit, or sample again. */
int mg_commit_resident(mg_ctx* ctx, int32_t timeout_ms);

/* ---- DENSE sampling (Algorithm 1) ---------------------------------------------------- */

/* Sample n_batches independent mini-batches in one pass.  Batch b has targets
 * targets[target_offsets[b] .. target_offsets[b+1]) (unique, resident node ids; caller order
 * is kept as Delta_k), seed seeds[b].  fanouts[h], h = 0..k-1, is the maximum number of
 * neighbours for the nodes first reached at hop h (h = 0: the targets) — ordered away from
 * the targets.  A node with at most f resident neighbours gets all of them; otherwise f
 * distinct row positions chosen by Floyd's algorithm from Philox4x32-10 words keyed by
 * (seed, node, hop, slot), kept in row order.  Each new delta is the ascending list of
 * unique new neighbours not yet in node_ids (computeNextDelta).
 * `targets` is a host pointer, or a device pointer if targets_on_device; target_offsets,
 * fanouts and seeds are host pointers.  *out: NULL to allocate a new mg_dense, or an
 * existing one (of this context) to reuse its buffers.
 * The call is synchronous: on return the sample is complete and its status checked.  The kernels run
 * on a library-owned sampling stream, ordered after the work queued on the context's stream so far.
 * Errors: MG_ERR_ARG, MG_ERR_STATE, MG_ERR_NONRESIDENT, MG_ERR_DUPLICATE, MG_ERR_CAPACITY,
 * MG_ERR_OOM.
 * Two environment variables switch off a fast path, for diagnosis (the results are the same): MG_NO_SAMPLE_GRAPH
 * (launch the sampler's kernels one by one instead of replaying the captured CUDA graph) and MG_GLOBAL_TABLES
 * (deduplicate the last hop through the id tables in global memory instead of shared memory). */
int mg_sample_many(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                   const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                   int32_t k, const uint64_t* seeds, const mg_sample_caps* caps /*nullable*/,
                   mg_dense** out);

/* The two halves of mg_sample_many, for callers that overlap sampling with other work (the
 * forward pass of the previous group, say).  mg_sample_many_begin queues the whole sample on the
 * library's sampling stream and returns; target_offsets, fanouts and seeds may be reused at once, a
 * device or pinned-host `targets` buffer must stay valid until mg_sample_many_end.  The mg_dense
 * (*out, allocated or reused as in mg_sample_many) must not be used until mg_sample_many_end has
 * waited for the sample and checked its status (same errors as mg_sample_many).  A sample begun into
 * an mg_dense that a forward pass is still reading waits for that pass on the device. */
int mg_sample_many_begin(mg_ctx* ctx, const int32_t* targets, int targets_on_device,
                         const int64_t* target_offsets, int32_t n_batches, const int32_t* fanouts,
                         int32_t k, const uint64_t* seeds, const mg_sample_caps* caps /*nullable*/,
                         mg_dense** out);
int mg_sample_many_end(mg_ctx* ctx, mg_dense* d);

/* One batch: mg_sample_many with n_batches = 1. */
int mg_sample(mg_ctx* ctx, const int32_t* targets, int targets_on_device, int32_t n_targets,
              const int32_t* fanouts, int32_t k, uint64_t seed, const mg_sample_caps* caps,
              mg_dense** out);

/* Sizes of a sample: nodes_per_hop is a HOST array of n_batches * (k+1) entries,
 * [b * (k+1) + h] = |Delta_{k-h}| of batch b; entries_per_hop a HOST array of n_batches * k,
 * [b * k + h] = neighbours sampled for hop h's nodes.  Either may be NULL. */
int mg_dense_counts(const mg_dense* d, int32_t* n_batches, int32_t* k, int64_t* nodes_per_hop,
                    int64_t* entries_per_hop);

/* Materialise batch `batch` in the paper's array layout (Section 4.1 plus repr_map,
 * Section 4.2) into a device buffer owned by `d`.  Ids inside a delta ascend; targets keep the caller's order.
 * On the device a delta is kept in the order in which its nodes were found (nothing on the sample / forward path
 * depends on that order); this call, mg_gather_h0 and mg_layer_output sort the mini-batch's ids (one radix sort per
 * call, on the context's stream, synchronous) and translate rows and repr_map entries. */
int mg_dense_view(mg_ctx* ctx, mg_dense* d, int32_t batch, mg_dense_arrays* out);

/* The canonical DENSE ordering for the whole sample in one pass (Algorithm 1's computeNextDelta leaves every delta
 * as the ascending list of its ids; on the device a delta is kept in the order its nodes were found).
 * mg_dense_export_many queues, on the library's sampling stream, ONE sort of all nodes of all mini-batches by id
 * inside their (mini-batch, delta) segments and the translation of every entry, and returns at once: no host
 * synchronisation, no work per mini-batch.  It overlaps whatever runs on the context's stream (the layers of this or another sample); a later
 * sample into `d` is ordered behind it.  mg_dense_export_view waits for that export (first call only) and hands out
 * mini-batch `batch` of it: the same five arrays as mg_dense_view, bit for bit, as DEVICE pointers into a buffer owned
 * by `d` that holds all mini-batches packed one after the other; valid until the next mg_dense_export_many or
 * mg_sample* on `d`.  The buffer is sized from the sample's capacities (4 x max_nodes_total + 2 x max_entries_total
 * int32) and allocated by the first export of a handle.  Errors: MG_ERR_ARG, MG_ERR_STATE (no completed sample / no
 * export), MG_ERR_CAPACITY (id and row index do not fit one 64-bit sort key), MG_ERR_OOM. */
int mg_dense_export_many(mg_ctx* ctx, mg_dense* d);
int mg_dense_export_view(mg_ctx* ctx, mg_dense* d, int32_t batch, mg_dense_arrays* out);

int mg_dense_free(mg_dense* d);

/* ---- GraphSage forward over DENSE (Section 4.2, Algorithms 2 and 3) -------------------- */

/* k layers of widths dims[0] -> dims[1] -> ... -> dims[k]; w_self[l], w_nbr[l] are HOST
 * row-major [dims[l], dims[l+1]] fp32, bias[l] HOST [dims[l+1]] (copied).  Layer l+1
 * computes act(self . w_self + mean(sampled neighbours) . w_nbr + bias) with ReLU on all
 * but the last layer.  dims must be multiples of 4.
 * MG_GEMM_TF32 with half-precision base representations (MG_DTYPE_F16 table): the first layer's GEMM then runs on fp16
 * operands (the rows as they are, the mean and the weights rounded to fp16: the same 10-bit mantissa as TF32, fp32
 * accumulate), provided the layer's weights sit well inside fp16's range (largest magnitude below 2^15, root mean
 * square above 2^-10) and the mean aggregator is used; otherwise on TF32 operands. */
int mg_model_create(mg_ctx* ctx, int32_t k, const int32_t* dims, const float* const* w_self,
                    const float* const* w_nbr, const float* const* bias, int gemm_precision,
                    mg_model** out);
/* Neighbour aggregator of every layer of the model: MG_AGGR_MEAN (default; GraphSage's mean over the sampled
 * neighbours) or MG_AGGR_SUM (their sum: Algorithm 3 as printed is this layer with identity weights, no bias and no
 * activation).  Takes effect from the next forward call.  Errors: MG_ERR_ARG. */
#define MG_AGGR_MEAN 0
#define MG_AGGR_SUM 1
int mg_model_set_aggregator(mg_model* m, int aggregator);
/* Storage of the intermediate layer outputs H^1 .. H^{k-1} inside mg_forward: MG_DTYPE_F32 (default) or
 * MG_DTYPE_F16.  The tensor-core layers round their inputs to a 10-bit mantissa anyway (TF32); fp16 keeps those bits,
 * so H^k stays within the tensor-core tolerance of the fp32 result, while a layer's output and the next layer's gather
 * move half the bytes in half the memory requests -- but fp16 has a 5-bit exponent: activations beyond 65504 overflow,
 * so this is an option, not the default (the paper stores 4-byte floats).  Takes effect when every layer runs in the
 * fused tensor-core kernel (MG_GEMM_TF32, widths <= 256), the intermediate widths are multiples of 128, the mean
 * aggregator is used, the weights suit fp16 (largest magnitude below 2^15, root mean square above 2^-10) and
 * mg_keep_layer_outputs is off; otherwise the call is accepted and fp32 is used.  Errors: MG_ERR_ARG. */
int mg_model_set_intermediates(mg_model* m, int dtype);
int mg_model_free(mg_model* m);

/* Forward pass for every batch of `d`.  H^0 is read straight from the feature buffer (rows
 * of d's node ids through the partition->slot map); layer l aggregates over the part of
 * DENSE Algorithm 2 would leave after l-1 updates.  `out` receives H^k: one row of dims[k]
 * fp32 per target, batches concatenated, caller's target order; a device pointer, or a host
 * pointer if out_on_device = 0.  Errors: MG_ERR_STATE (no features / sample and model
 * depths differ / feature dim != dims[0]), MG_ERR_OOM. */
int mg_forward(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out, int out_on_device);

/* Schedule of the layers inside mg_forward.  mini_batches = 0: every layer runs over all mini-batches
 * before the next starts, and H^1..H^{k-1} stay available for mg_layer_output.  mini_batches = w > 0: the
 * layers run over windows of w consecutive mini-batches through small reused buffers, so that a layer's
 * output is read back from L2 instead of DRAM; H^k is the same, the intermediate layers are not kept.
 * Only the fused tensor-core layers (MG_GEMM_TF32, widths <= 256) use windows. */
int mg_set_layer_window(mg_ctx* ctx, int32_t mini_batches);
/* enable = 1 forces the whole-layer schedule whatever the window, so that mg_layer_output works. */
int mg_keep_layer_outputs(mg_ctx* ctx, int enable);

/* mg_forward with a HOST output whose device-to-host copy does not block the caller: the kernels are
 * queued on the context's stream, the copy follows them on the library's side stream, and the call
 * returns at once.  out_host should be pinned memory (a pageable buffer makes the copy synchronous)
 * and holds H^k only after mg_wait_output returns MG_OK.  Calls made in between (sampling the next
 * group into another mg_dense) overlap the copy; the next forward on this context waits for it before
 * it reuses the layer workspace. */
int mg_forward_host_async(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out_host);
/* Block until the output copy of the last mg_forward_host_async has finished; reports a tensor-core
 * barrier time-out of that forward as MG_ERR_TIMEOUT. */
int mg_wait_output(mg_ctx* ctx);

/* H^0 of one batch: base representations of its node_ids, rows in the order of
 * mg_dense_view's node_ids, widened to fp32.  out_dev: DEVICE [n_nodes, feature dim]. */
int mg_gather_h0(mg_ctx* ctx, mg_dense* d, int32_t batch, float* out_dev);

/* After mg_forward: H^layer (1..k) of one batch, rows in the order of the paper's node_ids
 * from node_id_offsets[layer] on.  out_dev: DEVICE [rows, dims[layer]]. */
int mg_layer_output(mg_ctx* ctx, const mg_model* m, mg_dense* d, int32_t layer, int32_t batch,
                    float* out_dev);

/* Size of the scratch array built into the library for mg_forward_noalloc.  Every GPU that
 * loads the library holds this much device memory until the process exits. */
#define MG_NOALLOC_SCRATCH_BYTES (16u << 20)

/* mg_forward for callers that must not allocate device memory while they run.  (The paper has
 * no counterpart; this is a service of the library.)  Such callers exist: a serving process
 * whose device memory was handed out in full at start-up, so that a later cudaMalloc fails; a
 * host framework whose caching allocator owns the rest of the GPU; a latency-bound loop that
 * cannot afford the device-wide synchronisation an allocation or a free implies.  mg_forward
 * grows its workspaces with cudaMalloc when a sample is larger than any before it; this entry
 * point never calls cudaMalloc, cudaFree or any allocating routine.  It computes the same H^k
 * with the separate aggregation and GEMM kernels (mg_forward's default for MG_GEMM_TF32 is one
 * fused kernel, so the two agree to the tensor-core tolerance there, not bit for bit), keeping
 * the [self | mean] staging rows (first 4 MiB) and the intermediate layer outputs H^1..H^{k-1}
 * (remaining 12 MiB) in a scratch array of MG_NOALLOC_SCRATCH_BYTES that is part of the library
 * image.  The call is synchronous: it waits for the context's stream before it returns.
 *  - out_dev: DEVICE pointer, one row of dims[k] fp32 per target, as mg_forward writes it.
 *  - Limit: sum over l < k of rows(H^l) * dims[l] * 4 bytes must fit in 12 MiB; larger samples
 *    get MG_ERR_CAPACITY (nothing is launched) — use mg_forward or fewer mini-batches per call.
 *  - The first call on a device looks up the array's device address (cudaGetSymbolAddress);
 *    make that first call before any stream capture begins.  The CUDA runtime may also load
 *    the kernels' code on their first launch, which is memory management of its own: a caller
 *    that needs a steady state free of it makes one warm-up call per model shape first.
 *  - All calls in the process share the one array, and it keeps the previous call's contents.
 *    Nothing in it needs clearing (every value read was written earlier in the same call), but
 *    two calls that overlap on the GPU — from two contexts or two host threads — race on it:
 *    run them one after the other.
 * Other errors as mg_forward. */
int mg_forward_noalloc(mg_ctx* ctx, const mg_model* m, mg_dense* d, float* out_dev);

/* ---- link prediction: shared negatives, target union, DistMult ------------------------ */

/* Prepare a batch of n_edges training edges (HOST int32 src / rel / dst; dst aggregates
 * from src).  Edge i belongs to chunk floor(i * n_chunks / n_edges); chunk c shares
 * negs_per_chunk negatives, negative t being the resident node number
 * mulhi(Philox4x32-10(counter = (c, t, 0xFFFFFFFF, 0), key = seed).word0, #resident nodes)
 * counted in ascending partition order.  The targets of the batch are the ascending unique
 * union of all sources, destinations and negatives.  Errors as mg_sample_many. */
int mg_lp_prepare(mg_ctx* ctx, const int32_t* src, const int32_t* rel, const int32_t* dst,
                  int64_t n_edges, int32_t n_chunks, int32_t negs_per_chunk, uint64_t seed,
                  mg_lp_batch** out);
/* DEVICE pointers owned by the batch: the target ids (ascending), and for each edge /
 * negative its row in the target list.  Any out pointer may be NULL. */
int mg_lp_view(const mg_lp_batch* lp, int32_t* n_targets, const int32_t** targets,
               const int32_t** src_idx, const int32_t** dst_idx, const int32_t** neg_ids,
               const int32_t** neg_idx);
int mg_lp_free(mg_lp_batch* lp);

/* DistMult: pos[i] = sum_d h[s_i,d] rel_emb[r_i,d] h[o_i,d]; neg_dst[i,t] the same with the
 * destination replaced by negative t of edge i's chunk, neg_src[i,t] with the source
 * replaced.  h_dev: DEVICE [n_targets, dim] (mg_forward's output for the batch's targets);
 * rel_emb_dev: DEVICE [n_relations, dim]; outputs DEVICE: pos [n_edges],
 * neg_* [n_edges, negs_per_chunk] (only the sides `corrupt` names are written).  pos is always
 * computed in fp32; the negative scores are a contraction and run on the tensor cores
 * (MG_GEMM_TF32: operands rounded to nearest TF32, fp32 accumulate; needs dim % 4 == 0 and
 * dim <= 128) or on CUDA cores in fp32 (MG_GEMM_FP32, any dim).  The kernels are queued on the
 * context's stream; the call does not wait for them. */
int mg_distmult_score(mg_ctx* ctx, const mg_lp_batch* lp, const float* h_dev, int32_t dim,
                      const float* rel_emb_dev, int32_t n_relations, int corrupt, int gemm_precision,
                      float* pos_out, float* neg_dst_out, float* neg_src_out);

/* ---- instrumentation ------------------------------------------------------------------ */

/* Number of kernels this context has launched since creation. */
int64_t mg_kernel_launches(const mg_ctx* ctx);

/* Per-phase device timing.  While enabled, every group of kernels the library issues is
 * bracketed by CUDA events on the context's stream.  mg_profile_read synchronises the stream
 * and returns, for each phase, its name (static string), the summed milliseconds and the
 * number of kernel launches since the last reset; arrays must hold 32 entries. */
int mg_profile(mg_ctx* ctx, int enable);
int mg_profile_read(mg_ctx* ctx, int32_t* n_phases, const char** names, double* ms, int64_t* launches,
                    int reset);

/* ---- backward pass and optimiser step (Section 3: a mini-batch's gradients update the model and the base
 * representations) ------------------------------------------------------------------------ */

/* Gradients of a scalar loss through the last mg_forward of (m, d), which must have run with
 * mg_keep_layer_outputs(ctx, 1).  d_out_dev (DEVICE): dL/dH^k, one row of dims[k] floats per target, laid out like
 * mg_forward's output.  The weight and bias gradients of every layer are left in buffers owned by the model
 * (mg_model_grads), overwriting those of the previous call.  d_h0_dev (DEVICE, nullable): receives dL/dH^0, one row
 * of dims[0] floats per node of every mini-batch in the library's packed row order -- mg_dense_packed_ids gives the
 * node id of each row -- i.e. the gradient rows of the base representations.  fp32 arithmetic; sums over rows use
 * atomic adds (low-order bits vary from run to run).  Synchronous.  Errors: MG_ERR_ARG, MG_ERR_STATE (no matching
 * forward pass, layers not kept), MG_ERR_OOM. */
int mg_backward(mg_ctx* ctx, mg_model* m, mg_dense* d, const float* d_out_dev, float* d_h0_dev);

/* DEVICE pointers to the gradients mg_backward left for layer `layer` (1..k): d_w_self and d_w_nbr row-major
 * [dims[layer-1], dims[layer]], d_bias [dims[layer]].  Owned by the model.  Errors: MG_ERR_ARG, MG_ERR_STATE. */
int mg_model_grads(const mg_model* m, int32_t layer, const float** d_w_self, const float** d_w_nbr, const float** d_bias);

/* One step of stochastic gradient descent on every weight and bias of the model with the gradients of the last
 * mg_backward: w -= lr * dw.  Refreshes the copies the forward kernels read.  Synchronous. */
int mg_model_sgd_step(mg_ctx* ctx, mg_model* m, float lr);

/* One Adagrad step with the gradients of the last mg_backward: state += g^2 (state starts at zero with the first
 * call), w -= lr * g / (sqrt(state) + eps), for every weight and bias.  Synchronous.  Errors: MG_ERR_ARG, MG_ERR_STATE,
 * MG_ERR_OOM. */
int mg_model_adagrad_step(mg_ctx* ctx, mg_model* m, float lr, float eps);

/* One SGD step on the base representations of the sample's nodes, in the partition buffer: row(node) -= lr * its
 * gradient row(s) of d_h0_dev (as written by mg_backward; a node of several mini-batches receives all of its rows).
 * fp32 tables only.  With host backing the table handed to mg_load_features must be writable: a partition updated
 * here is copied back to it when mg_set_resident evicts it (side stream, before its slot is reused); partitions
 * still resident hold the only current copy.  With HBM backing the caller's device table is updated in place.
 * Synchronous.  Errors: MG_ERR_ARG, MG_ERR_STATE. */
int mg_apply_embedding_sgd(mg_ctx* ctx, mg_dense* d, const float* d_h0_dev, float lr);

/* ids_dev (DEVICE, int32, one per node of every mini-batch = the rows of H^0 in the library's packed order: batch
 * after batch, targets first, then delta after delta in the order the nodes were found): the node id of each row. */
int mg_dense_packed_ids(mg_ctx* ctx, mg_dense* d, int32_t* ids_dev);

/* ---- graph attention over DENSE (the GAT model of Section 7.1) --------------------------- */

typedef struct mg_gat_model mg_gat_model;

/* k single-head attention layers of widths dims[0] -> ... -> dims[k] (multiples of 4; dims[1..k] <= 512).  Layer l + 1:
 * z = h w[l] for every input row; for an output row i with sampled neighbours j (repeats count) and itself,
 * e_ij = LeakyReLU(a_dst[l] . z_i + a_src[l] . z_j) with slope negative_slope, alpha = softmax over {i} + neighbours,
 * h'_i = sum alpha_ij z_j + bias[l]; ReLU on all but the last layer; a node without neighbours attends to itself.
 * w[l] HOST row-major [dims[l], dims[l+1]]; a_src[l], a_dst[l], bias[l] HOST [dims[l+1]] (all copied).
 * gemm_precision as in mg_model_create.  Errors: MG_ERR_ARG, MG_ERR_OOM. */
int mg_gat_model_create(mg_ctx* ctx, int32_t k, const int32_t* dims, const float* const* w, const float* const* a_src,
                        const float* const* a_dst, const float* const* bias, float negative_slope, int gemm_precision,
                        mg_gat_model** out);
/* Attention heads of every layer of the model (1 .. 8; default 1): the columns of z, a_src and a_dst are cut into
 * `heads` equal blocks, every block attends on its own (its own scores and softmax), the blocks' results are
 * concatenated, so a layer's width stays dims[l + 1], which must be a multiple of `heads`.  Errors: MG_ERR_ARG. */
int mg_gat_model_set_heads(mg_gat_model* m, int32_t heads);
int mg_gat_model_free(mg_gat_model* m);

/* Attention forward pass for every batch of `d`; out_dev (DEVICE) receives one row of dims[k] floats per target, batch
 * after batch in the caller's target order.  Synchronous on the context's stream.  Errors as mg_forward. */
int mg_gat_forward(mg_ctx* ctx, const mg_gat_model* m, mg_dense* d, float* out_dev);

/* ---- COMET: partition replacement for link prediction out of core (Section 5.1, Section 6) ----
 * Host-side planning only; no context, no device work.  Partition ids are the physical partitions of
 * mg_set_partitioning; a plan's sets drive mg_set_resident, its bucket table says which set trains edge bucket
 * (i, j) = the edges from physical partition i to physical partition j. */

/* One epoch's plan.  p physical partitions are grouped at random into l logical ones (p a multiple of l):
 * logical_of_physical[p] (out).  The sequence of resident sets swaps ONE logical partition at a time, greedily by the
 * number of partition pairs that share a set for the first time, until every pair has: sets (out) holds n_sets rows
 * of c_l logical ids in buffer-slot order (a swap puts the new partition into the slot of the one it replaces;
 * row 0 = 0 .. c_l - 1), at most cap_sets rows.  bucket_set[p * p] (out): for each edge bucket a set chosen
 * uniformly among those that hold both of its partitions (deferred, randomised processing of training examples).
 * All randomness is Philox keyed by `seed`.  Errors: MG_ERR_ARG (null pointer, p not a positive multiple of l, not
 * 2 <= c_l <= l), MG_ERR_CAPACITY (more than cap_sets sets; l * l rows always suffice). */
int mg_comet_plan(int32_t p, int32_t l, int32_t c_l, uint64_t seed, int32_t cap_sets, int32_t* logical_of_physical,
                  int32_t* n_sets, int32_t* sets, int32_t* bucket_set);

/* Edge Permutation Bias B of a bucket assignment (Section 6) under the uniform-degree assumption: every node of a
 * physical partition shares one tally, bucket (i, j) counts once for i and once for j, tallies are normalised by
 * their final value; B = max over sets of (largest - smallest tally).  Errors: MG_ERR_ARG. */
int mg_comet_bias(int32_t p, int32_t n_sets, const int32_t* bucket_set, double* bias);

/* The rules of Section 6: p = floor(min(NO / D, sqrt(EO / D))) (NO = n_nodes * dim * 4, EO = n_edges *
 * bytes_per_edge, D = block_bytes), clamped to [2, max_parts]; c = the largest even buffer capacity with
 * c * NO / p + 2 * c^2 * EO / p^2 + fudge_bytes < cpu_bytes whose half divides p (two logical partitions fill the
 * buffer); l = 2 p / c.  Errors: MG_ERR_ARG, MG_ERR_CAPACITY when no capacity fits. */
int mg_comet_autotune(int64_t n_nodes, int32_t dim, int64_t n_edges, int32_t bytes_per_edge, int64_t cpu_bytes,
                      int64_t block_bytes, int64_t fudge_bytes, int32_t max_parts, int32_t* p, int32_t* l, int32_t* c);

#ifdef __cplusplus
}
#endif
#endif /* MGDENSE_H */
