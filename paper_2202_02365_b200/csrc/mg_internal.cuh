// Internal declarations shared by the translation units of libmgdense.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "mgdense.h"
#include "mg_device.cuh"

// ---------------------------------------------------------------------------------------
// status word written by kernels (never a trap): bit flags, read by the host after a call
// ---------------------------------------------------------------------------------------
enum : uint32_t {
    ST_RANGE = 1u,         // target id outside [0, n_nodes)
    ST_NONRESIDENT = 2u,   // target in a non-resident partition
    ST_DUPLICATE = 4u,     // same target twice in a batch
    ST_CAP_ENTRIES = 8u,   // neighbour arena too small
    ST_CAP_NODES = 16u,    // node arena too small
    ST_CAP_TABLE = 32u,    // per-batch id table full (max_nodes_per_batch too small)
    ST_INTERNAL = 64u,     // an invariant did not hold (bug guard; access skipped)
};

// Device-side header of a sample: counters every kernel sizes itself from.
struct DenseHeader {
    uint32_t status;
    uint32_t n_new;                       // length of the new-node list of the current hop
    int32_t hop_base[MG_MAX_HOPS + 2];    // node arena: hop h occupies [hop_base[h], hop_base[h+1])
    int32_t ent_base[MG_MAX_HOPS + 1];    // entry arena: hop h occupies [ent_base[h], ent_base[h+1])
    int32_t rows_total[MG_MAX_HOPS + 1];  // rows of H^l summed over batches, l = 0..k
};

struct ProfPhase {
    const char* name;
    double ms;
    int64_t launches;
};

enum {
    PH_SAMPLE_INIT = 0,
    PH_SAMPLE_COUNT,
    PH_SAMPLE_SCAN,
    PH_SAMPLE_PICK,
    PH_SAMPLE_SORT,
    PH_SAMPLE_PLACE,
    PH_SAMPLE_RELABEL,
    PH_SAMPLE_FINAL,
    PH_AGG_L1,
    PH_AGG_REST,
    PH_GEMM,
    PH_DISTMULT,
    PH_OTHER,
    PH_COUNT
};

struct mg_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    cudaStream_t side = nullptr;  // partition swaps, asynchronous output copies
    cudaStream_t sample_stream = nullptr;  // all sampling kernels
    cudaEvent_t ev_user = nullptr;
    std::string err;
    int64_t launches = 0;
    int n_sms = 148;
    uint32_t* d_flags = nullptr;  // device word the tensor-core GEMM reports a barrier time-out in

    // graph store (device)
    int64_t n_nodes = 0, n_edges = 0;
    int64_t* row_off = nullptr;  // [n_nodes + 1]
    int32_t* nbrs = nullptr;     // [n_edges]
    // in-buffer view (device); equal to the store when everything is resident
    int64_t* view_off = nullptr;
    int32_t* view_nbrs = nullptr;
    int64_t view_edges = 0;
    bool view_owned = false;
    char* view_ws = nullptr; size_t view_ws_bytes = 0;   // scratch of the view rebuild (keep bits, prefixes, tile bases)
    // second edge list (rows by source) and its in-buffer view; sample_inout = draw from both lists
    int64_t n_edges_out = 0;
    int64_t* row_off_out = nullptr;
    int32_t* nbrs_out = nullptr;
    int64_t* view_off_out = nullptr;
    int32_t* view_nbrs_out = nullptr;
    int64_t view_edges_out = 0;
    bool view_out_owned = false;
    bool sample_inout = false;

    // partitioning and buffer
    int32_t n_parts = 1;
    int64_t part_size = 0;
    int32_t capacity = 1;
    std::vector<int32_t> slot_of_part;  // committed; -1 = not resident
    std::vector<int32_t> pending_slot;  // after set_resident, before commit
    uint64_t resident_serial = 0;       // bumped whenever the committed slot map or the slots themselves change
    bool has_pending = false;
    std::vector<cudaEvent_t> pending_events;
    std::vector<char> dirty_part;       // host backing: the partition's slot was updated (mg_apply_embedding_sgd) and not written back yet
    // partition-id array (mg_set_partitioning with part_of_node): null for contiguous equal ranges
    uint8_t* d_part_of_node = nullptr;    // [n_nodes]
    int32_t* d_local_of_node = nullptr;   // [n_nodes] rank of the node inside its partition (ascending id)
    int32_t* d_nodes_by_part = nullptr;   // [n_nodes] node ids partition after partition, ascending inside a partition
    std::vector<int64_t> part_count, part_start;   // population of each partition; first row of its block in a partition-major table
    int32_t* d_slot_of_part = nullptr;   // [MG_MAX_PARTS]
    int64_t* d_res_prefix = nullptr;     // [MG_MAX_PARTS + 1] resident-node prefix counts
    int64_t* d_part_start = nullptr;     // [MG_MAX_PARTS + 1] first row of each partition's block (prefix of the populations)
    int64_t n_resident_nodes = 0;

    // features
    int feat_dtype = MG_DTYPE_F32;
    int32_t feat_dim = 0;
    int backing = MG_BACKING_HBM;
    const char* host_table = nullptr;  // MG_BACKING_HOST (may be null: then every partition needs a source of its own)
    std::vector<const char*> part_source;  // MG_BACKING_HOST: host block of a partition when it is not at its place in host_table
    char* slots = nullptr;             // device: slot s at slots + s * slot_bytes
    bool slots_owned = false;
    int32_t n_slots = 0;
    int64_t slot_bytes = 0;
    int64_t row_bytes = 0;

    // forward workspaces (grown on demand)
    float* ws_x = nullptr; size_t ws_x_bytes = 0;
    float* ws_h[2] = {nullptr, nullptr}; size_t ws_h_bytes[2] = {0, 0};
    float** ws_layer = nullptr;

    // forward schedule
    int32_t layer_window_batches = 0;  // mini-batches per window of the layer schedule; 0 = whole layers
    bool keep_layers = false;          // keep H^1..H^{k-1} for mg_layer_output (whole-layer schedule)
    bool layers_kept = false;          // what the last forward did

    // asynchronous output copy of mg_forward_host_async
    cudaEvent_t ev_fwd_done = nullptr, ev_out_done = nullptr;
    bool out_check_gemm = false;
    // H^k goes to one of two buffers in turn, so that a forward pass need not wait for the copy of the previous
    // pass's output to the host
    float* hk_buf[2] = {nullptr, nullptr};
    size_t hk_elems[2] = {0, 0};
    cudaEvent_t ev_hk_done[2] = {nullptr, nullptr};
    bool hk_pending[2] = {false, false};
    int hk_cur = 0;
    const float* last_hk = nullptr;

    // profiling
    // link-prediction batches: scratch of mg_lp_prepare (grows, never shrinks) and one spare result block, so that a
    // loop of prepare / free allocates nothing
    char* lp_ws = nullptr; size_t lp_ws_bytes = 0;
    char* lp_spare = nullptr; size_t lp_spare_bytes = 0;
    int32_t* lp_words = nullptr;       // mapped pinned host words {status, n_targets} that mg_lp_prepare's last kernel writes
    int32_t* lp_words_dev = nullptr;   // their device address
    int32_t* lp_range = nullptr;       // device {0, 32-word groups of the node bitmap}: the bounds of mg_lp_prepare's scan
    int64_t lp_range_words = -1;
    float* gat_x = nullptr; float* gat_z = nullptr; float* gat_s = nullptr; float* gat_h[2] = {nullptr, nullptr};   // mg_gat_forward scratch
    size_t gat_x_elems = 0, gat_z_elems = 0, gat_s_elems = 0, gat_h_elems[2] = {0, 0};
    const struct mg_model* last_fwd_model = nullptr; const struct mg_dense* last_fwd_dense = nullptr;   // what mg_backward may follow
    float* bw_g = nullptr; float* bw_x = nullptr; float* bw_dx = nullptr;   // mg_backward scratch
    size_t bw_g_elems = 0, bw_x_elems = 0, bw_dx_elems = 0;
    uint32_t* bw_off = nullptr; int2* bw_rev = nullptr;   // mg_backward: the turned-round entries of a layer
    size_t bw_off_elems = 0, bw_rev_elems = 0;
    char* dm_images = nullptr; size_t dm_images_bytes = 0;   // TF32 operand images of the negatives (mg_distmult_score)
    bool prof_on = false;
    bool sample_graphs = true;   // replay the sampler's launches from a CUDA graph
    ProfPhase prof[PH_COUNT];
    std::vector<std::pair<int, std::pair<cudaEvent_t, cudaEvent_t>>> prof_pending;
};

// everything the sampler's captured device work depends on
struct SampleSignature {
    int32_t B, k, table_size, fanouts[MG_MAX_HOPS];
    int64_t T, cap_batch, cap_nodes, cap_entries, n_nodes, part_size, inout;
    const void* ptrs[32];
};

struct mg_dense {
    mg_ctx* ctx = nullptr;
    int device = 0;
    int32_t k = 0, n_batches = 0;
    int32_t fanouts[MG_MAX_HOPS] = {0};
    int64_t cap_nodes = 0, cap_entries = 0;
    int32_t table_size = 0;  // slots per batch, power of two
    int64_t n_targets_total = 0;

    // device arrays
    DenseHeader* hdr = nullptr;
    int32_t* nodes = nullptr;       // [cap_nodes] hop-major, batch-major inside a hop
    int32_t* node_batch = nullptr;  // [cap_nodes]
    int32_t* ent_off = nullptr;     // [cap_nodes + 1] start of each sampled node's entries
    int64_t* node_r0 = nullptr;     // [cap_nodes] start of the node's row in the in-buffer view
    uint32_t* node_deg = nullptr;   // [cap_nodes] its (resident) degree
    int64_t* node_r0_out = nullptr; // the same for the outgoing edge list (incoming + outgoing sampling only)
    uint32_t* node_deg_out = nullptr;
    int64_t cap_nodes_out = 0;
    int2* pairs = nullptr;          // last hop, shared-memory deduplication: (id, entry) grouped by (batch, share, bucket)
    int32_t* share_off = nullptr;   // its group bounds
    int64_t cap_pairs = 0, cap_share = 0;
    int32_t* ent_nbrs = nullptr;    // [cap_entries] neighbour ids
    int32_t* ent_repr = nullptr;    // [cap_entries] neighbour's local row in its batch
    int32_t* node_off = nullptr;    // [(k+1) * (B+1)] arena index where batch b's hop-h nodes start
    int32_t* cum = nullptr;         // [B * (k+2)] local row of the first node of hop h; [k+1] = V
    int32_t* rowbase = nullptr;     // [(k+1) * (B+1)] first packed row of batch b in H^l
    int32_t* hkeys = nullptr;       // [B * table_size]
    int32_t* hvals = nullptr;       // [B * table_size]
    uint64_t* newlist[2] = {nullptr, nullptr};  // [cap_nodes] composite keys
    uint64_t* d_seeds = nullptr;    // [B]
    int32_t* scan_tmp = nullptr;    // block sums
    uint32_t* sort_hist = nullptr;  // radix histograms
    size_t scan_tmp_elems = 0, sort_hist_elems = 0;
    void* seg_tiles = nullptr;      // tile table of the export's sort inside (mini-batch, delta) segments
    int64_t cap_sort_tiles = 0;     // tiles the sort scratch (histograms, block sums, tile table) is sized for
    int64_t alloc_batches = 0, alloc_table = 0;

    // export buffer for mg_dense_view
    int32_t* exp_buf = nullptr; size_t exp_elems = 0;

    // host mirror
    DenseHeader h_hdr;
    std::vector<int32_t> h_cum;      // [B * (k+2)]
    std::vector<int32_t> h_node_off; // [(k+1) * (B+1)]
    std::vector<int32_t> h_rowbase;  // [(k+1) * (B+1)]
    std::vector<int32_t> h_ent_hop;  // [k * (B+1)] arena entry index where batch b's hop-h entries start
    int32_t* d_ent_hop = nullptr;    // device copy of the same
    bool valid = false;
    // the slot map the sample was drawn under: its feature rows are addressed through it, so a later call may only
    // use the sample while every partition resident then still sits in the same slot
    uint64_t resident_serial = 0;
    std::vector<int32_t> slot_of_part_at_sample;
    // export of all mini-batches at once (mg_dense_export_many): one buffer, laid out by export_layout()
    int32_t* expm_buf = nullptr; size_t expm_elems = 0;
    cudaEvent_t ev_exported = nullptr;
    bool export_valid = false, export_pending = false;
    int32_t* perm_buf = nullptr; size_t perm_elems = 0;   // perm | inv of mini-batch perm_batch (mg_dense_batch_perm)
    int perm_batch = -1;
    uint32_t* batch_cnt = nullptr;   // [k][B] new nodes per hop and mini-batch
    // asynchronous sampling: the summary lands in pinned memory, ev_sampled marks its arrival
    int32_t* h_pinned = nullptr; size_t h_pinned_ints = 0;
    int32_t* h_pinned_dev = nullptr; // the same memory as the device sees it
    int32_t* h_stage = nullptr; size_t h_stage_ints = 0;   // pinned, mapped: header, offsets, seeds of the call being queued
    int32_t* h_stage_dev = nullptr;                        // the same memory as the device sees it
    cudaGraphExec_t graph_exec = nullptr;                 // the sampler's device work for graph_sig
    SampleSignature graph_sig;
    int64_t graph_launches = 0;
    cudaEvent_t ev_sampled = nullptr;
    cudaEvent_t ev_read_done = nullptr;  // recorded after the last kernel that read this sample
    bool pending = false;
};

struct mg_model {
    mg_ctx* ctx = nullptr;
    int device = 0;
    int32_t k = 0;
    int32_t dims[MG_MAX_HOPS + 1] = {0};
    int precision = MG_GEMM_TF32;
    bool sum_aggr = false;   // neighbour term: sum instead of mean (Algorithm 3 as printed)
    float* w_cat[MG_MAX_HOPS] = {nullptr};  // device [2*d_in, d_out]: rows 0..d_in-1 self, then neighbour
    float* w_cat_t[MG_MAX_HOPS] = {nullptr}; // device [d_out, 2*d_in] (K-major copy for the tensor-core path)
    float* w_pad_t[MG_MAX_HOPS] = {nullptr}; // device [d_out, 2*roundup32(d_in)], zero padded, for the fused layer kernel
    // device fp16 [dims[l+1], 2*roundup64(dims[l])]: a layer's weights for fp16 operands (layer 1 over fp16 base
    // representations, later layers over fp16 intermediate outputs); null when the weights do not suit fp16
    void* w_pad_h[MG_MAX_HOPS] = {nullptr};
    bool f16_intermediates = false;   // store H^1 .. H^{k-1} as fp16 (mg_model_set_intermediates)
    float* bias[MG_MAX_HOPS] = {nullptr};
    // mg_backward: gradients of w_cat and bias (allocated by the first backward pass), a zero vector
    float* g_w_cat[MG_MAX_HOPS] = {nullptr};
    float* g_bias[MG_MAX_HOPS] = {nullptr};
    float* s_w_cat[MG_MAX_HOPS] = {nullptr};   // Adagrad: accumulated squared gradients
    float* s_bias[MG_MAX_HOPS] = {nullptr};
    float* zeros = nullptr;
};

struct mg_lp_batch {
    mg_ctx* ctx = nullptr;
    int device = 0;
    int64_t n_edges = 0;
    int32_t n_chunks = 0, negs = 0, n_targets = 0;
    int32_t* targets = nullptr;  // device
    int32_t* src_idx = nullptr;
    int32_t* dst_idx = nullptr;
    int32_t* rel = nullptr;
    int32_t* neg_ids = nullptr;
    int32_t* neg_idx = nullptr;
    char* block = nullptr;       // the one device allocation the six arrays above live in
    size_t block_bytes = 0;
};

// ---------------------------------------------------------------------------------------
// host helpers
// ---------------------------------------------------------------------------------------
int mg_fail(mg_ctx* ctx, int code, const char* fmt, ...);
// MG_OK when the partitions that were resident while `d` was sampled are still resident in the same slots (the
// sample's feature rows are then where its ids say); MG_ERR_STATE otherwise.  Host-side check, no device work.
int mg_check_sample_residency(mg_ctx* ctx, const mg_dense* d);
int mg_cuda_fail(mg_ctx* ctx, cudaError_t e, const char* what);

#define MG_CUDA(ctx, call)                                      \
    do {                                                        \
        cudaError_t e__ = (call);                               \
        if (e__ != cudaSuccess) return mg_cuda_fail(ctx, e__, #call); \
    } while (0)

// grow-only device buffer
template <typename T>
static inline int mg_ensure(mg_ctx* ctx, T** ptr, size_t* have_elems, size_t need_elems) {
    if (*ptr && *have_elems >= need_elems) return MG_OK;
    if (*ptr) cudaFree(*ptr);
    *ptr = nullptr;
    *have_elems = 0;
    if (need_elems == 0) need_elems = 1;
    cudaError_t e = cudaMalloc((void**)ptr, need_elems * sizeof(T));
    if (e != cudaSuccess) {
        cudaGetLastError();
        return mg_fail(ctx, MG_ERR_OOM, "device allocation of %zu bytes failed", need_elems * sizeof(T));
    }
    *have_elems = need_elems;
    return MG_OK;
}

void mg_prof_begin(mg_ctx* ctx, int phase);
void mg_prof_end(mg_ctx* ctx, int phase, int n_launches);

struct ProfScope {
    mg_ctx* c; int ph; int n;
    ProfScope(mg_ctx* ctx, int phase, int launches) : c(ctx), ph(phase), n(launches) { mg_prof_begin(c, ph); }
    ~ProfScope() { mg_prof_end(c, ph, n); }
};

static inline int mg_grid(const mg_ctx* ctx, int ctas_per_sm) { return ctx->n_sms * ctas_per_sm; }

// how kernels find a node's partition and its row in the feature buffer
static inline FeatGeom mg_feat_geom(const mg_ctx* ctx) {
    FeatGeom g;
    g.slot_of_part = ctx->d_slot_of_part;
    g.part_of_node = ctx->d_part_of_node;
    g.local_of_node = ctx->d_local_of_node;
    g.part_size = (uint32_t)ctx->part_size;
    g.identity = ctx->backing == MG_BACKING_HBM ? 1 : 0;   // the whole table in device memory, in node order
    return g;
}

// ---- generic device-sized scan and sort (mg_sample.cu) -------------------------------------
struct SortParams {   // device-resident
    int32_t zero;
    int32_t n;        // keys
    int32_t ntiles;   // ceil(n / 4096)
    int32_t hist_len; // bins * ntiles
};
size_t mg_sort_hist_elems(int64_t max_keys);
void mg_sort_params_host(SortParams* sp, int64_t n);
// The device keeps every delta in discovery order; exports go through a permutation of the mini-batch's local rows
// (perm[c] = local row of canonical row c: deltas in the paper's order, ids ascending inside a delta, targets in the
// caller's order; inv = its inverse).  Device arrays owned by d; on ctx->stream, synchronous, off the hot path.
int mg_dense_batch_perm(mg_ctx* ctx, mg_dense* d, int b, const int32_t** perm, const int32_t** inv);
size_t mg_scan_tmp_elems(int64_t max_elems);
void mg_sort_u64(mg_ctx* ctx, uint64_t* const buf[2], const SortParams* sp, int lo_bit, int bits, uint32_t* hist,
                 uint32_t* scan_tmp, int* res_buf, const void* seg_tiles = nullptr);
void mg_scan_u32(mg_ctx* ctx, uint32_t* data, const int32_t* lo, const int32_t* hi, const int32_t* base,
                 uint32_t* scan_tmp, uint32_t* total_out);
