/*
 * rmuscle.h -- C ABI of the activation-masked gated MLP of a diffusion action expert (the compute side of the
 * paper's Action Cache, Sec. 4.1 "Action Cache", Eq. 1 and Eq. 4), implemented as CUDA kernels for sm_100a.
 *
 * Notation (paper / this header): L layers, H model width, I intermediate neurons per layer, T tokens per
 * episode, B independent episodes per call, S_l the active neuron set of layer l (the mask M stored as indices),
 * K_l = |S_l|.  bf16 tensors are passed as raw 2-byte elements.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  The caller allocates and owns every
 *     buffer, including packed weights and workspace; the library allocates only its small context in rm_create.
 *   - Device buffers must be 16-byte aligned (RM_ERR_ALIGN otherwise).  Inputs are never written.
 *   - `stream` is a cudaStream_t passed as void*.  All work is enqueued on it; no call synchronises the host
 *     unless its comment says so.  Argument validation is synchronous and returns a negative rm_status.
 *   - Conditions detected on the device (index >= I, count > stride) never trap: the kernel clamps or skips,
 *     records the code in the context's status word, and rm_device_status reports it.
 *   - Index lists are strictly ascending int32.  The number of valid entries is read from DEVICE memory, so a
 *     list built by rm_mask_compact can be consumed without a host round trip.  A count of 0 is legal.
 */
#ifndef RMUSCLE_H
#define RMUSCLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rm_ctx rm_ctx;      /* opaque */
typedef void* rm_stream_t;         /* a cudaStream_t */

typedef enum {
    RM_OK = 0,
    RM_ERR_INVALID_ARG = -1,       /* NULL where a pointer is required, negative size, bad enum           */
    RM_ERR_SHAPE = -2,             /* size outside what the context was created for                       */
    RM_ERR_ALIGN = -3,             /* a device pointer is not 16-byte aligned                             */
    RM_ERR_WORKSPACE = -4,         /* workspace NULL or smaller than rm_workspace_bytes                   */
    RM_ERR_CUDA = -5,              /* a CUDA runtime call failed (launch error, no device)                */
    RM_ERR_INDEX = -6,             /* device status: a neuron index was out of range or count > stride    */
    RM_ERR_TIMEOUT = -7,           /* device status: a bounded wait expired                               */
    RM_ERR_UNSUPPORTED = -8        /* valid request that this build does not implement                    */
} rm_status;

enum { RM_ACT_GELU_TANH = 0 };     /* the gated unit's activation (Eq. 1 takes it after the GeGLU)     */

/* Model geometry fixed at context creation.  H must be a multiple of 64, I >= 1, L >= 1.
 * T_max / B_max bound the T and B of later calls (they size rm_workspace_bytes). */
typedef struct {
    int32_t L, H, I, T_max, B_max;
    int32_t act;                   /* RM_ACT_GELU_TANH */
} rm_model_desc;

/* Creates a context on the CURRENT CUDA device.  Allocates a few hundred bytes of device memory (the status
 * word and per-call parameter blocks).  Host-synchronous.  *out is NULL on failure. */
int rm_create(rm_ctx** out, const rm_model_desc* desc);
int rm_destroy(rm_ctx* ctx);

/* Bytes of one layer in the library's private neuron-major layout (3*H bf16 per neuron: the neuron's gate row,
 * up row and down column stored next to one another so that one active neuron is one contiguous read). */
size_t rm_packed_layer_bytes(const rm_ctx* ctx);

/* Bytes of scratch that rm_sparse_mlp / rm_action_expert_step need for B episodes of T tokens. */
size_t rm_workspace_bytes(const rm_ctx* ctx, int B, int T);

/* One-off repacking of a layer (not on the timed path).
 *   Wg, Wu [I,H] bf16 row-major (row n = neuron n);  Wd [H,I] bf16 row-major (column n = neuron n).
 *   packed_out: rm_packed_layer_bytes bytes.  down_colnorm (nullable) [I] fp32 receives ||Wd[:,n]||_2, the weight
 *   factor of the contribution score (Eq. 1). */
int rm_pack_weights(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, void* packed_out,
                    float* down_colnorm, rm_stream_t stream);

/* ---- rm_mask_compact: important-neuron selection (Sec. 3.4 Eq. 1 ranking; Sec. 5 "Constructing Group Neuron
 * Masks": K_l = ceil(rho_n * I) is computed by the caller and passed as k). */
enum { RM_SRC_BOOL_U8 = 0,         /* records are uint8 [n_lists, I]; nonzero = selected                  */
       RM_SRC_SCORE_F32 = 1 };     /* records are fp32 activation records [n_lists, I]                    */
enum { RM_REDUCE_NONE = 0,         /* boolean source only                                                 */
       RM_REDUCE_THRESHOLD = 1,    /* score > threshold (strict)                                          */
       RM_REDUCE_TOPK = 2,         /* the k largest scores; equal scores: lower index first               */
       RM_REDUCE_GROUP = 3 };      /* union of the records' top-k sets, ranked by the fp32 sum of the
                                      records' scores (added in record order), top k kept                 */
typedef struct {
    int32_t kind;                  /* RM_SRC_*                                                            */
    int32_t reduce;                /* RM_REDUCE_*                                                         */
    float   threshold;
    int32_t k;
    int32_t n_records;             /* W >= 1 (at most 16) records per list                                */
    int32_t min_votes;             /* a neuron is kept when >= min_votes of the W per-record sets hold it
                                      (1 = union, W = intersection); ignored by RM_REDUCE_GROUP           */
    const void* const* records;    /* HOST array of W device pointers, each [n_lists, I]                  */
    const float* scale;            /* nullable; score = record * scale (one fp32 multiply)                */
    int32_t scale_per_list;        /* 0: scale is [I];  1: scale is [n_lists, I]                          */
    int32_t n_lists;
    int32_t I;
} rm_mask_src;

/* Writes, for every list, the selected indices in ascending order to idx_out[list*stride ...] and their number
 * to count_out[list] (both device).  stride >= I is always sufficient; a list longer than stride is truncated
 * and RM_ERR_INDEX is recorded.  Float ordering: -0 == +0, NaN ranks below every number. */
int rm_mask_compact(rm_ctx* ctx, const rm_mask_src* src, int32_t* idx_out, int32_t* count_out, int64_t stride,
                    rm_stream_t stream);

/* ---- rm_gather_weights: the paper's own preparation of the selected weights (Sec. 4.1, last
 * paragraph: the rows a group's mask selects are copied once into compact buffers that all steps of the group read;
 * Sec. 5 "Overlapping Retrieval and Weight Gathering"), as a comparison variant to gathering inside the products.
 * Copies the packed rows of the listed neurons to the front of compact_out: compact row p = packed row idx[p] for
 * p < count; the rows from count up to the next multiple of 64 (where the buffer has them) are cleared, because a
 * kernel may fetch the last 64-neuron tile whole and multiply its unused rows by zero -- a compact layer built by
 * other means must hold finite values there too.  compact_out holds at least min(list_cap, I) rows of 3*H bf16 (rm_packed_layer_bytes is always enough) and is itself a packed layer: pass it to
 * rm_sparse_mlp / rm_action_expert_step with idx = NULL and the same count_dev (the leading count neurons), and the
 * result is the masked layer over the listed neurons.  Activation records and anchor activations of such a call are
 * indexed by compact position.  Call it on a side stream to overlap it with other work; ordering is the caller's. */
int rm_gather_weights(rm_ctx* ctx, const void* packed_layer, const int32_t* idx, const int32_t* count_dev,
                      int64_t list_cap, void* compact_out, rm_stream_t stream);

/* ---- rm_sparse_mlp: one layer, zero-fill form of the masked evaluation (Sec. 4.1: hidden activations are computed
 * for the selected neurons only, and only their down-projection columns update the output):
 *     y[t,:] = residual[t,:] + sum_{n in S} gelu_tanh(<x_t, Wg_n>) * <x_t, Wu_n> * Wd[:,n]
 *   packed_layer: output of rm_pack_weights.   x [T,H] bf16.   residual [T,H] fp32, nullable (=> 0).
 *   idx [>= count] int32 ascending, nullable => every neuron (dense);  count_dev [1] int32 on the device.
 *   idx NULL with count_dev given: the leading count neurons of the layer (a compact layer from rm_gather_weights).
 *   y [T,H] fp32; may equal residual (in place).
 *   record_out (nullable) [I] fp32: dense mode only; receives A[n] = sum_t |h[t,n]| (* record_scale[n] when
 *   record_scale is given) -- the activation part of Eq. 1, or Eq. 1 itself with record_scale = down_colnorm.
 *   ws / ws_bytes: scratch of at least rm_workspace_bytes(ctx, 1, T). */
int rm_sparse_mlp(rm_ctx* ctx, const void* packed_layer, const void* x, const float* residual,
                  const int32_t* idx, const int32_t* count_dev, float* y, float* record_out,
                  const float* record_scale, int T, void* ws, size_t ws_bytes, rm_stream_t stream);

/* ---- rm_action_expert_step: the L-layer stack for one denoising step of B independent episodes, with masks
 * reused from an earlier step (Sec. 4.1 "Group-Shared Neuron Masks"):
 *     r_0 = r_in;  x_l = bf16(r_l / sqrt(mean_k r_l[t,k]^2 + 1e-6));  r_{l+1} = r_l + MLP_l(x_l; S_l);  r_out = r_L
 *   The residual stream stays fp32.  Attention, conditioning and the adaptive gate are not part of this path.
 *   packed_layers: HOST array of L device pointers.   r_in, r_out [B,T,H] fp32 (r_out may equal r_in).
 *   idx [B,L,stride] int32, nullable => dense;  count_dev [B,L] int32 (device); idx NULL with count_dev given:
 *   layer l of episode b uses the leading count_dev[b,l] neurons of packed_layers[l] (compact layers).
 *   records_out (nullable, dense only) [B,L,I] fp32;  record_scale (nullable) [L,I] fp32. */
int rm_action_expert_step(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                          const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                          const float* record_scale, int B, int T, void* ws, size_t ws_bytes, rm_stream_t stream);

/* The same step for callers whose activations live in HOST memory: copies r_in_host [B,T,H] fp32 to the device,
 * runs the step, copies the result to r_out_host and waits for the stream (host-synchronous).  Pinned host
 * memory makes the copies asynchronous with respect to other streams.  Needs rm_workspace_bytes(ctx,B,T) of
 * workspace like the device variant (the staging buffer is part of it). */
int rm_action_expert_step_host(rm_ctx* ctx, const void* const* packed_layers, const float* r_in_host,
                               const int32_t* idx, const int32_t* count_dev, int64_t stride, float* r_out_host,
                               int B, int T, void* ws, size_t ws_bytes, rm_stream_t stream);

/* ---- rm_action_expert_step_ex: the same stack with the anchor-relative local update of the Action Cache (Sec. 4.1
 * "Anchors with Mask Recomputation", Eq. 4) and the output gate that follows it (after Eq. 4 the paper applies the model's
 * usual adaptive gate and then adds the residual).  Per layer l and episode:
 *   RM_ANCHOR_WRITE  (the group's anchor step; normally dense, idx = NULL):
 *       y_a = sum_{n in S} h_n Wd[:,n]   (S = every neuron when idx is NULL),   r_{l+1} = r_l + gate * y_a,
 *       and the call retains y_a in y_anchor and h_n[t] (n in S) in h_anchor.
 *   RM_ANCHOR_UPDATE (a non-anchor step with mask M = the list):
 *       y_hat = y_a + sum_{n in M} (h_n - h_a,n) Wd[:,n],                         r_{l+1} = r_l + gate * y_hat,
 *       with y_a, h_a read from y_anchor / h_anchor: neurons outside M keep the anchor step's contribution.
 *   RM_ANCHOR_NONE: rm_action_expert_step with the gate applied (zero-fill form).
 *   y_anchor [L,B,T,H] fp32 (pre-gate, pre-residual).   h_anchor [L,B,I,h_stride] fp32, neuron-major: the T
 *   activations of a neuron are contiguous, so a step may use any mask without an index map (the paper keeps
 *   h_a^M compact for one fixed mask); h_stride >= T and a multiple of 4.   out_gate [L,B,H] fp32 or NULL (= 1).
 *   With zero anchors (y_anchor = 0, h_anchor = 0) RM_ANCHOR_UPDATE equals the zero-fill form.
 *   In RM_ANCHOR_WRITE the call clears y_anchor itself.  Everything else as for rm_action_expert_step. */
enum { RM_ANCHOR_NONE = 0, RM_ANCHOR_WRITE = 1, RM_ANCHOR_UPDATE = 2 };
int rm_action_expert_step_ex(rm_ctx* ctx, const void* const* packed_layers, const float* r_in, const int32_t* idx,
                             const int32_t* count_dev, int64_t stride, float* r_out, float* records_out,
                             const float* record_scale, int B, int T, int anchor_mode, float* y_anchor,
                             float* h_anchor, int64_t h_stride, const float* out_gate, void* ws, size_t ws_bytes,
                             rm_stream_t stream);

/* ---- Context Cache: visual-token selective recomputation of one VLM FFN layer (Sec. 4.1 "Visual-Token
 * Recomputation", Eq. 2 and Eq. 3).  This path uses the model's own weight layouts (no packing): Wg, Wu [I,H] and
 * Wd [H,I] bf16 row-major; H and I multiples of 128.
 *
 * rm_context_drift (Eq. 2): score_out[p] = RMS(x_p - x_ref_p) / max(RMS(x_p), 1e-6) for the P visual rows;
 *   x, x_ref [P,H] bf16 (FFN inputs after RMSNorm, current and reference).  The rows to recompute are then the
 *   ceil(rho_p * P) largest scores: rm_mask_compact with RM_SRC_SCORE_F32 / RM_REDUCE_TOPK and I := P.
 *
 * rm_context_ffn (Eq. 3): y_out[p] = F(x_p) for the listed visual rows and for the S rows that follow the visual
 *   rows in x (instruction and state rows, always recomputed); every other visual row keeps y_ref[p].
 *   F(x) = Wd (gelu_tanh(Wg x) * (Wu x)), fp32 accumulation, the hidden activations rounded to bf16 between the two
 *   products (as the model does).  x [P+S,H] bf16; rows [>= count] int32 ascending, count_dev [1] int32 (device);
 *   y_ref [P,H] fp32; y_out [P+S,H] fp32 (may equal y_ref when that buffer has P+S rows).
 *   R_max >= count + S is the row capacity of the call, at most 1024 (RM_ERR_SHAPE above); a count that does not fit
 *   is truncated and RM_ERR_INDEX recorded.  Up to 256 rows go through the two products at once; a larger capacity
 *   takes one pass over the weights per 256 rows (the setting of the paper's Context Cache table, rho_p = 0.4 of 768
 *   visual rows plus 48 others = 356 rows, takes two).  A listed index outside [0, P) is skipped and RM_ERR_INDEX
 *   recorded.  ws: rm_context_workspace_bytes(ctx, R_max) bytes. */
int rm_context_drift(rm_ctx* ctx, const void* x, const void* x_ref, int P, float* score_out, rm_stream_t stream);
size_t rm_context_workspace_bytes(const rm_ctx* ctx, int R_max);
int rm_context_ffn(rm_ctx* ctx, const void* Wg, const void* Wu, const void* Wd, const void* x, const int32_t* rows,
                   const int32_t* count_dev, int P, int S, int R_max, const float* y_ref, float* y_out, void* ws,
                   size_t ws_bytes, rm_stream_t stream);

/* ---- rm_sparse_mlp_static: the one-layer call of rm_sparse_mlp for callers that cannot allocate.
 * (The paper has no counterpart for this entry point; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a robot's control loop that has frozen its
 * memory after start-up, a plug-in living inside a host framework's arena, a process whose device-memory budget is
 * fixed by an operator.  rm_create itself calls cudaMalloc, so such callers cannot even make a context.  This call takes no context and no workspace, and it calls neither
 * cudaMalloc / cudaFree nor any allocating library routine.
 *
 * How: the scratch that the two-kernel portable path needs (the compact hidden activations h [T, I] in fp32) is a
 * fixed 4 MiB array that is part of the library image; every GPU that loads the library carries it until the
 * process exits.  Limit: T * I <= 1,048,576 (for example T = 64 with I = 16384); larger requests return
 * RM_ERR_SHAPE.  H must be a multiple of 64 and at most 7232 (the gate/up kernel stages 32 * H bytes of x per CTA;
 * RM_ERR_SHAPE above).
 *
 * Arguments as for rm_sparse_mlp (packed_layer from rm_pack_weights with the same H and I; x [T,H] bf16; residual
 * [T,H] fp32 or NULL; idx ascending int32 or NULL for dense; count_dev [1] int32 on the device, required with idx,
 * and with idx NULL it selects the leading count neurons of the layer exactly as in rm_sparse_mlp; y [T,H] fp32, may
 * equal residual).  All pointers are device pointers, 16-byte aligned; the caller passes inputs and outputs as usual.
 * No activation record is produced.  Out-of-range indices are skipped silently (there is no status word without a
 * context).  The work is enqueued on `stream`; the call does not wait for it.
 *
 * First call on a device: looks up the array's device address and raises the gate/up kernel's shared-memory limit
 * (no allocation, but host-side set-up).  Make that first call before starting any stream capture on that device.
 * Sharing: every call on a device uses the same array and finds the previous call's contents in it.  Nothing needs
 * clearing (each call overwrites exactly the entries it reads), but two calls whose kernels overlap on the GPU --
 * different streams, or different host threads on different streams -- race on it: serialise them. */
int rm_sparse_mlp_static(const void* packed_layer, const void* x, const float* residual, const int32_t* idx,
                         const int32_t* count_dev, float* y, int T, int H, int I, rm_stream_t stream);

/* Measurement aids (not part of the method; the paper has no counterpart).
 * rm_debug_gather_read: reads the whole packed rows (6*H bytes each) of the listed neurons (idx NULL: every neuron) with
 * the instruction the layer kernels gather with -- 16-byte cp.async into shared memory, one CTA per SM, 12 rows in
 * flight per CTA -- and discards them.  Timed by the caller it gives the rate at which this list can leave HBM at all.
 * rm_debug_gather_read_step: the same for the L lists of one episode's step in ONE launch (packed_layers: host array of
 * L device pointers; list l at idx + l * stride, its count at count_dev[l]; idx NULL: every neuron of every layer). */
int rm_debug_gather_read(rm_ctx* ctx, const void* packed_layer, const int32_t* idx, const int32_t* count_dev,
                         int64_t list_cap, rm_stream_t stream);
int rm_debug_gather_read_step(rm_ctx* ctx, const void* const* packed_layers, const int32_t* idx, const int32_t* count_dev,
                              int64_t stride, rm_stream_t stream);

/* Test aid for the failure path: launches one CTA that waits on a barrier nobody arrives at, with a budget of `polls`
 * polls (1 .. 2^20; a few thousand take microseconds).  The wait runs out, the kernel records RM_ERR_TIMEOUT and the
 * place where it gave up exactly as the layer kernels' bounded waits do, and returns: rm_device_status then reports
 * RM_ERR_TIMEOUT, rm_get_info("status_detail") the source line and CTA, and the next rm_device_status is clean.
 * Nothing is left waiting and the context stays usable. */
int rm_debug_wait_timeout(rm_ctx* ctx, int polls, rm_stream_t stream);

/* Reads and clears the device status word (0 or the first RM_ERR_* a kernel recorded).  Synchronises `stream`. */
int rm_device_status(rm_ctx* ctx, int* host_out, rm_stream_t stream);

/* Number of kernels the library has launched through this context since creation (host counter). */
int64_t rm_launch_count(const rm_ctx* ctx);

/* Tuning knobs (host-side, take effect on later calls).  Names:
 *   "path"                0 = choose per shape (default), 1 = portable CUDA-core kernels only, 2 = the tcgen05
 *                         cluster kernel or RM_ERR_UNSUPPORTED
 *   "pdl"                 1 = chain the layers of a step with programmatic dependent launch (default)
 *   "neurons_per_cluster" active neurons a cluster should get before another cluster is used (default 64)
 *   "count_hint"          expected active neurons per layer and episode: the kernel family is chosen by it, and a
 *                         per-layer launch uses only as many clusters as it needs, so that the next layer's CTAs can
 *                         become resident early.  0 (default) = the k of the last top-k or group rm_mask_compact call
 *                         made through this context, if there was one, else unknown (the counts themselves stay on the
 *                         device and are never read by the host)
 *   "max_clusters"        cap on the clusters per launch (0 = none)
 *   "l2_prefetch"         warp-specialised kernel: number of tiles ahead for which the weights are pulled into L2
 *                         (0 = off, the default)
 *   "variant"             tcgen05 kernel variant: 0 = choose per launch, 1 = lean (one tile at a time, two CTAs per
 *                         SM at H = 1024), 2 = two tiles in flight per cluster, 3 = warp-specialised (the phases
 *                         of consecutive tiles run concurrently; for clusters that walk many tiles), 4 = streaming
 *                         (no clusters: every CTA owns whole tiles; for launches with many tiles), 5 = the whole-step
 *                         kernel (every layer of a step in one launch; zero-fill form, B <= 16; calls it does not
 *                         cover are chosen per launch)
 *   "stream_min_tiles"    launches with at least this many 64-neuron tiles use variant 4 when the variant is chosen
 *                         per launch (default 48 at H = 1024, 64 at H = 2048)
 *   "persist_max_batch"   largest B for which the whole-step kernel may be chosen per call (default 1)
 *   "persist_prefetch_kb" whole-step kernel: KB of weight rows a CTA may ask into L2 ahead of its loaders (default 0:
 *                         measured slower than no prefetch)                                                    */
int rm_set_option(rm_ctx* ctx, const char* name, int value);

/* Read-only facts: "fused_clusters" (co-resident clusters of the tcgen05 kernel, 0 when that path is
 * unavailable for this geometry or device), "fused_blocks_per_sm", "persist_clusters" (co-resident clusters of the
 * whole-step kernel), "sm_count", "path", "last_variant" (kernel family of the last layer or step launched through this
 * context: 0 portable, 1-5 as for the "variant" option), and "status_detail": for
 * the last non-zero status that rm_device_status returned, where the kernel gave up (a bounded wait that ran out:
 * source line of the wait << 12 | CTA index & 0xfff); 0 when that status carried no detail.
 * "last_cuda_error" (ctx may be NULL) is the cudaError_t of the last runtime call that made an entry point return
 * RM_ERR_CUDA.  "status_log_count" and "status_log:<i>" give the detail words of up to 60 errors of that launch in the order in
 * which they were recorded. */
int rm_get_info(const rm_ctx* ctx, const char* name, int* out);

/* Profiling aid, available only in builds made with -DRM_PHASE_TIMING (RM_ERR_UNSUPPORTED otherwise): copies the
 * per-CTA clock stamps the fused layer kernel took at its phase boundaries (host_out: n int64 values, 32 per CTA).
 * n = -(1 << 20) - m with m > 0 copies m values of the whole-step kernel's stamps instead, laid out
 * [item < 64][CTA < 128][32 slots]: slots 0-9 are globaltimer values in ns (x ready, first gate/up product, gate/up
 * complete, h sent, first down product, down complete, adds issued, arrival, normalisation start, normalisation done),
 * the others clock counts of a -DRM_PHASE_TIMING=2 build.  Host-synchronous. */
int rm_debug_phase_times(rm_ctx* ctx, long long* host_out, int n);

const char* rm_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* RMUSCLE_H */
