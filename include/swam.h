/*
 * swam - one action-guided sparse denoising step of a world-action model's
 * joint attention (Sparse-WAM), for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every call returns an int status (0 = SWAM_OK), never throws, never
 * allocates device memory and, unless stated otherwise, never synchronises: work
 * is enqueued on the caller's stream (`stream` is a cudaStream_t passed as
 * void*; NULL is the default stream).  The caller owns every tensor and the
 * workspace; the context owns host memory only.  The calls that do block the
 * host: swam_bind_workspace (one small synchronous cudaMemset of the status
 * word), swam_check (synchronises the stream and the internal copy streams)
 * and swam_destroy (destroys the internal streams and events, if any);
 * swam_bind_host_io creates two internal streams and six events on first use.
 *
 * Tracing: every call that enqueues work opens an NVTX range named after itself
 * in the NVTX domain "swam" for the time it spends on the host, and swam_step
 * opens one more range per stage inside its own ("dense_attention", "swam_score",
 * "select", "swam_pack", "packed_attention", "swam_scatter"; Sec. 4.2's full and
 * sparse step).  Without an NVTX tool attached to the process a range costs two
 * calls of an empty function.
 *
 * Notation (the paper's): B batch, N_o observed tokens, F future latent frames,
 * N_s tokens per future frame, H action tokens, N_h heads, D head dim,
 * g = H/F queries per frame-aligned group, K = K_c + K_s retained tokens per
 * frame, L = N_o + F*N_s + H, L' = N_o + F*K + H.
 * Sequence order: [observed | future frame 0 .. F-1 | action].
 * Tensor layout: [B, L, N_h, D] contiguous (token-major rows of N_h*D elements),
 * element type given by swam_shape.dtype.  "dev" = device pointer, "host" =
 * host pointer.  Device pointers must be 16-byte aligned.
 */
#ifndef SWAM_H_
#define SWAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct swam_ctx swam_ctx;

enum {
  SWAM_OK = 0,
  SWAM_ERR_INVALID_ARG = 1,  /* NULL / misaligned pointer, inconsistent shape */
  SWAM_ERR_UNSUPPORTED = 2,  /* valid request without a kernel (e.g. head_dim, group size) */
  SWAM_ERR_WORKSPACE = 3,    /* workspace missing or too small */
  SWAM_ERR_STATE = 4,        /* reuse requested before any refresh */
  SWAM_ERR_CUDA = 5,         /* a CUDA runtime call failed; see swam_last_error */
  SWAM_ERR_DEVICE_CHECK = 6, /* a kernel met an out-of-range map entry or an impossible count */
  SWAM_ERR_TIMEOUT = 7       /* a bounded device-side wait ran out */
};

enum { SWAM_F32 = 0, SWAM_BF16 = 1 };

/* swam_step modes */
enum {
  SWAM_REUSE = 0,         /* sparse step: pack -> packed attention -> scatter with the cached maps */
  SWAM_REFRESH_FULL = 1,  /* full step: dense attention (fills the cache) -> score -> select */
  SWAM_REFRESH_LIGHT = 2  /* score (normaliser computed here) -> select -> pack -> packed attention -> scatter */
};

typedef struct {
  int32_t batch, n_obs, n_frames, n_spatial, n_action, n_heads, head_dim;
  int32_t k_core, k_anchor;   /* K_c, K_s; K_c + K_s <= N_s (Sec. 4.1) */
  int32_t dtype;              /* SWAM_F32 | SWAM_BF16 */
  float softmax_scale;        /* 0 => 1/sqrt(head_dim) */
  float cv_beta;              /* coefficient of the cross-frame variation penalty; the paper uses 1.0 */
  const float* query_weights; /* host, [H/F], non-negative, sums to 1; NULL => central half 2x outer quarters */
  int32_t n_kv_heads;         /* key/value heads (grouped-query attention); 0 => n_heads; must divide n_heads */
} swam_shape;

/* Tensor layouts.  Q and every output are [B, L, n_heads, head_dim]; K and V are [B, L, n_kv_heads, head_dim]
 * (packed tensors likewise with L' rows).  Query head h reads key/value head h / (n_heads / n_kv_heads): the backbone's
 * head mapping, which the scoring follows (App. A.2).  With n_kv_heads = n_heads (the default) all four tensors have the
 * same shape. */

/* Context: validates the shape (H divisible by F, Eq. 8; K_c + K_s <= N_s; head_dim in {32, 64, 128};
 * NULL weights need H/F divisible by 4; at most 65535 samples, half of that with more than 128 action tokens; L at most
 * 2^24 and B*L at most 2^30: SWAM_ERR_UNSUPPORTED beyond) and fixes the workspace layout.  The shape (and the weights) are
 * copied.  The current CUDA device at creation is the device every later call must run on. */
int swam_create(const swam_shape* shape, swam_ctx** out_ctx);
int swam_destroy(swam_ctx* ctx);

/* Device workspace, caller-allocated (256-byte aligned).  It holds the cross-step state (scores, action-row
 * normalisers, selection, maps, status word) and the packed Q/K/V/O buffers that swam_step uses.  Binding
 * zeroes the status word and clears the "has selection" state (synchronous, small). */
int swam_workspace_bytes(const swam_ctx* ctx, size_t* bytes);
int swam_bind_workspace(swam_ctx* ctx, void* dev_ptr, size_t bytes);

/* (1) Action-to-future scoring, Eq. 12 (extraction form of Eq. 1-2):
 *   S[b,f,j] = 1/N_h * sum_{i in I_f} sum_h alpha_i * exp(scale * q_{i,h} . k_{(f,j),h} - lambda[b,h,i])
 * q, k: dev, full tensors [B, L, N_h, D] (only the action rows of q and, when lambda is given, only the
 * future rows of k are read).  lse_action: dev float [B, N_h, H], log-sum-exp of each action query over ALL
 * L keys (Sec. 4.2 "reuses the original normalisers"); NULL => computed here over all L keys (uses workspace
 * scratch).  scores: dev float [B, F, N_s].  quality: dev float [B, 3] = (R, E, Q) of Eq. 9, or NULL. */
int swam_score(swam_ctx* ctx, const void* q, const void* k, const float* lse_action,
               float* scores, float* quality, void* stream);

/* Scoring for callers that cannot allocate device memory.  (The paper has no counterpart; this is a packaging
 * variant of call (1) with the normalisers computed here.)  Some users of this library run the scorer from places
 * where a workspace cannot be obtained: a policy server whose framework reserved all device memory at start-up so
 * that cudaMalloc fails, or a control-loop thread that must not call cudaMalloc because it stalls the whole device.
 * For them the scratch that call (1) keeps in the workspace (the action-row normalisers and the per-chunk partial
 * maxima and sums) lives in an 8 MiB array inside the library image, which every GPU that loads the library
 * holds until the process exits.  No workspace needs to be bound and nothing is allocated or freed, on the host or
 * on the device.  q, k, scores: dev, as in call (1); results equal swam_score(ctx, q, k, NULL, scores, NULL, stream).
 * Shapes whose scratch exceeds the array (B*N_h*H*4 bytes rounded up to 256, plus B*ceil(L/128)*N_h*H*8 bytes
 * for bf16) return SWAM_ERR_UNSUPPORTED with the two sizes in swam_last_error.  The first call on each device looks
 * up the array's device address (with that device current); make that call before any stream capture.  All calls
 * share the one array and leave their intermediate values in it: nothing in it has to be cleared between calls,
 * but two calls whose kernels overlap on the GPU (different streams, or different contexts) race on it. */
int swam_score_noalloc(swam_ctx* ctx, const void* q, const void* k, float* scores, void* stream);

/* (2) Selection and packing metadata, Eq. 4-6, 10-11 with one profiled layer (V = V_all = S):
 * pool = top (N_s - K_s) of max_f S; core_f = top K_c of S[f] within the pool; anchors = top K_s of
 * mu_j / (1 + beta * CV_j) over positions that are core in no frame (population std, fp64, mu_j = 0 => CV_j = 0).
 * Equal keys go to the lower index.  scores: dev float [B, F, N_s] (finite).  sel_idx: dev int32 [B, F, K]
 * ascending spatial indices; pack_map: dev int32 [B, L'] original row of each packed row (strictly increasing);
 * inv_map: dev int32 [B, L] packed row of each original row, -1 if omitted.  Any output may be NULL. */
int swam_select(swam_ctx* ctx, const float* scores, int32_t* sel_idx, int32_t* pack_map, int32_t* inv_map,
                void* stream);

/* (2b) Several profiled layers (Sec. 4.1, App. A.1).  swam_aggregate forms the core score map
 *   V = sum_{l in L_core} Q_l S_l / sum_{l in L_core} Q_l (Eq. 3), L_core = the k_layer layers with the largest Q_l,
 * and the anchor score map V_all, the same sum over all layers (Eq. 11), from per-layer scores and qualities as
 * swam_score writes them: layer_scores dev float [n_layers, B, F, N_s], layer_quality dev float [n_layers, B, 3]
 * (R, E, Q of Eq. 9; only Q is used).  fp64 accumulation in ascending layer order, results stored as fp32; equal
 * qualities go to the lower layer index; if the weights of a set sum to zero the plain mean is used.  v_core, v_all:
 * dev float [B, F, N_s]; core_layers: dev int32 [B, k_layer] ascending, or NULL.  n_layers <= 256.
 * swam_select_maps is call (2) with pool and cores ranked on core_scores (V) and anchors on anchor_scores (V_all). */
int swam_aggregate(swam_ctx* ctx, const float* layer_scores, const float* layer_quality, int32_t n_layers,
                   int32_t k_layer, float* v_core, float* v_all, int32_t* core_layers, void* stream);
int swam_select_maps(swam_ctx* ctx, const float* core_scores, const float* anchor_scores, int32_t* sel_idx,
                     int32_t* pack_map, int32_t* inv_map, void* stream);

/* (3) Packing (Sec. 4.2): xp[b, p, :] = x[b, pack_map[b, p], :] for x in {q, k, v}; xp: dev [B, L', N_h, D].
 * Any of the three pairs may be NULL/NULL.  Out-of-range map entries are skipped and flagged in the status word. */
int swam_pack(swam_ctx* ctx, const void* q, const void* k, const void* v, const int32_t* pack_map,
              void* qp, void* kp, void* vp, void* stream);

/* (4) Joint attention over a compact (or the full) sequence, plain softmax attention with full visibility:
 * out[b,r,h,:] = sum_c softmax_c(scale * q[b,r,h,:] . k[b,c,h,:]) v[b,c,h,:], tensors [B, seq_len, N_h, D].
 * lse: dev float [B, N_h, seq_len] natural-log normalisers, or NULL.  bf16: fp32 accumulation. */
int swam_sparse_attn(swam_ctx* ctx, const void* qp, const void* kp, const void* vp, int32_t seq_len,
                     void* out_p, float* lse, void* stream);

/* (5) Scatter back, Eq. 7: out[b, pack_map[b,p], :] = out_p[b, p, :]; every omitted row takes cached's row.
 * cached may equal out (in place: omitted rows are left untouched, which is Eq. 7 when out still holds the
 * last full step's result).  inv_map is only read when cached != out. */
int swam_scatter(swam_ctx* ctx, const void* out_p, const int32_t* pack_map, const int32_t* inv_map,
                 const void* cached, void* out, void* stream);

/* One denoising step (Sec. 4.2).  q, k, v, out: dev [B, L, N_h, D]; out persists across steps and holds the
 * last full step's result on omitted rows.  mode: SWAM_REFRESH_FULL runs dense attention into out, scores the
 * future tokens with the dense pass's action-row normalisers, selects and builds the maps; SWAM_REUSE packs by
 * the cached maps, attends over L' tokens and scatters into out (SWAM_ERR_STATE before any refresh);
 * SWAM_REFRESH_LIGHT recomputes normalisers, scores and selection from this step's q, k without a dense pass,
 * then runs the sparse step with the new maps. */
int swam_step(swam_ctx* ctx, const void* q, const void* k, const void* v, int32_t mode, void* out, void* stream);

/* The same step for callers whose tensors live in (pinned) host memory.  The call enqueues a three-stage pipeline
 * and does not synchronise: q, k, v travel to a device staging slot on an internal copy stream, swam_step runs on
 * `stream`, and out leaves for out_host on a second internal copy stream, so that consecutive calls overlap one
 * step's copies with the neighbouring steps' compute and the two PCIe directions with each other.  The staging area
 * (10 full tensors: three input slots and the persistent out; caller-allocated, dev) is bound once; binding creates the
 * internal streams and events.  A SWAM_REUSE step brings only the rows its maps retain across PCIe when the host
 * buffers are pinned memory the device can address (see SWAM_OPT_HOST_ROWS); a kernel then reads the caller's
 * buffers directly.  The host input buffers of a call must stay unchanged, and out_host is complete,
 * once swam_check (which also waits for the internal streams) or a device-wide synchronisation has returned.  On
 * SWAM_REUSE steps the staged out of the previous step is the cache, so the staging area must not be touched between
 * steps.  Not capturable in a CUDA graph. */
int swam_host_io_bytes(const swam_ctx* ctx, size_t* bytes);
int swam_bind_host_io(swam_ctx* ctx, void* dev_ptr, size_t bytes);
int swam_step_host(swam_ctx* ctx, const void* q_host, const void* k_host, const void* v_host, int32_t mode,
                   void* out_host, void* stream);
/* Makes `stream` wait (on the device, without blocking the host) until the result of the most recent
 * swam_step_host call has arrived in its out_host; work enqueued on `stream` afterwards may read out_host. */
int swam_host_join(swam_ctx* ctx, void* stream);

/* Device pointers (inside the workspace) of the state swam_step keeps; any argument may be NULL. */
int swam_get_selection(const swam_ctx* ctx, const int32_t** sel_idx, const int32_t** pack_map,
                       const int32_t** inv_map);
int swam_get_scores(const swam_ctx* ctx, const float** scores, const float** lse_action, const float** quality);

/* Installs a selection made elsewhere as the state that SWAM_REUSE steps use: sel_idx [B, F, K], pack_map [B, L'] and
 * inv_map [B, L] (device pointers, int32, the layouts swam_select writes) are copied into the workspace on `stream`.
 * Uses: the unconditional forward of a guided denoising step reuses the selection of the conditional forward, from
 * which the scores come (Sec. 4.2; Table 5 lists the guidance scales); the selection ablations of Sec. 5.4 (core only,
 * anchors only, random) run swam_select on scores of their own and install the result; a saved state is restored.
 * The maps are not checked here: the kernels that follow them skip and flag entries out of range (swam_check).
 * Errors: SWAM_ERR_INVALID_ARG (null pointer), SWAM_ERR_WORKSPACE (none bound), SWAM_ERR_CUDA. */
int swam_set_selection(swam_ctx* ctx, const int32_t* sel_idx, const int32_t* pack_map, const int32_t* inv_map,
                       void* stream);

/* The whole cross-step state of swam_step (scores, Eq. 9 diagnostics, action-row normalisers, selection, maps) as one
 * opaque device buffer: swam_state_bytes gives its size, swam_state_export copies the state into dev_buf and
 * swam_state_import installs a buffer written by a context of the same shape, after which SWAM_REUSE steps continue
 * where the exporting context stood (the cached output tensor `out` belongs to the caller and travels separately).
 * Both copies are asynchronous on `stream`.  Errors: SWAM_ERR_STATE (export before any refresh), SWAM_ERR_WORKSPACE,
 * SWAM_ERR_INVALID_ARG, SWAM_ERR_CUDA. */
int swam_state_bytes(const swam_ctx* ctx, size_t* bytes);
int swam_state_export(swam_ctx* ctx, void* dev_buf, void* stream);
int swam_state_import(swam_ctx* ctx, const void* dev_buf, void* stream);

/* Synchronises `stream`, reads and clears the device status word; returns SWAM_OK, SWAM_ERR_DEVICE_CHECK,
 * SWAM_ERR_TIMEOUT or SWAM_ERR_CUDA. */
int swam_check(swam_ctx* ctx, void* stream);

/* Self-test of the failure reporting of device-side waits (no counterpart in the paper).  Every wait inside the
 * library's kernels is bounded; when a bound runs out the kernel raises the timeout bit of the status word and returns.
 * This call makes that happen harmlessly: it enqueues a one-warp kernel that waits on a barrier nothing ever completes,
 * gives up after limit_cycles SM clock cycles (1 .. 1e8, i.e. at most some 50 ms) and returns by itself.  The next
 * swam_check then yields SWAM_ERR_TIMEOUT (and clears the word); the context stays usable.  Needs a bound workspace. */
int swam_selftest_timeout(swam_ctx* ctx, uint64_t limit_cycles, void* stream);

/* Enqueues an empty kernel (no counterpart in the paper).  Selection (call 2) reads at most a few hundred KB and is
 * bound by launch and dependent-pass latency, not by memory bandwidth; timing this call in the same harness gives the
 * launch floor that its time is reported against. */
int swam_launch_floor(swam_ctx* ctx, void* stream);

/* Options.  SWAM_OPT_ATTN_VARIANT selects the bf16 attention kernel: SWAM_ATTN_AUTO (default) runs the
 * tcgen05/TMEM kernel for head_dim 64 and 128 and the warp-level mma.sync kernel for head_dim 32;
 * SWAM_ATTN_WARP_MMA forces the mma.sync kernel (an independent on-device second opinion used by the tests).
 *
 * SWAM_OPT_SPARSE_PATH selects how swam_step runs a REUSE or REFRESH_LIGHT step (Sec. 4.2, Eq. 7):
 * SWAM_SPARSE_FUSED (default) packs only K and V; the tcgen05 attention kernel fetches its query rows from the full
 * Q through pack_map and writes each retained row straight to its original position in `out`, so that the packed Q,
 * the packed output and the scatter pass do not exist; SWAM_SPARSE_STAGED runs swam_pack, swam_sparse_attn and
 * swam_scatter one after the other; SWAM_SPARSE_FUSED_KV goes one step beyond FUSED: the attention kernel also
 * fetches the key and value rows through pack_map (TMA row gathers), so that nothing is packed at all and the sparse
 * step is one launch.  Every query tile pair of a head then repeats the gather of that head's rows, which measures
 * slower than packing K and V once at the benchmark shapes; it is offered for shapes with few query tiles.  The fused
 * paths need bf16, head_dim 64 or 128 and SWAM_ATTN_AUTO; every other configuration runs staged.  All three paths
 * produce the same bits.
 *
 * SWAM_OPT_VISIBILITY sets the backbone's visibility constraints (App. A.2) in the form this library supports: the
 * joint sequence is [observed | future | action], and the rows of each of the three segments see a prefix of it, up to
 * the end of the observed tokens (SWAM_SEES_OBSERVED), of the future tokens (SWAM_SEES_FUTURE) or of the whole
 * sequence (SWAM_SEES_ALL).  value = SWAM_VISIBILITY(observed_rows_see, future_rows_see, action_rows_see); the default
 * is SWAM_SEES_ALL for all three (full visibility).  Future rows must see at least the future tokens and action rows
 * at least the future tokens (they score them).  The setting applies to swam_step, to swam_sparse_attn at the full
 * and the packed length (segment boundaries N_o and N_o + F*N_s, or N_o and N_o + F*K; other lengths return
 * SWAM_ERR_UNSUPPORTED unless visibility is full) and to the normalisers swam_score computes, which then run over the
 * keys the action rows see.
 *
 * SWAM_OPT_HOST_ROWS selects what a SWAM_REUSE step of swam_step_host brings across PCIe: SWAM_HOST_ROWS_RETAINED
 * (default) only the rows the cached maps retain (Sec. 4.2: the sparse step processes the compact sequence), fetched
 * by a kernel on the library's copy-in stream straight from the caller's buffers, which must then be pinned memory
 * the device can address (cudaHostAlloc / cudaHostRegister); buffers that are not are copied whole, as with
 * SWAM_HOST_ROWS_ALL.  The result is the same either way. */
enum { SWAM_OPT_ATTN_VARIANT = 1, SWAM_OPT_SPARSE_PATH = 2, SWAM_OPT_VISIBILITY = 3, SWAM_OPT_HOST_ROWS = 4 };
enum { SWAM_HOST_ROWS_RETAINED = 0, SWAM_HOST_ROWS_ALL = 1 };
enum { SWAM_ATTN_AUTO = 0, SWAM_ATTN_WARP_MMA = 1 };
enum { SWAM_SPARSE_FUSED = 0, SWAM_SPARSE_STAGED = 1, SWAM_SPARSE_FUSED_KV = 2 };
enum { SWAM_SEES_OBSERVED = 0, SWAM_SEES_FUTURE = 1, SWAM_SEES_ALL = 2 };
#define SWAM_VISIBILITY(observed_rows_see, future_rows_see, action_rows_see) \
  ((observed_rows_see) | ((future_rows_see) << 2) | ((action_rows_see) << 4))
int swam_set_option(swam_ctx* ctx, int32_t option, int32_t value);

/* Number of kernels this context has launched so far (host-side counter). */
int swam_launch_count(const swam_ctx* ctx, int64_t* count);

const char* swam_last_error(const swam_ctx* ctx);
const char* swam_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SWAM_H_ */
