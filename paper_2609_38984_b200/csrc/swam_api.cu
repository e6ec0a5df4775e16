// C-ABI layer of libswam: context, validation, workspace layout, and the step state machine.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include <nvtx3/nvToolsExt.h>

#include "../../include/swam.h"
#include "swam_internal.cuh"

using namespace swam;

struct swam_ctx {
  Dims d;
  Alpha alpha;
  int device;
  // workspace (device)
  unsigned char* ws;
  size_t ws_bytes;
  size_t off_status, off_scores, off_quality, off_lse, off_sel, off_pack, off_inv, off_scratch, off_qp, off_kp,
      off_vp, off_op, off_attn, off_logits, off_lam2, off_counters, attn_scratch, ws_need;
  bool has_selection;
  bool maps_own;     // the cached maps were built by this context's selection kernel (not installed or imported)
  int attn_variant;  // SWAM_ATTN_AUTO | SWAM_ATTN_WARP_MMA
  int sparse_path;   // SWAM_SPARSE_FUSED | SWAM_SPARSE_STAGED
  int host_rows;     // SWAM_HOST_ROWS_RETAINED | SWAM_HOST_ROWS_ALL: what a reuse step with host buffers brings in
  int sees[3];       // what observed / future / action rows see: SWAM_SEES_*
  // host-io staging (device): two input slots of (q, k, v) and the persistent output, plus the copy pipeline
  unsigned char* io;
  size_t io_need;
  cudaStream_t s_in, s_out;           // host-to-device and device-to-host copy streams
  cudaStream_t s_rows;                // the retained-row fetches of reuse steps (they wait for the maps; whole copies need not)
  cudaEvent_t ev_h2d[3], ev_done[3];  // per input slot: inputs arrived / step finished with the slot
  cudaEvent_t ev_d2h;                 // the previous result has left the staged output
  cudaEvent_t ev_pre;                 // everything the caller's stream held when a reuse step with host buffers was called
  cudaEvent_t ev_obs;                 // the observed rows of a reuse step's inputs have arrived (plain copies on s_in)
  int64_t host_steps;
  int launches_i;
  int64_t launches;
  char err[256];
};

namespace {

// Tracing: every call below that launches work opens an NVTX range named after itself in the domain "swam", and
// swam_step opens one more per stage inside its own, so that a timeline tool shows which kernels belong to which
// call and stage.  NVTX is header-only; without a tool attached a push or pop is a call through a pointer to an empty
// function.
nvtxDomainHandle_t trace_domain() {
  static nvtxDomainHandle_t dom = nvtxDomainCreateA("swam");
  return dom;
}
struct Range {
  explicit Range(const char* name) {
    nvtxEventAttributes_t a;
    memset(&a, 0, sizeof(a));
    a.version = NVTX_VERSION;
    a.size = NVTX_EVENT_ATTRIB_STRUCT_SIZE;
    a.messageType = NVTX_MESSAGE_TYPE_ASCII;
    a.message.ascii = name;
    nvtxDomainRangePushEx(trace_domain(), &a);
  }
  ~Range() { nvtxDomainRangePop(trace_domain()); }
  Range(const Range&) = delete;
  Range& operator=(const Range&) = delete;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int fail(swam_ctx* c, int code, const char* msg) {
  if (c) snprintf(c->err, sizeof(c->err), "%s", msg);
  return code;
}
int fail_cuda(swam_ctx* c, cudaError_t e, const char* where) {
  if (c) snprintf(c->err, sizeof(c->err), "%s: %s", where, cudaGetErrorString(e));
  return SWAM_ERR_CUDA;
}
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t elem_bytes(const Dims& d) { return d.dtype == SWAM_F32 ? 4 : 2; }
size_t full_bytes(const Dims& d) { return (size_t)d.B * d.L * d.N_h * d.D * elem_bytes(d); }
size_t packed_bytes(const Dims& d) { return (size_t)d.B * d.Lp * d.N_h * d.D * elem_bytes(d); }
size_t kv_full_bytes(const Dims& d) { return (size_t)d.B * d.L * d.N_kv * d.D * elem_bytes(d); }
size_t kv_packed_bytes(const Dims& d) { return (size_t)d.B * d.Lp * d.N_kv * d.D * elem_bytes(d); }

void count(swam_ctx* c) {
  c->launches += c->launches_i;
  c->launches_i = 0;
}

bool full_visibility(const swam_ctx* c) {
  return c->sees[0] == SWAM_SEES_ALL && c->sees[1] == SWAM_SEES_ALL && c->sees[2] == SWAM_SEES_ALL;
}

// keys of the full sequence that the action rows see (the normalisers of the scorer run over them)
int action_keys(const swam_ctx* c) { return c->sees[2] == SWAM_SEES_ALL ? c->d.L : c->d.L - c->d.H; }

// Fills the visibility fields of `a` for a sequence of a.n tokens: the full sequence (future segment of F * N_s
// tokens) or the packed one (F * K).  False when the context restricts visibility and a.n is neither length.
bool set_visibility(const swam_ctx* c, AttnArgs& a) {
  const Dims& d = c->d;
  a.obs_end = a.fut_end = a.n;
  a.lim[0] = a.lim[1] = a.lim[2] = a.n;
  if (full_visibility(c)) return true;
  if (a.n != d.L && a.n != d.Lp) return false;
  a.obs_end = d.n_obs;
  a.fut_end = a.n - d.H;
  const int ends[3] = {a.obs_end, a.fut_end, a.n};
  for (int s = 0; s < 3; ++s) a.lim[s] = ends[c->sees[s]];
  return true;
}

int run_attention(swam_ctx* c, const void* q, const void* k, const void* v, int n, void* out, float* lse, int lse_row0,
                  int lse_rows, cudaStream_t st) {
  AttnArgs a{q, k, v, out, lse, lse_row0, lse_rows, c->d.B, n, c->d.N_h, c->d.D, c->d.scale, c->d.N_kv};
  if (!set_visibility(c, a))
    return fail(c, SWAM_ERR_UNSUPPORTED, "restricted visibility needs the full or the packed sequence length");
  cudaError_t e;
  if (c->d.dtype == SWAM_F32) {
    e = launch_attn_f32(a, st, &c->launches_i);
  } else if (c->d.D >= 64 && c->attn_variant == SWAM_ATTN_AUTO) {
    if (!c->ws) return fail(c, SWAM_ERR_WORKSPACE, "no workspace bound");
    e = launch_attn_bf16_tc(a, (int*)(c->ws + c->off_status), c->ws + c->off_attn, c->attn_scratch, st, &c->launches_i);
  } else {
    e = launch_attn_bf16_mma(a, st, &c->launches_i);
  }
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "attention launch");
  return SWAM_OK;
}

int need_ws(swam_ctx* c) {
  if (!c->ws) return fail(c, SWAM_ERR_WORKSPACE, "no workspace bound");
  return SWAM_OK;
}

int check_device(swam_ctx* c) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail_cuda(c, e, "cudaGetDevice");
  if (dev != c->device) return fail(c, SWAM_ERR_INVALID_ARG, "current device differs from the context's device");
  return SWAM_OK;
}

}  // namespace

extern "C" {

const char* swam_version(void) { return "swam 0.1 (sm_100a)"; }

const char* swam_last_error(const swam_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int swam_create(const swam_shape* s, swam_ctx** out_ctx) {
  if (!s || !out_ctx) return SWAM_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  if (s->batch <= 0 || s->n_obs < 0 || s->n_frames <= 0 || s->n_spatial <= 0 || s->n_action <= 0 || s->n_heads <= 0 ||
      s->k_core < 0 || s->k_anchor < 0)
    return SWAM_ERR_INVALID_ARG;
  if (s->n_action % s->n_frames != 0) return SWAM_ERR_INVALID_ARG;          // Eq. 8 needs H divisible by F
  if (s->k_core + s->k_anchor > s->n_spatial) return SWAM_ERR_INVALID_ARG;   // K_c + K_s <= N_s
  if (s->dtype != SWAM_F32 && s->dtype != SWAM_BF16) return SWAM_ERR_INVALID_ARG;
  if (!(s->softmax_scale >= 0.f) || !(s->cv_beta >= 0.f)) return SWAM_ERR_INVALID_ARG;
  if (s->head_dim != 32 && s->head_dim != 64 && s->head_dim != 128) return SWAM_ERR_UNSUPPORTED;
  if (s->n_kv_heads < 0 || (s->n_kv_heads > 0 && s->n_heads % s->n_kv_heads != 0)) return SWAM_ERR_INVALID_ARG;
  const int g = s->n_action / s->n_frames;
  if (g > kMaxGroup) return SWAM_ERR_UNSUPPORTED;
  if (!s->query_weights && (g % 4) != 0) return SWAM_ERR_INVALID_ARG;
  const long long L = (long long)s->n_obs + (long long)s->n_frames * s->n_spatial + s->n_action;
  if (L > (1 << 24) || (long long)s->batch * L > (1ll << 30)) return SWAM_ERR_UNSUPPORTED;
  // samples are a grid dimension of most kernels (times the chunks of 128 action queries in the one-pass scorer)
  if ((long long)s->batch * ((s->n_action + 127) / 128) > 65535) return SWAM_ERR_UNSUPPORTED;

  swam_ctx* c = new (std::nothrow) swam_ctx();
  if (!c) return SWAM_ERR_INVALID_ARG;
  memset(c, 0, sizeof(*c));
  c->sees[0] = c->sees[1] = c->sees[2] = SWAM_SEES_ALL;
  Dims& d = c->d;
  d.B = s->batch; d.n_obs = s->n_obs; d.F = s->n_frames; d.N_s = s->n_spatial; d.H = s->n_action;
  d.N_h = s->n_heads; d.N_kv = s->n_kv_heads > 0 ? s->n_kv_heads : s->n_heads; d.D = s->head_dim; d.Kc = s->k_core; d.Ks = s->k_anchor; d.K = d.Kc + d.Ks;
  d.L = (int)L; d.Lp = d.n_obs + d.F * d.K + d.H; d.g = g; d.dtype = s->dtype;
  d.scale = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf((float)d.D);
  d.beta = s->cv_beta;
  if (s->query_weights) {
    double sum = 0.0;
    for (int i = 0; i < g; ++i) {
      if (!(s->query_weights[i] >= 0.f)) { delete c; return SWAM_ERR_INVALID_ARG; }
      c->alpha.w[i] = s->query_weights[i];
      sum += s->query_weights[i];
    }
    if (fabs(sum - 1.0) > 1e-4) { delete c; return SWAM_ERR_INVALID_ARG; }
  } else {
    // central half of the group weighs twice the outer quarters; normalised: 2/(3g) outside, 4/(3g) inside
    for (int i = 0; i < g; ++i)
      c->alpha.w[i] = (float)(((i >= g / 4 && i < g - g / 4) ? 4.0 : 2.0) / (3.0 * g));
  }
  if (select_smem_bytes(d) > 227 * 1024) { delete c; return SWAM_ERR_UNSUPPORTED; }
  if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return SWAM_ERR_CUDA; }

  // workspace layout, every block 256-byte aligned
  size_t off = 0;
  auto put = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  c->off_status = put(256);
  c->off_counters = put(score_counter_bytes(d));   // directly behind the status word: one memset clears both
  c->off_scores = put((size_t)d.B * d.F * d.N_s * 4);
  c->off_quality = put((size_t)d.B * 3 * 4);
  c->off_lse = put((size_t)d.B * d.N_h * d.H * 4);
  c->off_sel = put((size_t)d.B * d.F * d.K * 4);
  c->off_pack = put((size_t)d.B * d.Lp * 4);
  c->off_inv = put((size_t)d.B * d.L * 4);
  c->off_scratch = put(lse_scratch_bytes(d));
  c->off_qp = put(packed_bytes(d));
  c->off_kp = put(kv_packed_bytes(d));
  c->off_vp = put(kv_packed_bytes(d));
  c->off_op = put(packed_bytes(d));
  c->attn_scratch = (d.dtype == SWAM_BF16 && d.D >= 64) ? attn_tc_scratch_bytes(d.D) : 0;
  c->off_attn = put(c->attn_scratch);
  c->off_logits = put(score_logits_bytes(d));
  c->off_lam2 = put((size_t)d.B * d.N_h * d.H * 4);
  c->ws_need = off;
  c->io_need = 10 * align_up(full_bytes(d), 256);   // three input slots of (q, k, v) and the staged output
  *out_ctx = c;
  return SWAM_OK;
}

int swam_destroy(swam_ctx* ctx) {
  if (ctx && ctx->s_in) {
    cudaStreamDestroy(ctx->s_in);
    cudaStreamDestroy(ctx->s_rows);
    cudaStreamDestroy(ctx->s_out);
    for (int i = 0; i < 3; ++i) { cudaEventDestroy(ctx->ev_h2d[i]); cudaEventDestroy(ctx->ev_done[i]); }
    cudaEventDestroy(ctx->ev_d2h);
    cudaEventDestroy(ctx->ev_pre);
    cudaEventDestroy(ctx->ev_obs);
  }
  delete ctx;
  return SWAM_OK;
}

int swam_workspace_bytes(const swam_ctx* ctx, size_t* bytes) {
  if (!ctx || !bytes) return SWAM_ERR_INVALID_ARG;
  *bytes = ctx->ws_need;
  return SWAM_OK;
}

int swam_bind_workspace(swam_ctx* c, void* dev_ptr, size_t bytes) {
  Range trace_range("swam_bind_workspace");
  if (!c || !dev_ptr) return SWAM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return fail(c, SWAM_ERR_INVALID_ARG, "workspace not 256-byte aligned");
  if (bytes < c->ws_need) return fail(c, SWAM_ERR_WORKSPACE, "workspace too small");
  if (int r = check_device(c)) return r;
  cudaError_t e = select_prepare(c->d);
  if (e != cudaSuccess) return fail_cuda(c, e, "select_prepare");
  e = cudaMemset(dev_ptr, 0, c->off_counters + score_counter_bytes(c->d));   // status word and arrival tickets
  if (e != cudaSuccess) return fail_cuda(c, e, "cudaMemset(status)");
  c->ws = (unsigned char*)dev_ptr;
  c->ws_bytes = bytes;
  c->has_selection = false;
  c->maps_own = false;
  return SWAM_OK;
}

int swam_host_io_bytes(const swam_ctx* ctx, size_t* bytes) {
  if (!ctx || !bytes) return SWAM_ERR_INVALID_ARG;
  *bytes = ctx->io_need;
  return SWAM_OK;
}

int swam_bind_host_io(swam_ctx* c, void* dev_ptr, size_t bytes) {
  Range trace_range("swam_bind_host_io");
  if (!c || !dev_ptr) return SWAM_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return fail(c, SWAM_ERR_INVALID_ARG, "staging not 256-byte aligned");
  if (bytes < c->io_need) return fail(c, SWAM_ERR_WORKSPACE, "staging area too small");
  if (int r = check_device(c)) return r;
  if (!c->s_in) {
    cudaError_t e = cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->s_rows, cudaStreamNonBlocking);
    for (int i = 0; i < 3 && e == cudaSuccess; ++i) {
      e = cudaEventCreateWithFlags(&c->ev_h2d[i], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_d2h, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_pre, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_obs, cudaEventDisableTiming);
    if (e != cudaSuccess) return fail_cuda(c, e, "swam_bind_host_io: stream/event creation");
  }
  c->io = (unsigned char*)dev_ptr;
  c->host_steps = 0;
  return SWAM_OK;
}

int swam_score(swam_ctx* c, const void* q, const void* k, const float* lse_action, float* scores, float* quality,
               void* stream) {
  Range trace_range("swam_score");
  if (!c || !q || !k || !scores) return fail(c, SWAM_ERR_INVALID_ARG, "swam_score: null argument");
  if (!aligned16(q) || !aligned16(k) || !aligned16(scores)) return fail(c, SWAM_ERR_INVALID_ARG, "swam_score: misaligned pointer");
  cudaStream_t st = (cudaStream_t)stream;
  const float* lse = lse_action;
  if (!lse && score_one_pass_supported(c->d)) {
    // one pass over the keys: the normalisers' kernel leaves the future keys' products behind and a small second
    // kernel turns them into scores, instead of a second read of every future key
    if (int r = need_ws(c)) return r;
    cudaError_t e = launch_score_one_pass(c->d, c->alpha, q, k, (float*)(c->ws + c->off_lse), (float*)(c->ws + c->off_lam2),
                                          c->ws + c->off_scratch, (unsigned int*)(c->ws + c->off_counters),
                                          (float*)(c->ws + c->off_logits), (int*)(c->ws + c->off_status), scores, st,
                                          &c->launches_i, action_keys(c));
    count(c);
    if (e != cudaSuccess) return fail_cuda(c, e, "one-pass score launch");
  } else {
    if (!lse) {
      if (int r = need_ws(c)) return r;
      float* own = (float*)(c->ws + c->off_lse);
      cudaError_t e = launch_action_lse(c->d, q, k, own, c->ws + c->off_scratch, st, &c->launches_i, action_keys(c));
      count(c);
      if (e != cudaSuccess) return fail_cuda(c, e, "action lse launch");
      lse = own;
    }
    cudaError_t e = launch_score(c->d, c->alpha, q, k, lse, scores, st, &c->launches_i);
    count(c);
    if (e != cudaSuccess) return fail_cuda(c, e, "score launch");
  }
  if (quality) {
    cudaError_t e = launch_quality(c->d, scores, quality, st, &c->launches_i);
    count(c);
    if (e != cudaSuccess) return fail_cuda(c, e, "quality launch");
  }
  return SWAM_OK;
}

int swam_score_noalloc(swam_ctx* c, const void* q, const void* k, float* scores, void* stream) {
  Range trace_range("swam_score_noalloc");
  if (!c || !q || !k || !scores) return fail(c, SWAM_ERR_INVALID_ARG, "swam_score_noalloc: null argument");
  if (!aligned16(q) || !aligned16(k) || !aligned16(scores))
    return fail(c, SWAM_ERR_INVALID_ARG, "swam_score_noalloc: misaligned pointer");
  if (int r = check_device(c)) return r;   // the built-in array's address differs from device to device
  if (static_scratch_need(c->d) > kStaticScratchBytes) {
    snprintf(c->err, sizeof(c->err), "swam_score_noalloc: this shape needs %zu bytes of scratch, the built-in array holds %zu",
             static_scratch_need(c->d), (size_t)kStaticScratchBytes);
    return SWAM_ERR_UNSUPPORTED;
  }
  float* lse = nullptr;
  void* partial = nullptr;
  cudaError_t e = static_scratch(c->d, &lse, &partial);
  if (e != cudaSuccess) return fail_cuda(c, e, "swam_score_noalloc: cudaGetSymbolAddress");
  cudaStream_t st = (cudaStream_t)stream;
  // every normaliser and every partial is written before it is read, so nothing has to start at zero
  e = launch_action_lse(c->d, q, k, lse, partial, st, &c->launches_i, action_keys(c));
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "action lse launch");
  e = launch_score(c->d, c->alpha, q, k, lse, scores, st, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "score launch");
  return SWAM_OK;
}

int swam_select(swam_ctx* c, const float* scores, int32_t* sel_idx, int32_t* pack_map, int32_t* inv_map, void* stream) {
  Range trace_range("swam_select");
  if (!c || !scores) return fail(c, SWAM_ERR_INVALID_ARG, "swam_select: null argument");
  if (int r = need_ws(c)) return r;
  cudaError_t e = launch_select(c->d, scores, nullptr, sel_idx, pack_map, inv_map, (int*)(c->ws + c->off_status),
                                (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "select launch");
  return SWAM_OK;
}

int swam_aggregate(swam_ctx* c, const float* layer_scores, const float* layer_quality, int32_t n_layers, int32_t k_layer,
                   float* v_core, float* v_all, int32_t* core_layers, void* stream) {
  Range trace_range("swam_aggregate");
  if (!c || !layer_scores || !layer_quality || !v_core || !v_all) return fail(c, SWAM_ERR_INVALID_ARG, "swam_aggregate: null argument");
  if (n_layers <= 0 || k_layer <= 0 || k_layer > n_layers) return fail(c, SWAM_ERR_INVALID_ARG, "swam_aggregate: need 0 < k_layer <= n_layers");
  if (n_layers > max_layers()) return fail(c, SWAM_ERR_UNSUPPORTED, "swam_aggregate: too many layers");
  cudaError_t e = launch_aggregate(c->d, layer_scores, layer_quality, n_layers, k_layer, v_core, v_all, core_layers,
                                   (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "aggregate launch");
  return SWAM_OK;
}

int swam_select_maps(swam_ctx* c, const float* core_scores, const float* anchor_scores, int32_t* sel_idx, int32_t* pack_map,
                     int32_t* inv_map, void* stream) {
  Range trace_range("swam_select_maps");
  if (!c || !core_scores || !anchor_scores) return fail(c, SWAM_ERR_INVALID_ARG, "swam_select_maps: null argument");
  if (int r = need_ws(c)) return r;
  cudaError_t e = launch_select(c->d, core_scores, anchor_scores, sel_idx, pack_map, inv_map, (int*)(c->ws + c->off_status),
                                (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "select launch");
  return SWAM_OK;
}

int swam_pack(swam_ctx* c, const void* q, const void* k, const void* v, const int32_t* pack_map, void* qp, void* kp,
              void* vp, void* stream) {
  Range trace_range("swam_pack");
  if (!c || !pack_map) return fail(c, SWAM_ERR_INVALID_ARG, "swam_pack: null argument");
  if ((!q) != (!qp) || (!k) != (!kp) || (!v) != (!vp)) return fail(c, SWAM_ERR_INVALID_ARG, "swam_pack: unpaired tensor");
  const void* ptrs[6] = {q, k, v, qp, kp, vp};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return fail(c, SWAM_ERR_INVALID_ARG, "swam_pack: misaligned pointer");
  if (int r = need_ws(c)) return r;
  const void* src[3] = {q, k, v};
  void* dst[3] = {qp, kp, vp};
  cudaError_t e = launch_pack(c->d, src, dst, pack_map, (int*)(c->ws + c->off_status), (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "pack launch");
  return SWAM_OK;
}

int swam_sparse_attn(swam_ctx* c, const void* qp, const void* kp, const void* vp, int32_t seq_len, void* out_p, float* lse,
                     void* stream) {
  Range trace_range("swam_sparse_attn");
  if (!c || !qp || !kp || !vp || !out_p) return fail(c, SWAM_ERR_INVALID_ARG, "swam_sparse_attn: null argument");
  if (seq_len <= 0 || seq_len > c->d.L) return fail(c, SWAM_ERR_INVALID_ARG, "swam_sparse_attn: seq_len out of range");
  if (!aligned16(qp) || !aligned16(kp) || !aligned16(vp) || !aligned16(out_p))
    return fail(c, SWAM_ERR_INVALID_ARG, "swam_sparse_attn: misaligned pointer");
  return run_attention(c, qp, kp, vp, seq_len, out_p, lse, 0, seq_len, (cudaStream_t)stream);
}

int swam_scatter(swam_ctx* c, const void* out_p, const int32_t* pack_map, const int32_t* inv_map, const void* cached,
                 void* out, void* stream) {
  Range trace_range("swam_scatter");
  if (!c || !out_p || !pack_map || !out || !cached) return fail(c, SWAM_ERR_INVALID_ARG, "swam_scatter: null argument");
  if (cached != out && !inv_map) return fail(c, SWAM_ERR_INVALID_ARG, "swam_scatter: inv_map needed when cached != out");
  if (!aligned16(out_p) || !aligned16(cached) || !aligned16(out)) return fail(c, SWAM_ERR_INVALID_ARG, "swam_scatter: misaligned pointer");
  if (int r = need_ws(c)) return r;
  cudaError_t e = launch_scatter(c->d, out_p, pack_map, inv_map, cached, out, (int*)(c->ws + c->off_status),
                                 (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "scatter launch");
  return SWAM_OK;
}

int swam_step(swam_ctx* c, const void* q, const void* k, const void* v, int32_t mode, void* out, void* stream) {
  Range trace_range("swam_step");
  if (!c || !q || !k || !v || !out) return fail(c, SWAM_ERR_INVALID_ARG, "swam_step: null argument");
  if (mode != SWAM_REUSE && mode != SWAM_REFRESH_FULL && mode != SWAM_REFRESH_LIGHT)
    return fail(c, SWAM_ERR_INVALID_ARG, "swam_step: unknown mode");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
    return fail(c, SWAM_ERR_INVALID_ARG, "swam_step: misaligned pointer");
  if (int r = need_ws(c)) return r;
  if (mode == SWAM_REUSE && !c->has_selection)
    return fail(c, SWAM_ERR_STATE, "swam_step: reuse requested before any refresh");
  cudaStream_t st = (cudaStream_t)stream;
  const Dims& d = c->d;
  float* scores = (float*)(c->ws + c->off_scores);
  float* quality = (float*)(c->ws + c->off_quality);
  float* lse = (float*)(c->ws + c->off_lse);
  int32_t* sel = (int32_t*)(c->ws + c->off_sel);
  int32_t* pm = (int32_t*)(c->ws + c->off_pack);
  int32_t* im = (int32_t*)(c->ws + c->off_inv);

  if (mode == SWAM_REFRESH_FULL) {
    // dense joint attention fills the cache and yields the action-row normalisers over all L keys
    Range stage("dense_attention");
    if (int r = run_attention(c, q, k, v, d.L, out, lse, d.L - d.H, d.H, st)) return r;
  }
  if (mode != SWAM_REUSE) {
    const float* lse_in = (mode == SWAM_REFRESH_FULL) ? lse : nullptr;
    // the Eq. 9 diagnostics ride along with the selection kernel, which holds the scores in shared memory anyway
    const bool fold = select_can_fold_quality(d);
    if (int r = swam_score(c, q, k, lse_in, scores, fold ? nullptr : quality, stream)) return r;
    Range stage("select");
    cudaError_t e = launch_select(d, scores, nullptr, sel, pm, im, (int*)(c->ws + c->off_status), st, &c->launches_i,
                                  quality);
    count(c);
    if (e != cudaSuccess) return fail_cuda(c, e, "select launch");
    c->has_selection = true;
    c->maps_own = true;     // built by the selection kernel: the observed rows lead the packed sequence in order
  }
  if (mode != SWAM_REFRESH_FULL && c->sparse_path != SWAM_SPARSE_STAGED && d.dtype == SWAM_BF16 && d.D >= 64 &&
      c->attn_variant == SWAM_ATTN_AUTO) {
    // K and V are packed by the copy kernel (every query tile of a head reads them); the attention kernel fetches
    // its query rows from the full Q itself and writes each result row straight to its place in `out`.  The omitted
    // rows keep the cached value they already hold (Eq. 7), so neither a packed Q, nor a packed output, nor a scatter
    // pass exist.
    // With SWAM_SPARSE_FUSED_KV the kernel gathers the key and value rows as well and nothing is packed.
    const bool gather_kv = c->sparse_path == SWAM_SPARSE_FUSED_KV;
    const void* kp = k;
    const void* vp = v;
    // The observed tokens lead the packed sequence as they lead the full one: whole key tiles of them are read from
    // the full K and V and are left out of the pack.
    const int direct_rows = (gather_kv || !c->maps_own) ? 0 : (d.n_obs / 128) * 128;
    if (!gather_kv) {
      kp = c->ws + c->off_kp;
      vp = c->ws + c->off_vp;
      Range stage_pack("swam_pack");
      const void* src[3] = {nullptr, k, v};
      void* dst[3] = {nullptr, c->ws + c->off_kp, c->ws + c->off_vp};
      cudaError_t e = launch_pack(d, src, dst, pm, (int*)(c->ws + c->off_status), st, &c->launches_i, direct_rows);
      count(c);
      if (e != cudaSuccess) return fail_cuda(c, e, "pack launch");
    }
    Range stage("packed_attention");
    AttnArgs a{q, kp, vp, out, nullptr, 0, 0, d.B, d.Lp, d.N_h, d.D, d.scale, d.N_kv};
    a.k_full = k;
    a.v_full = v;
    a.direct_rows = direct_rows;
    set_visibility(c, a);
    cudaError_t e = launch_attn_bf16_tc_gather(a, pm, d.L, gather_kv, (int*)(c->ws + c->off_status), c->ws + c->off_attn,
                                               c->attn_scratch, st, &c->launches_i);
    count(c);
    if (e != cudaSuccess) return fail_cuda(c, e, "fused sparse attention launch");
  } else if (mode != SWAM_REFRESH_FULL) {
    void* qp = c->ws + c->off_qp;
    void* kp = c->ws + c->off_kp;
    void* vp = c->ws + c->off_vp;
    void* op = c->ws + c->off_op;
    if (int r = swam_pack(c, q, k, v, pm, qp, kp, vp, stream)) return r;
    {
      Range stage("packed_attention");
      if (int r = run_attention(c, qp, kp, vp, d.Lp, op, nullptr, 0, 0, st)) return r;
    }
    if (int r = swam_scatter(c, op, pm, im, out, out, stream)) return r;
  }
  return SWAM_OK;
}

int swam_step_host(swam_ctx* c, const void* q_host, const void* k_host, const void* v_host, int32_t mode, void* out_host,
                   void* stream) {
  Range trace_range("swam_step_host");
  if (!c || !q_host || !k_host || !v_host || !out_host) return fail(c, SWAM_ERR_INVALID_ARG, "swam_step_host: null argument");
  if (!c->io) return fail(c, SWAM_ERR_WORKSPACE, "swam_step_host: no staging area bound");
  cudaStream_t st = (cudaStream_t)stream;
  const size_t fb = full_bytes(c->d), kvb = kv_full_bytes(c->d), stride = align_up(fb, 256);
  // Three-stage pipeline over three input slots: this step's inputs travel on a copy-in stream while the previous
  // steps still compute, the step runs on the caller's stream, and the result leaves on the copy-out stream while
  // the next inputs arrive (PCIe is full duplex).  The third slot lets the whole-tensor copy of the refresh step after
  // a reuse step start while the refresh step before it still computes (the reuse step's own rows cannot: they are
  // only known once that step has rebuilt the maps), so the host-to-device link never idles.
  const int slot = (int)(c->host_steps % 3);
  unsigned char* in = c->io + (size_t)slot * 3 * stride;
  void* dq = in;
  void* dk = in + stride;
  void* dv = in + 2 * stride;
  void* dout = c->io + 9 * stride;
  // A reuse step reads only the rows its maps retain: where the caller's buffers are pinned memory the device can
  // address, a kernel on the row-fetch stream brings just those rows across PCIe (Sec. 4.2's compact execution applied
  // to the transfer as well); the other rows of the slot keep stale values that the sparse step never touches.
  const void* mapped[3] = {nullptr, nullptr, nullptr};
  bool retained_only = mode == SWAM_REUSE && c->has_selection && c->host_rows == SWAM_HOST_ROWS_RETAINED && c->ws;
  if (retained_only) {
    const void* host[3] = {q_host, k_host, v_host};
    for (int i = 0; i < 3 && retained_only; ++i) {
      cudaPointerAttributes at;
      if (cudaPointerGetAttributes(&at, host[i]) != cudaSuccess || at.type != cudaMemoryTypeHost || !at.devicePointer) {
        cudaGetLastError();          // pageable or foreign memory: plain copies of the whole tensors below
        retained_only = false;
      } else {
        mapped[i] = at.devicePointer;
      }
    }
  }
  cudaStream_t s_copy = retained_only ? c->s_rows : c->s_in;
  cudaError_t e = cudaStreamWaitEvent(s_copy, c->ev_done[slot], 0);   // the step three calls ago has read this slot
  if (retained_only) {
    // The observed rows are retained whatever the selection and lead every sample in one block: they travel as plain
    // strided copies on the whole-copy stream at once (they need not wait for the maps).  With maps that this context
    // did not build itself the block is not assumed and the kernel fetches every listed row.
    const int n_block = c->maps_own ? c->d.n_obs : 0;
    if (n_block > 0) {
      const size_t row = fb / ((size_t)c->d.B * c->d.L), row_kv = kvb / ((size_t)c->d.B * c->d.L);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(c->s_in, c->ev_done[slot], 0);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(dq, c->d.L * row, q_host, c->d.L * row, n_block * row, c->d.B, cudaMemcpyHostToDevice, c->s_in);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(dk, c->d.L * row_kv, k_host, c->d.L * row_kv, n_block * row_kv, c->d.B, cudaMemcpyHostToDevice, c->s_in);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(dv, c->d.L * row_kv, v_host, c->d.L * row_kv, n_block * row_kv, c->d.B, cudaMemcpyHostToDevice, c->s_in);
      if (e == cudaSuccess) e = cudaEventRecord(c->ev_obs, c->s_in);
    }
    // the maps are final once everything already on the caller's stream has run (the previous step, or a selection
    // installed since)
    if (e == cudaSuccess) e = cudaEventRecord(c->ev_pre, st);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s_copy, c->ev_pre, 0);
    if (e == cudaSuccess) {
      void* dst[3] = {dq, dk, dv};
      e = launch_host_rows(c->d, mapped, dst, (const int32_t*)(c->ws + c->off_pack), (int*)(c->ws + c->off_status), s_copy,
                           &c->launches_i, n_block);
      count(c);
    }
    if (e == cudaSuccess && n_block > 0) e = cudaStreamWaitEvent(s_copy, c->ev_obs, 0);
  } else {
    if (e == cudaSuccess) e = cudaMemcpyAsync(dq, q_host, fb, cudaMemcpyHostToDevice, s_copy);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dk, k_host, kvb, cudaMemcpyHostToDevice, s_copy);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v_host, kvb, cudaMemcpyHostToDevice, s_copy);
  }
  if (e == cudaSuccess) e = cudaEventRecord(c->ev_h2d[slot], s_copy);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_h2d[slot], 0);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c->ev_d2h, 0);     // the previous result has been copied out
  if (e != cudaSuccess) return fail_cuda(c, e, "host to device copy");
  if (int r = swam_step(c, dq, dk, dv, mode, dout, stream)) return r;
  e = cudaEventRecord(c->ev_done[slot], st);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(c->s_out, c->ev_done[slot], 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, dout, fb, cudaMemcpyDeviceToHost, c->s_out);
  if (e == cudaSuccess) e = cudaEventRecord(c->ev_d2h, c->s_out);
  if (e != cudaSuccess) return fail_cuda(c, e, "device to host copy");
  ++c->host_steps;
  return SWAM_OK;
}

int swam_host_join(swam_ctx* c, void* stream) {
  Range trace_range("swam_host_join");
  if (!c) return SWAM_ERR_INVALID_ARG;
  if (!c->s_in) return fail(c, SWAM_ERR_WORKSPACE, "swam_host_join: no staging area bound");
  cudaError_t e = cudaStreamWaitEvent((cudaStream_t)stream, c->ev_d2h, 0);
  if (e != cudaSuccess) return fail_cuda(c, e, "swam_host_join");
  return SWAM_OK;
}

int swam_get_selection(const swam_ctx* c, const int32_t** sel_idx, const int32_t** pack_map, const int32_t** inv_map) {
  if (!c || !c->ws) return SWAM_ERR_WORKSPACE;
  if (sel_idx) *sel_idx = (const int32_t*)(c->ws + c->off_sel);
  if (pack_map) *pack_map = (const int32_t*)(c->ws + c->off_pack);
  if (inv_map) *inv_map = (const int32_t*)(c->ws + c->off_inv);
  return SWAM_OK;
}

int swam_set_selection(swam_ctx* c, const int32_t* sel_idx, const int32_t* pack_map, const int32_t* inv_map, void* stream) {
  Range trace_range("swam_set_selection");
  if (!c || !sel_idx || !pack_map || !inv_map) return fail(c, SWAM_ERR_INVALID_ARG, "swam_set_selection: null argument");
  if (int r = need_ws(c)) return r;
  const Dims& d = c->d;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(c->ws + c->off_sel, sel_idx, (size_t)d.B * d.F * d.K * sizeof(int32_t),
                                  cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(c->ws + c->off_pack, pack_map, (size_t)d.B * d.Lp * sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(c->ws + c->off_inv, inv_map, (size_t)d.B * d.L * sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
  if (e != cudaSuccess) return fail_cuda(c, e, "swam_set_selection");
  c->has_selection = true;
  c->maps_own = false;     // installed maps are the caller's: the observed rows need not lead them
  return SWAM_OK;
}

// the state blocks are laid out back to back in the workspace: scores, quality, normalisers, selection, maps
int swam_state_bytes(const swam_ctx* c, size_t* bytes) {
  if (!c || !bytes) return SWAM_ERR_INVALID_ARG;
  *bytes = c->off_scratch - c->off_scores;
  return SWAM_OK;
}

int swam_state_export(swam_ctx* c, void* dev_buf, void* stream) {
  Range trace_range("swam_state_export");
  if (!c || !dev_buf) return fail(c, SWAM_ERR_INVALID_ARG, "swam_state_export: null argument");
  if (int r = need_ws(c)) return r;
  if (!c->has_selection) return fail(c, SWAM_ERR_STATE, "swam_state_export: no refresh step has run yet");
  cudaError_t e = cudaMemcpyAsync(dev_buf, c->ws + c->off_scores, c->off_scratch - c->off_scores, cudaMemcpyDeviceToDevice,
                                  (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e, "swam_state_export");
  return SWAM_OK;
}

int swam_state_import(swam_ctx* c, const void* dev_buf, void* stream) {
  Range trace_range("swam_state_import");
  if (!c || !dev_buf) return fail(c, SWAM_ERR_INVALID_ARG, "swam_state_import: null argument");
  if (int r = need_ws(c)) return r;
  cudaError_t e = cudaMemcpyAsync(c->ws + c->off_scores, dev_buf, c->off_scratch - c->off_scores, cudaMemcpyDeviceToDevice,
                                  (cudaStream_t)stream);
  if (e != cudaSuccess) return fail_cuda(c, e, "swam_state_import");
  c->has_selection = true;
  c->maps_own = false;     // restored maps: their origin is not known
  return SWAM_OK;
}

int swam_get_scores(const swam_ctx* c, const float** scores, const float** lse_action, const float** quality) {
  if (!c || !c->ws) return SWAM_ERR_WORKSPACE;
  if (scores) *scores = (const float*)(c->ws + c->off_scores);
  if (lse_action) *lse_action = (const float*)(c->ws + c->off_lse);
  if (quality) *quality = (const float*)(c->ws + c->off_quality);
  return SWAM_OK;
}

int swam_check(swam_ctx* c, void* stream) {
  Range trace_range("swam_check");
  if (!c) return SWAM_ERR_INVALID_ARG;
  if (int r = need_ws(c)) return r;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e == cudaSuccess && c->s_in) e = cudaStreamSynchronize(c->s_in);
  if (e == cudaSuccess && c->s_rows) e = cudaStreamSynchronize(c->s_rows);
  if (e == cudaSuccess && c->s_out) e = cudaStreamSynchronize(c->s_out);
  if (e != cudaSuccess) return fail_cuda(c, e, "cudaStreamSynchronize");
  int word = 0;
  e = cudaMemcpy(&word, c->ws + c->off_status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(c, e, "status read");
  if (word != 0) {
    // the arrival tickets of the one-pass scorer too: a launch that gave up may have left some behind
    e = cudaMemset(c->ws + c->off_status, 0, c->off_counters - c->off_status + score_counter_bytes(c->d));
    if (e != cudaSuccess) return fail_cuda(c, e, "status clear");
    snprintf(c->err, sizeof(c->err), "device status word 0x%x%s%s%s", word, (word & ST_BAD_MAP) ? " [map entry out of range]" : "",
             (word & ST_BAD_COUNT) ? " [selection count mismatch]" : "", (word & ST_TIMEOUT) ? " [bounded wait ran out]" : "");
    return (word & ST_TIMEOUT) ? SWAM_ERR_TIMEOUT : SWAM_ERR_DEVICE_CHECK;
  }
  return SWAM_OK;
}

int swam_selftest_timeout(swam_ctx* c, uint64_t limit_cycles, void* stream) {
  if (!c) return SWAM_ERR_INVALID_ARG;
  if (limit_cycles == 0 || limit_cycles > 100000000ull)
    return fail(c, SWAM_ERR_INVALID_ARG, "swam_selftest_timeout: limit must lie in [1, 1e8] cycles");
  if (int r = need_ws(c)) return r;
  if (int r = check_device(c)) return r;
  cudaError_t e = launch_wait_probe((int*)(c->ws + c->off_status), limit_cycles, (cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "wait self-test launch");
  return SWAM_OK;
}

int swam_launch_floor(swam_ctx* c, void* stream) {
  if (!c) return SWAM_ERR_INVALID_ARG;
  cudaError_t e = launch_noop((cudaStream_t)stream, &c->launches_i);
  count(c);
  if (e != cudaSuccess) return fail_cuda(c, e, "empty kernel launch");
  return SWAM_OK;
}

int swam_set_option(swam_ctx* c, int32_t option, int32_t value) {
  if (!c) return SWAM_ERR_INVALID_ARG;
  if (option == SWAM_OPT_ATTN_VARIANT && (value == SWAM_ATTN_AUTO || value == SWAM_ATTN_WARP_MMA)) {
    c->attn_variant = value;
    return SWAM_OK;
  }
  if (option == SWAM_OPT_VISIBILITY) {
    const int o = value & 3, f = (value >> 2) & 3, a = (value >> 4) & 3;
    if ((value >> 6) != 0 || o > SWAM_SEES_ALL || f > SWAM_SEES_ALL || a > SWAM_SEES_ALL)
      return fail(c, SWAM_ERR_INVALID_ARG, "swam_set_option: malformed visibility value");
    if (f < SWAM_SEES_FUTURE || a < SWAM_SEES_FUTURE)
      return fail(c, SWAM_ERR_INVALID_ARG, "swam_set_option: future and action rows must see the future tokens");
    c->sees[0] = o; c->sees[1] = f; c->sees[2] = a;
    return SWAM_OK;
  }
  if (option == SWAM_OPT_HOST_ROWS && (value == SWAM_HOST_ROWS_RETAINED || value == SWAM_HOST_ROWS_ALL)) {
    c->host_rows = value;
    return SWAM_OK;
  }
  if (option == SWAM_OPT_SPARSE_PATH &&
      (value == SWAM_SPARSE_FUSED || value == SWAM_SPARSE_STAGED || value == SWAM_SPARSE_FUSED_KV)) {
    c->sparse_path = value;
    return SWAM_OK;
  }
  return fail(c, SWAM_ERR_INVALID_ARG, "swam_set_option: unknown option or value");
}

int swam_launch_count(const swam_ctx* c, int64_t* n) {
  if (!c || !n) return SWAM_ERR_INVALID_ARG;
  *n = c->launches;
  return SWAM_OK;
}

}  // extern "C"
