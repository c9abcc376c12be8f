// C ABI entry points that route to the kernels, and the whole-net step (Sec. 4.2 for arbitrary
// depth: every layer input is stored through its own mask, dW_l comes from store l, the rest of
// backprop is exact).
#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace rad {

int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RAD_ECUDA;
  static int cached_dev = -1, cached_rc = RAD_ECUDA;
  if (dev == cached_dev) return cached_rc;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return RAD_ECUDA;
  cached_rc = (major == 10) ? RAD_OK : RAD_EUNSUPPORTED;
  cached_dev = dev;
  return cached_rc;
}

static int64_t g_launches = 0;
void count_launch(int n) { g_launches += n; }

static uint64_t g_wait_limit_ns = 2000000000ull;   // 2 s: far beyond any legitimate wait in these kernels
uint64_t wait_limit_ns() { return g_wait_limit_ns; }

namespace {

// Named range on the host timeline for a profiler that is attached (header-only NVTX: a no-op otherwise).
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

bool valid_dtype(int d) { return d == RAD_F32 || d == RAD_BF16; }
int64_t esize(int dtype) { return dtype == RAD_BF16 ? 2 : 4; }

// Tile-major twin of a static-shape (RAD_ROWS_SAMPLE) store, laid out in a workspace: same key, same mask.
struct TileTwin { rad_store st; int64_t bytes; };
TileTwin tile_twin(const rad_store* rows, char* ws) {
  TileTwin t;
  const int64_t k = draws_per_row_host(rows->p, rows->D);
  const int64_t ntiles = ceil_div(rows->B, kTileRows) * ceil_div(rows->D, kTileCols);
  const int64_t cap = round_up(rows->B * k + ntiles * (kValueAlign - 1), kValueAlign);
  int64_t off = 0;
  auto take = [&](int64_t bytes) { const int64_t at = off; off += round_up(bytes, 256); return at; };
  t.st = *rows;
  t.st.variant = RAD_DIFFERENT_SAMPLE;
  t.st.values_capacity = cap;
  t.st.values_ld = 0;
  const int64_t v = take(cap * esize(rows->dtype)), kb = take(ntiles * kTileWords * 4), of = take((ntiles + 1) * 4), nz = take(16);
  t.st.values = ws != nullptr ? ws + v : nullptr;
  t.st.keepbits = ws != nullptr ? reinterpret_cast<uint32_t*>(ws + kb) : nullptr;
  t.st.offsets = ws != nullptr ? reinterpret_cast<uint32_t*>(ws + of) : nullptr;
  t.st.nnz = ws != nullptr ? reinterpret_cast<int64_t*>(ws + nz) : nullptr;
  t.st.relubits = nullptr;
  t.bytes = off;
  return t;
}

// Full different-sample twin of a RAD_REDRAWN_SAMPLE store for the backward pass: keep bits, row offsets, tile
// offsets and counts are drawn again into the workspace, the values are the held ones.
TileTwin redrawn_twin(const rad_store* held, char* ws) {
  TileTwin t;
  const int64_t ntiles = ceil_div(held->B, kTileRows) * ceil_div(held->D, kTileCols);
  int64_t off = 0;
  auto take = [&](int64_t bytes) { const int64_t at = off; off += round_up(bytes, 256); return at; };
  t.st = *held;
  t.st.variant = RAD_DIFFERENT_SAMPLE;
  const int64_t kb = take(redrawn_index_bytes(held->B, held->D)), of = take((ntiles + 1) * 4), nz = take(16);
  t.st.keepbits = ws != nullptr ? reinterpret_cast<uint32_t*>(ws + kb) : reinterpret_cast<uint32_t*>(256);
  t.st.offsets = ws != nullptr ? reinterpret_cast<uint32_t*>(ws + of) : reinterpret_cast<uint32_t*>(256);
  t.st.nnz = ws != nullptr ? reinterpret_cast<int64_t*>(ws + nz) : reinterpret_cast<int64_t*>(256);
  t.st.relubits = nullptr;
  t.bytes = off;
  return t;
}
bool redrawn_args_ok(const rad_store* st) {
  return st != nullptr && st->B > 0 && st->D > 0 && valid_dtype(st->dtype) && st->values != nullptr &&
         st->offsets != nullptr && st->nnz != nullptr && keep_threshold_host(st->p) != 0 &&
         (st->law == RAD_LAW_BERNOULLI || st->law == RAD_LAW_FIXED) &&
         (double)st->B * (double)st->D < 4294967296.0 * 0.75;
}

bool store_args_ok(const rad_store* st) {
  if (st == nullptr || st->B <= 0 || st->D <= 0) return false;
  if (st->variant != RAD_DIFFERENT_SAMPLE && st->variant != RAD_SAME_SAMPLE) return false;
  if (!valid_dtype(st->dtype)) return false;
  if (st->values == nullptr || st->keepbits == nullptr || st->offsets == nullptr || st->nnz == nullptr) return false;
  if (keep_threshold_host(st->p) == 0) return false;
  if (st->variant == RAD_SAME_SAMPLE && (st->values_ld <= 0 || st->values_ld % 8 != 0)) return false;
  return true;
}

// ---- workspace plan of rad_mlp_step ---------------------------------------------------------------
struct LayerPlan {
  int64_t values, keepbits, offsets, nnz, relubits, preact;   // byte offsets; -1 if absent
  int64_t capacity, values_ld;
};
struct StepPlan {
  LayerPlan layer[64];
  int64_t act[2], dz[2], logits, scratch, status_unused;
  int64_t scratch_bytes, total;
  rad_step_stats stats;
};

int make_plan(const rad_mlp_desc* net, StepPlan* plan) {
  if (net == nullptr || net->dims == nullptr || net->L < 1 || net->L > 64 || net->B <= 0) return RAD_EINVAL;
  if (!valid_dtype(net->dtype)) return RAD_EINVAL;
  if (net->variant != RAD_DIFFERENT_SAMPLE && net->variant != RAD_SAME_SAMPLE && net->variant != RAD_PROJECT &&
      net->variant != RAD_REDRAWN_SAMPLE)
    return RAD_EINVAL;
  if (net->act != RAD_ACT_RELU && net->act != RAD_ACT_GELU) return RAD_EINVAL;
  if (keep_threshold_host(net->p) == 0) return RAD_EINVAL;
  if (net->law != RAD_LAW_BERNOULLI && net->law != RAD_LAW_REPLACE && net->law != RAD_LAW_FIXED) return RAD_EINVAL;
  const int64_t B = net->B, es = esize(net->dtype);
  int64_t off = 0;
  auto take = [&](int64_t bytes) { const int64_t at = off; off += round_up(bytes, 256); return at; };
  rad_step_stats st = {};
  int64_t max_hidden = 8, max_out = 8, scratch = B * 4;
  for (int l = 0; l < net->L; ++l) {
    const int64_t D = net->dims[l], H = net->dims[l + 1];
    if (D <= 0 || H <= 0) return RAD_EINVAL;
    rad_store_sizes sz;
    int rc = rad_store_size_query_law(net->variant, net->dtype, net->law, B, D, net->p, &sz);
    if (rc != RAD_OK) return rc;
    LayerPlan& lp = plan->layer[l];
    lp.capacity = sz.values_typical;
    lp.values_ld = sz.values_ld_typical;
    lp.values = take(lp.capacity * es);
    lp.keepbits = take(sz.keepbits_words * 4);
    lp.offsets = take(sz.offsets_words * 4);
    lp.nnz = take(16);
    lp.relubits = (l > 0 && net->act == RAD_ACT_RELU) ? take(sz.relubits_words * 4) : -1;
    lp.preact = (l > 0 && net->act == RAD_ACT_GELU) ? take(B * D * es) : -1;
    st.value_bytes += lp.capacity * es;
    st.index_bytes += (sz.keepbits_words + sz.offsets_words) * 4;
    if (lp.relubits >= 0) st.relu_bytes += sz.relubits_words * 4;
    if (lp.preact >= 0) st.preact_bytes += B * D * es;
    st.full_backprop_bytes += B * D * es;
    if (l > 0) max_hidden = max(max_hidden, D);
    max_out = max(max_out, H);
    scratch = max(scratch, sz.workspace_bytes);
    scratch = max(scratch, column_sums_workspace(B, H));
    rad_store tmp = {};
    tmp.variant = net->variant; tmp.dtype = net->dtype; tmp.B = B; tmp.D = D; tmp.p = net->p;
    tmp.law = net->law;
    tmp.values_ld = lp.values_ld; tmp.values_capacity = lp.capacity;
    int64_t dw_scratch = 0;
    rc = rad_weight_grad_workspace(&tmp, H, &dw_scratch);
    if (rc != RAD_OK) return rc;
    scratch = max(scratch, dw_scratch);
  }
  st.unsampled_bytes = B * net->dims[net->L] * 4;
  st.full_backprop_bytes += st.unsampled_bytes;
  plan->act[0] = take(B * max_hidden * es);
  plan->act[1] = take(B * max_hidden * es);
  plan->dz[0] = take(B * max_out * es);
  plan->dz[1] = take(B * max_out * es);
  plan->logits = take(B * net->dims[net->L] * 4);
  plan->scratch_bytes = round_up(scratch, 256);
  plan->scratch = take(plan->scratch_bytes);
  plan->total = off;
  plan->stats = st;
  return RAD_OK;
}

}  // namespace
}  // namespace rad

using namespace rad;

extern "C" int64_t rad_launch_count(void) { return g_launches; }
extern "C" int32_t rad_sm_pairs(void) { return sm_pairs(); }

extern "C" uint64_t rad_set_wait_limit_ns(uint64_t limit_ns) {
  const uint64_t prev = g_wait_limit_ns;
  if (limit_ns != 0) g_wait_limit_ns = limit_ns;
  return prev;
}

extern "C" int rad_wait_probe(int32_t which, uint64_t limit_ns, int32_t* dev_status, void* stream) {
  if (limit_ns == 0 || limit_ns > 1000000000ull) return RAD_EINVAL;      // a probe waits a second at most
  const int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  switch (which) {
    case RAD_WAIT_PAIR_BARRIER: return launch_wait_probe_pair(limit_ns, dev_status, s);
    case RAD_WAIT_PIPE_BARRIER: return launch_wait_probe_pipe(limit_ns, dev_status, s);
    case RAD_WAIT_LOOKBACK:     return launch_wait_probe_lookback(limit_ns, dev_status, s);
    default: return RAD_EINVAL;
  }
}

extern "C" const char* rad_version(void) { return "rad-b200 0.1 (sm_100a)"; }

extern "C" const char* rad_strerror(int code) {
  switch (code) {
    case RAD_OK: return "ok";
    case RAD_EINVAL: return "invalid argument";
    case RAD_EUNSUPPORTED: return "unsupported device or alignment";
    case RAD_ECUDA: return "CUDA call failed";
    case RAD_EWORKSPACE: return "workspace too small";
    case RAD_ELIMIT: return "problem larger than the built-in scratch buffer";
    case RAD_DEV_ECAPACITY: return "device: compact store capacity exceeded";
    case RAD_DEV_ETIMEOUT: return "device: bounded wait expired";
    case RAD_DEV_EINTERNAL: return "device: index out of range, access skipped";
    default: return "unknown code";
  }
}

namespace rad {
namespace {
// Does the input gradient of these operands run on the tensor cores?
bool input_grad_on_tc(int32_t dtype, int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz, const void* W,
                      int64_t ldw, const void* z_prev, int64_t ld_zprev, const void* dZ_prev, int64_t ldp) {
  return dtype == RAD_BF16 && tc_shape_ok(B, D, H, dZ, ldz, W, ldw) && ((uintptr_t)dZ_prev & 15) == 0 && ldp % 8 == 0 &&
         (z_prev == nullptr || (((uintptr_t)z_prev & 15) == 0 && ld_zprev % 8 == 0));
}

// rad_linear_weight_grad for a bitmask or column-list store (index held or drawn again); where the contraction
// runs on the CUDA cores and passes over dZ anyway, it also leaves the bias gradient in `db` (*db_written says
// whether it did).
// ig (optional): the input gradient of the same layer; where both contractions run on CUDA cores they share one
// launch and *ig_done is set, otherwise the caller runs rad_linear_input_grad as usual.
int weight_grad_and_bias(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW, int64_t ldw, void* workspace,
                         int64_t workspace_bytes, int32_t* dev_status, void* stream, float* db, bool* db_written,
                         const SimtInputGrad* ig = nullptr, bool* ig_done = nullptr) {
  if (db_written != nullptr) *db_written = false;
  if (ig_done != nullptr) *ig_done = false;
  if (st != nullptr && st->variant == RAD_REDRAWN_SAMPLE) {
    // the index part from the key alone, into the workspace; then the contraction of a different-sample store
    if (!redrawn_args_ok(st) || dZ == nullptr || dW == nullptr || H <= 0 || ldz < H || ldw < H) return RAD_EINVAL;
    int rcd = check_device();
    if (rcd != RAD_OK) return rcd;
    int64_t need = 0;
    rcd = rad_weight_grad_workspace(st, H, &need);
    if (rcd != RAD_OK) return rcd;
    if (workspace == nullptr || workspace_bytes < need || ((uintptr_t)workspace & 255) != 0) return RAD_EWORKSPACE;
    const TileTwin t = redrawn_twin(st, static_cast<char*>(workspace));
    rcd = launch_store_index(&t.st, false, dev_status, static_cast<cudaStream_t>(stream));
    if (rcd != RAD_OK) return rcd;
    return weight_grad_and_bias(&t.st, dZ, ldz, H, dW, ldw, static_cast<char*>(workspace) + t.bytes, workspace_bytes - t.bytes,
                                dev_status, stream, db, db_written, ig, ig_done);
  }
  if (!store_args_ok(st) || dZ == nullptr || dW == nullptr || H <= 0 || ldz < H || ldw < H) return RAD_EINVAL;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (st->dtype == RAD_BF16 && tc_shape_ok(st->B, st->D, H, dZ, ldz, st->values, 8) &&
      ((uintptr_t)dW & 15) == 0 && ldw % 4 == 0) {
    if (workspace_bytes < tc_weight_grad_workspace(st, H) || (workspace == nullptr && tc_weight_grad_workspace(st, H) > 0))
      return RAD_EWORKSPACE;
    return tc_weight_grad(st, dZ, ldz, H, dW, ldw, workspace, workspace_bytes, dev_status, s);
  }
  if (ig != nullptr && ig->dZ_prev != nullptr && (st->variant == RAD_DIFFERENT_SAMPLE || st->variant == RAD_SAME_SAMPLE) &&
      !input_grad_on_tc(st->dtype, st->B, st->D, H, dZ, ldz, ig->W, ig->ldw, ig->z_prev, ig->ld_zprev, ig->dZ_prev, ig->ldp))
    return simt_weight_grad(st, dZ, ldz, H, dW, ldw, dev_status, s, db, db_written, ig, ig_done);
  return simt_weight_grad(st, dZ, ldz, H, dW, ldw, dev_status, s, db, db_written);
}
}  // namespace
}  // namespace rad

extern "C" int rad_weight_grad_workspace(const rad_store* st, int64_t H, int64_t* bytes) {
  if (st == nullptr || bytes == nullptr || H <= 0 || st->B <= 0 || st->D <= 0) return RAD_EINVAL;
  if (st->variant == RAD_PROJECT) {
    if (st->values_ld <= 0) return RAD_EINVAL;
    *bytes = project_weight_grad_workspace(st, H);
    return RAD_OK;
  }
  if (st->variant == RAD_ROWS_SAMPLE) {
    if (draws_per_row_host(st->p, st->D) == 0) return RAD_EINVAL;
    const TileTwin t = tile_twin(st, nullptr);
    *bytes = t.bytes + round_up(tc_weight_grad_workspace(&t.st, H), 256);
    return RAD_OK;
  }
  if (st->variant == RAD_REDRAWN_SAMPLE) {
    const TileTwin t = redrawn_twin(st, nullptr);
    *bytes = t.bytes + round_up(tc_weight_grad_workspace(&t.st, H), 256);
    return RAD_OK;
  }
  *bytes = round_up(tc_weight_grad_workspace(st, H), 256);
  return RAD_OK;
}

extern "C" int rad_linear_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW,
                                      int64_t ldw, void* workspace, int64_t workspace_bytes,
                                      int32_t* dev_status, void* stream) {
  if (st != nullptr && st->variant == RAD_PROJECT) {
    if (st->B <= 0 || st->D <= 0 || !valid_dtype(st->dtype) || dZ == nullptr || dW == nullptr || H <= 0 || ldz < H ||
        ldw < H)
      return RAD_EINVAL;
    const int rcp = check_device();
    return rcp != RAD_OK ? rcp
                         : project_weight_grad(st, dZ, ldz, H, dW, ldw, workspace, workspace_bytes, dev_status, stream);
  }
  if (st != nullptr && st->variant == RAD_ROWS_SAMPLE) {
    // static-shape store: index part of the tile-major layout from the key alone, values moved into it, then
    // the same contraction as for a bitmask store
    if (st->B <= 0 || st->D <= 0 || !valid_dtype(st->dtype) || dZ == nullptr || dW == nullptr || H <= 0 || ldz < H || ldw < H ||
        !rows_store_ok(st))
      return RAD_EINVAL;
    int rcr = check_device();
    if (rcr != RAD_OK) return rcr;
    int64_t need = 0;
    rcr = rad_weight_grad_workspace(st, H, &need);
    if (rcr != RAD_OK) return rcr;
    if (workspace == nullptr || workspace_bytes < need || ((uintptr_t)workspace & 255) != 0) return RAD_EWORKSPACE;
    const TileTwin t = tile_twin(st, static_cast<char*>(workspace));
    cudaStream_t sr = static_cast<cudaStream_t>(stream);
    rcr = launch_fixed_index(&t.st, true, dev_status, sr);
    if (rcr != RAD_OK) return rcr;
    rcr = rows_to_tiles(st, &t.st, dev_status, sr);
    if (rcr != RAD_OK) return rcr;
    return rad_linear_weight_grad(&t.st, dZ, ldz, H, dW, ldw, static_cast<char*>(workspace) + t.bytes, workspace_bytes - t.bytes,
                                  dev_status, stream);
  }
  return weight_grad_and_bias(st, dZ, ldz, H, dW, ldw, workspace, workspace_bytes, dev_status, stream, nullptr, nullptr);
}

extern "C" int rad_linear_forward(int32_t dtype, int32_t act, int64_t B, int64_t D, int64_t H, const void* A,
                                  int64_t lda, const void* W, int64_t ldw, const float* bias, void* out_act,
                                  int64_t ld_act, float* out_z, int64_t ld_z, void* out_zlow, int64_t ld_zlow,
                                  uint32_t* relubits, int32_t* dev_status, void* stream) {
  if (!valid_dtype(dtype) || B <= 0 || D <= 0 || H <= 0 || A == nullptr || W == nullptr) return RAD_EINVAL;
  if (act != RAD_ACT_NONE && act != RAD_ACT_RELU && act != RAD_ACT_GELU) return RAD_EINVAL;
  if (lda < D || ldw < H) return RAD_EINVAL;
  if (out_act == nullptr && out_z == nullptr && out_zlow == nullptr) return RAD_EINVAL;
  if ((out_act != nullptr && ld_act < H) || (out_z != nullptr && ld_z < H) || (out_zlow != nullptr && ld_zlow < H))
    return RAD_EINVAL;
  if (relubits != nullptr && out_act == nullptr) return RAD_EINVAL;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dtype == RAD_BF16 && tc_shape_ok(B, D, H, A, lda, W, ldw) && ((uintptr_t)bias & 15) == 0 &&
      (out_act == nullptr || (((uintptr_t)out_act & 15) == 0 && ld_act % 8 == 0)) &&
      (out_zlow == nullptr || (((uintptr_t)out_zlow & 15) == 0 && ld_zlow % 8 == 0)) &&
      (out_z == nullptr || (((uintptr_t)out_z & 15) == 0 && ld_z % 4 == 0)))
    return tc_forward(act, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, out_z, ld_z, out_zlow, ld_zlow,
                      relubits, dev_status, s);
  return simt_forward(dtype, act, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, out_z, ld_z, out_zlow,
                      ld_zlow, relubits, s);
}

namespace rad {
namespace {
// Whether the forward GEMM can fill `next` from its epilogue: tensor-core shapes, a different-sample store under a
// law whose index can be made from the key alone.
bool fill_can_fuse(int dtype, int64_t B, int64_t D, int64_t H, const void* A, int64_t lda, const void* W, int64_t ldw,
                   const float* bias, const void* out_act, int64_t ld_act, const void* out_zlow, int64_t ld_zlow,
                   const rad_store* next) {
  return dtype == RAD_BF16 && next->variant == RAD_DIFFERENT_SAMPLE &&
         (next->law == RAD_LAW_BERNOULLI || (next->law == RAD_LAW_FIXED && H <= 65536)) && store_args_ok(next) &&
         tc_shape_ok(B, D, H, A, lda, W, ldw) && ((uintptr_t)bias & 15) == 0 && ((uintptr_t)out_act & 15) == 0 &&
         ld_act % 8 == 0 && ((uintptr_t)next->keepbits & 15) == 0 &&
         (out_zlow == nullptr || (((uintptr_t)out_zlow & 15) == 0 && ld_zlow % 8 == 0)) &&
         (double)B * (double)H < 4294967296.0 * 0.75;
}

}  // namespace
}  // namespace rad

extern "C" int rad_linear_forward_fill(int32_t dtype, int32_t act, int64_t B, int64_t D, int64_t H, const void* A,
                                       int64_t lda, const void* W, int64_t ldw, const float* bias, void* out_act,
                                       int64_t ld_act, void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
                                       const rad_store* next, int32_t index_ready, void* workspace,
                                       int64_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!valid_dtype(dtype) || B <= 0 || D <= 0 || H <= 0 || A == nullptr || W == nullptr || out_act == nullptr)
    return RAD_EINVAL;
  if (act != RAD_ACT_NONE && act != RAD_ACT_RELU && act != RAD_ACT_GELU) return RAD_EINVAL;
  if (lda < D || ldw < H || ld_act < H || (out_zlow != nullptr && ld_zlow < H)) return RAD_EINVAL;
  if (next == nullptr || next->B != B || next->D != H || next->dtype != dtype) return RAD_EINVAL;
  if (next->variant == RAD_REDRAWN_SAMPLE) {
    // the index part goes to the head of the workspace, then as for a different-sample store
    if (!redrawn_args_ok(next) || index_ready) return RAD_EINVAL;
    const int64_t head = redrawn_index_bytes(B, H);
    if (workspace == nullptr || workspace_bytes < head) return RAD_EWORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return RAD_EINVAL;
    rad_store full = *next;
    full.variant = RAD_DIFFERENT_SAMPLE;
    full.keepbits = static_cast<uint32_t*>(workspace);
    return rad_linear_forward_fill(dtype, act, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, out_zlow, ld_zlow, relubits,
                                   &full, 0, static_cast<char*>(workspace) + head, workspace_bytes - head, dev_status, stream);
  }
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  bool fused = fill_can_fuse(dtype, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, out_zlow, ld_zlow, next);
  if (fused && !index_ready) {
    rc = launch_store_index(next, true, dev_status, s);
    if (rc == RAD_EUNSUPPORTED) fused = false;        // rows too long for the fixed-count index: the separate calls below
    else if (rc != RAD_OK) return rc;
  }
  if (fused)
    return tc_forward(act, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, nullptr, 0, out_zlow, ld_zlow, relubits,
                      dev_status, s, next);
  // shapes the fused epilogue does not take: the same results from the two separate calls
  // Where the forward runs on the CUDA cores its ReLU bits would be one more launch: there they come from the
  // store kernels, which look at every entry anyway (not from the projection store, which does not).
  const bool bits_from_store = next->variant != RAD_PROJECT && !(dtype == RAD_BF16 && tc_shape_ok(B, D, H, A, lda, W, ldw));
  rc = rad_linear_forward(dtype, act, B, D, H, A, lda, W, ldw, bias, out_act, ld_act, nullptr, 0, out_zlow, ld_zlow,
                          bits_from_store ? nullptr : relubits, dev_status, stream);
  if (rc != RAD_OK) return rc;
  rad_store tmp = *next;
  tmp.relubits = bits_from_store ? relubits : nullptr;
  return rad_linear_forward_store(out_act, ld_act, &tmp, workspace, workspace_bytes, dev_status, stream);
}

extern "C" int rad_input_grad_workspace(int64_t B, int64_t H, int64_t* bytes) {
  if (bytes == nullptr || B <= 0 || H <= 0) return RAD_EINVAL;
  *bytes = column_sums_workspace(B, H);
  return RAD_OK;
}

extern "C" int rad_linear_input_grad(int32_t dtype, int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz,
                                     const void* W, int64_t ldw, const uint32_t* relubits_prev,
                                     const void* z_prev, int64_t ld_zprev, void* dZ_prev, int64_t ldp,
                                     float* db, void* workspace, int64_t workspace_bytes,
                                     int32_t* dev_status, void* stream) {
  if (!valid_dtype(dtype) || B <= 0 || D <= 0 || H <= 0 || dZ == nullptr || W == nullptr) return RAD_EINVAL;
  if (ldz < H || ldw < H) return RAD_EINVAL;
  if (dZ_prev == nullptr && db == nullptr) return RAD_EINVAL;
  if (dZ_prev != nullptr && ldp < D) return RAD_EINVAL;
  if (z_prev != nullptr && ld_zprev < D) return RAD_EINVAL;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (db != nullptr) {
    rc = column_sums(dtype, B, H, dZ, ldz, db, workspace, workspace_bytes, s);
    if (rc != RAD_OK) return rc;
  }
  if (dZ_prev == nullptr) return RAD_OK;
  if (input_grad_on_tc(dtype, B, D, H, dZ, ldz, W, ldw, z_prev, ld_zprev, dZ_prev, ldp))
    return tc_input_grad(B, D, H, dZ, ldz, W, ldw, relubits_prev, z_prev, ld_zprev, dZ_prev, ldp, dev_status, s);
  return simt_input_grad(dtype, B, D, H, dZ, ldz, W, ldw, relubits_prev, z_prev, ld_zprev, dZ_prev, ldp, s);
}

extern "C" int rad_mlp_workspace(const rad_mlp_desc* net, int64_t* bytes, rad_step_stats* stats) {
  if (bytes == nullptr) return RAD_EINVAL;
  StepPlan plan;
  int rc = make_plan(net, &plan);
  if (rc != RAD_OK) return rc;
  *bytes = plan.total;
  if (stats != nullptr) *stats = plan.stats;
  return RAD_OK;
}

extern "C" int rad_mlp_held_bytes(const rad_mlp_desc* net, const int64_t* nnz, rad_step_stats* stats) {
  if (nnz == nullptr || stats == nullptr) return RAD_EINVAL;
  StepPlan plan;
  const int rc = make_plan(net, &plan);
  if (rc != RAD_OK) return rc;
  *stats = plan.stats;
  // values as kept by the step that produced `nnz` (padding of the tile-major layout included), not as reserved
  int64_t held = 0;
  for (int l = 0; l < net->L; ++l) {
    if (nnz[2 * l] < 0 || nnz[2 * l + 1] < nnz[2 * l]) return RAD_EINVAL;
    const int64_t elems = (net->variant == RAD_DIFFERENT_SAMPLE || net->variant == RAD_REDRAWN_SAMPLE) ? nnz[2 * l + 1]
                        : net->variant == RAD_SAME_SAMPLE      ? net->B * nnz[2 * l]
                                                               : net->B * plan.layer[l].values_ld;
    held += elems * esize(net->dtype);
  }
  stats->value_bytes = held;
  return RAD_OK;
}

extern "C" int rad_mlp_step(const rad_mlp_desc* net, const void* X, const int32_t* labels, const void* const* W,
                            const float* const* b, float* const* dW, float* const* db, float* loss,
                            int64_t* nnz_out, void* workspace, int64_t workspace_bytes, int32_t* dev_status,
                            void* stream) {
  StepPlan plan;
  int rc = make_plan(net, &plan);
  if (rc != RAD_OK) return rc;
  if (X == nullptr || labels == nullptr || W == nullptr || dW == nullptr || db == nullptr || loss == nullptr)
    return RAD_EINVAL;
  if (workspace == nullptr || workspace_bytes < plan.total) return RAD_EWORKSPACE;
  if (((uintptr_t)workspace & 255) != 0) return RAD_EINVAL;
  rc = check_device();
  if (rc != RAD_OK) return rc;
  char* ws = static_cast<char*>(workspace);
  const int L = net->L;
  const int64_t B = net->B;
  rad_store st[64] = {};
  for (int l = 0; l < L; ++l) {
    if (W[l] == nullptr || dW[l] == nullptr || db[l] == nullptr) return RAD_EINVAL;
    const LayerPlan& lp = plan.layer[l];
    rad_store& s = st[l];
    s.variant = net->variant; s.dtype = net->dtype; s.B = B; s.D = net->dims[l]; s.p = net->p;
    s.layer = (uint32_t)l; s.step = net->step; s.seed = net->seed; s.law = net->law;
    s.values = ws + lp.values; s.values_capacity = lp.capacity; s.values_ld = lp.values_ld;
    s.keepbits = net->variant == RAD_REDRAWN_SAMPLE ? nullptr : reinterpret_cast<uint32_t*>(ws + lp.keepbits);
    s.offsets = reinterpret_cast<uint32_t*>(ws + lp.offsets);
    s.nnz = nnz_out != nullptr ? nnz_out + 2 * l : reinterpret_cast<int64_t*>(ws + lp.nnz);
    // the ReLU bits of a hidden layer's input are written by the epilogue of the layer that produces it
    s.relubits = nullptr;
  }
  // the network input is stored by the stand-alone kernel; every hidden layer's input is stored from the
  // epilogue of the GEMM that produces it (or by the same stand-alone call where that kernel does not apply)
  TraceRange step_range("rad_mlp_step");
  {
    TraceRange r("store input");
    rc = rad_linear_forward_store(X, net->dims[0], &st[0], ws + plan.scratch, plan.scratch_bytes, dev_status, stream);
  }
  if (rc != RAD_OK) return rc;
  const void* a_in = X;
  int64_t ld_in = net->dims[0];
  for (int l = 0; l < L; ++l) {
    TraceRange r("forward layer");
    const int64_t D = net->dims[l], H = net->dims[l + 1];
    const bool last = (l == L - 1);
    if (last) {
      rc = rad_linear_forward(net->dtype, RAD_ACT_NONE, B, D, H, a_in, ld_in, W[l], H, b != nullptr ? b[l] : nullptr,
                              nullptr, H, reinterpret_cast<float*>(ws + plan.logits), H, nullptr, H, nullptr,
                              dev_status, stream);
      if (rc != RAD_OK) return rc;
      break;
    }
    void* a_out = ws + plan.act[l & 1];
    // a GELU net keeps the pre-activation of layer l for the backward of layer l + 1's input
    void* zlow = net->act == RAD_ACT_GELU ? ws + plan.layer[l + 1].preact : nullptr;
    uint32_t* rbits = plan.layer[l + 1].relubits >= 0 ? reinterpret_cast<uint32_t*>(ws + plan.layer[l + 1].relubits) : nullptr;
    rc = rad_linear_forward_fill(net->dtype, net->act, B, D, H, a_in, ld_in, W[l], H, b != nullptr ? b[l] : nullptr,
                                 a_out, H, zlow, H, rbits, &st[l + 1], 0, ws + plan.scratch,
                                 plan.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    a_in = a_out;
    ld_in = H;
  }
  for (int l = 1; l < L; ++l)
    st[l].relubits = plan.layer[l].relubits >= 0 ? reinterpret_cast<uint32_t*>(ws + plan.layer[l].relubits) : nullptr;
  const int64_t C = net->dims[L];
  void* dz = ws + plan.dz[(L - 1) & 1];
  rc = rad_softmax_xent(net->dtype, B, C, reinterpret_cast<const float*>(ws + plan.logits), C, labels, loss, dz,
                        C, ws + plan.scratch, plan.scratch_bytes, stream);
  if (rc != RAD_OK) return rc;
  for (int l = L - 1; l >= 0; --l) {
    TraceRange r("backward layer");
    const int64_t D = net->dims[l], H = net->dims[l + 1];
    bool db_done = false, dx_done = false;
    void* dz_prev = l > 0 ? ws + plan.dz[(l - 1) & 1] : nullptr;
    const void* z_prev = plan.layer[l].preact >= 0 ? ws + plan.layer[l].preact : nullptr;
    const SimtInputGrad ig = {W[l], H, st[l].relubits, z_prev, D, dz_prev, D};
    if (net->variant == RAD_DIFFERENT_SAMPLE || net->variant == RAD_SAME_SAMPLE || net->variant == RAD_REDRAWN_SAMPLE)
      rc = weight_grad_and_bias(&st[l], dz, H, H, dW[l], H, ws + plan.scratch, plan.scratch_bytes, dev_status, stream, db[l],
                                &db_done, dz_prev != nullptr ? &ig : nullptr, &dx_done);
    else
      rc = rad_linear_weight_grad(&st[l], dz, H, H, dW[l], H, ws + plan.scratch, plan.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    if ((dz_prev != nullptr && !dx_done) || !db_done) {
      rc = rad_linear_input_grad(net->dtype, B, D, H, dz, H, W[l], H, st[l].relubits, z_prev, D,
                                 dx_done ? nullptr : dz_prev, D, db_done ? nullptr : db[l], ws + plan.scratch,
                                 plan.scratch_bytes, dev_status, stream);
      if (rc != RAD_OK) return rc;
    }
    dz = dz_prev;
  }
  return RAD_OK;
}
