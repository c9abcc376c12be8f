// One training step of a small convolutional net (3x3 conv + ReLU + 2x2 average pool blocks, then
// linear layers) with activation sampling on the input of every conv and linear layer
// (paper, Fig. "Convnet activation sampling"; Sec. 4.2).  Host-side sequencing only: every step
// of the path is a kernel of this library.
#include <algorithm>

#include "common.cuh"

namespace rad {
namespace {

constexpr int kMaxLayers = 16;

struct CnnPlan {
  int nc, nf;
  int H[kMaxLayers], W[kMaxLayers], Cin[kMaxLayers], Cout[kMaxLayers];     // conv layer l: input H x W x Cin
  int64_t fdim[kMaxLayers + 1];                                             // linear dims
  // byte offsets into the workspace
  int64_t values[2 * kMaxLayers], keepbits[2 * kMaxLayers], offsets[2 * kMaxLayers], nnz[2 * kMaxLayers];
  int64_t capacity[2 * kMaxLayers], values_ld[2 * kMaxLayers];
  int64_t relubits[2 * kMaxLayers];
  int64_t act[2], grad[2], dz, logits, scratch, scratch_bytes, total;
  rad_step_stats stats;
};

int64_t esize(int dtype) { return dtype == RAD_BF16 ? 2 : 4; }

int make_cnn_plan(const rad_cnn_desc* d, CnnPlan* pl) {
  if (d == nullptr || d->B <= 0 || d->n_conv < 1 || d->n_conv > kMaxLayers || d->n_fc < 1 || d->n_fc > kMaxLayers)
    return RAD_EINVAL;
  if (d->conv_channels == nullptr || d->fc_dims == nullptr || d->H <= 0 || d->W <= 0 || d->Cin <= 0) return RAD_EINVAL;
  if (d->dtype != RAD_F32 && d->dtype != RAD_BF16) return RAD_EINVAL;
  if (d->variant != RAD_DIFFERENT_SAMPLE && d->variant != RAD_SAME_SAMPLE) return RAD_EINVAL;
  if (keep_threshold_host(d->p) == 0) return RAD_EINVAL;
  const int64_t B = d->B, es = esize(d->dtype);
  pl->nc = d->n_conv; pl->nf = d->n_fc;
  int h = (int)d->H, w = (int)d->W, c = (int)d->Cin;
  int64_t off = 0, max_act = 0, max_conv_out = 0, scratch = B * 4;
  auto take = [&](int64_t bytes) { const int64_t at = off; off += round_up(bytes, 256); return at; };
  rad_step_stats st = {};
  auto plan_store = [&](int idx, int64_t D) -> int {
    rad_store_sizes sz;
    int rc = rad_store_size_query(d->variant, d->dtype, B, D, d->p, &sz);
    if (rc != RAD_OK) return rc;
    pl->capacity[idx] = sz.values_typical; pl->values_ld[idx] = sz.values_ld_typical;
    pl->values[idx] = take(sz.values_typical * es);
    pl->keepbits[idx] = take(sz.keepbits_words * 4);
    pl->offsets[idx] = take(sz.offsets_words * 4);
    pl->nnz[idx] = take(16);
    st.value_bytes += sz.values_typical * es;
    st.index_bytes += (sz.keepbits_words + sz.offsets_words) * 4;
    st.full_backprop_bytes += B * D * es;
    scratch = std::max(scratch, sz.workspace_bytes);
    return RAD_OK;
  };
  for (int l = 0; l < pl->nc; ++l) {
    const int co = (int)d->conv_channels[l];
    if (co <= 0 || co % 8 != 0 || h % 2 != 0 || w % 2 != 0) return RAD_EUNSUPPORTED;
    pl->H[l] = h; pl->W[l] = w; pl->Cin[l] = c; pl->Cout[l] = co;
    int rc = plan_store(l, (int64_t)h * w * c);
    if (rc != RAD_OK) return rc;
    pl->relubits[l] = take(B * h * w * co / 8);                       // one bit per conv output
    st.relu_bytes += B * h * w * co / 8;
    max_conv_out = std::max<int64_t>(max_conv_out, (int64_t)h * w * co);
    max_act = std::max<int64_t>(max_act, (int64_t)h * w * c);
    scratch = std::max(scratch, conv_weight_grad_workspace(B, c, co));
    scratch = std::max(scratch, conv_tc_weight_grad_workspace(B, h, w, c, co));
    scratch = std::max(scratch, column_sums_workspace(B * h * w, co));
    h /= 2; w /= 2; c = co;
    max_act = std::max<int64_t>(max_act, (int64_t)h * w * c);
  }
  pl->fdim[0] = (int64_t)h * w * c;
  for (int l = 0; l < pl->nf; ++l) {
    pl->fdim[l + 1] = d->fc_dims[l];
    if (pl->fdim[l + 1] <= 0) return RAD_EINVAL;
    int rc = plan_store(pl->nc + l, pl->fdim[l]);
    if (rc != RAD_OK) return rc;
    pl->relubits[pl->nc + l] = -1;
    if (l > 0) {                                                       // input of linear layer l is a ReLU output
      pl->relubits[pl->nc + l] = take(B * ceil_div(pl->fdim[l], 32) * 4);
      st.relu_bytes += B * ceil_div(pl->fdim[l], 32) * 4;
    }
    max_act = std::max(max_act, pl->fdim[l + 1]);
    scratch = std::max(scratch, column_sums_workspace(B, pl->fdim[l + 1]));
    rad_store tmp = {};
    tmp.variant = d->variant; tmp.dtype = d->dtype; tmp.B = B; tmp.D = pl->fdim[l]; tmp.p = d->p;
    tmp.values_ld = pl->values_ld[pl->nc + l]; tmp.values_capacity = pl->capacity[pl->nc + l];
    scratch = std::max(scratch, tc_weight_grad_workspace(&tmp, pl->fdim[l + 1]));
  }
  st.unsampled_bytes = B * pl->fdim[pl->nf] * 4;
  st.full_backprop_bytes += st.unsampled_bytes;
  pl->act[0] = take(B * max_act * es);
  pl->act[1] = take(B * max_act * es);
  pl->grad[0] = take(B * max_act * es);
  pl->grad[1] = take(B * max_act * es);
  pl->dz = take(B * max_conv_out * es);
  pl->logits = take(B * pl->fdim[pl->nf] * 4);
  pl->scratch_bytes = round_up(scratch, 256);
  pl->scratch = take(pl->scratch_bytes);
  pl->total = off;
  pl->stats = st;
  return RAD_OK;
}

}  // namespace
}  // namespace rad

using namespace rad;

extern "C" int rad_cnn_workspace(const rad_cnn_desc* d, int64_t* bytes, rad_step_stats* stats) {
  if (bytes == nullptr) return RAD_EINVAL;
  CnnPlan pl;
  int rc = make_cnn_plan(d, &pl);
  if (rc != RAD_OK) return rc;
  *bytes = pl.total;
  if (stats != nullptr) *stats = pl.stats;
  return RAD_OK;
}

extern "C" int rad_cnn_step(const rad_cnn_desc* d, const void* X, const int32_t* labels, const void* const* conv_W,
                            const float* const* conv_b, const void* const* fc_W, const float* const* fc_b,
                            float* const* dconv_W, float* const* dconv_b, float* const* dfc_W, float* const* dfc_b,
                            float* loss, int64_t* nnz_out, void* workspace, int64_t workspace_bytes,
                            int32_t* dev_status, void* stream) {
  CnnPlan pl;
  int rc = make_cnn_plan(d, &pl);
  if (rc != RAD_OK) return rc;
  if (X == nullptr || labels == nullptr || conv_W == nullptr || fc_W == nullptr || dconv_W == nullptr ||
      dconv_b == nullptr || dfc_W == nullptr || dfc_b == nullptr || loss == nullptr)
    return RAD_EINVAL;
  if (workspace == nullptr || workspace_bytes < pl.total) return RAD_EWORKSPACE;
  if (((uintptr_t)workspace & 255) != 0) return RAD_EINVAL;
  rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  const int64_t B = d->B;
  const int nl = pl.nc + pl.nf;
  rad_store st[2 * kMaxLayers] = {};
  auto make_store = [&](int idx, int64_t D) {
    rad_store& q = st[idx];
    q.variant = d->variant; q.dtype = d->dtype; q.B = B; q.D = D; q.p = d->p;
    q.layer = (uint32_t)idx; q.step = d->step; q.seed = d->seed;
    q.values = ws + pl.values[idx]; q.values_capacity = pl.capacity[idx]; q.values_ld = pl.values_ld[idx];
    q.keepbits = reinterpret_cast<uint32_t*>(ws + pl.keepbits[idx]);
    q.offsets = reinterpret_cast<uint32_t*>(ws + pl.offsets[idx]);
    q.nnz = nnz_out != nullptr ? nnz_out + 2 * idx : reinterpret_cast<int64_t*>(ws + pl.nnz[idx]);
    q.relubits = nullptr;
  };
  // ---- forward ----
  const void* a_in = X;
  for (int l = 0; l < pl.nc; ++l) {
    if (conv_W[l] == nullptr || dconv_W[l] == nullptr || dconv_b[l] == nullptr) return RAD_EINVAL;
    make_store(l, (int64_t)pl.H[l] * pl.W[l] * pl.Cin[l]);
    rc = rad_linear_forward_store(a_in, st[l].D, &st[l], ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    void* a_out = ws + pl.act[l & 1];
    // tensor cores where the shape allows (Cin 16 / 32 / 64: the later convolutions), CUDA cores otherwise
    if (conv_tc_ok(d->dtype, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], a_in, conv_W[l]))
      rc = conv_tc_forward_pool(B, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], a_in, conv_W[l],
                                conv_b != nullptr ? conv_b[l] : nullptr, a_out, reinterpret_cast<uint32_t*>(ws + pl.relubits[l]),
                                dev_status, s);
    else
      rc = conv_forward_pool(d->dtype, B, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], a_in, conv_W[l],
                             conv_b != nullptr ? conv_b[l] : nullptr, a_out, reinterpret_cast<uint32_t*>(ws + pl.relubits[l]), s);
    if (rc != RAD_OK) return rc;
    a_in = a_out;
  }
  for (int l = 0; l < pl.nf; ++l) {
    const int idx = pl.nc + l;
    if (fc_W[l] == nullptr || dfc_W[l] == nullptr || dfc_b[l] == nullptr) return RAD_EINVAL;
    const int64_t D = pl.fdim[l], H = pl.fdim[l + 1];
    make_store(idx, D);
    rc = rad_linear_forward_store(a_in, D, &st[idx], ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    const bool last = l == pl.nf - 1;
    void* a_out = last ? nullptr : ws + pl.act[idx & 1];
    rc = rad_linear_forward(d->dtype, last ? RAD_ACT_NONE : RAD_ACT_RELU, B, D, H, a_in, D, fc_W[l], H,
                            fc_b != nullptr ? fc_b[l] : nullptr, a_out, H,
                            last ? reinterpret_cast<float*>(ws + pl.logits) : nullptr, H, nullptr, 0,
                            last ? nullptr : reinterpret_cast<uint32_t*>(ws + pl.relubits[idx + 1]), dev_status, stream);
    if (rc != RAD_OK) return rc;
    a_in = a_out;
  }
  // ---- loss ----
  const int64_t C = pl.fdim[pl.nf];
  void* g = ws + pl.grad[(nl - 1) & 1];
  rc = rad_softmax_xent(d->dtype, B, C, reinterpret_cast<const float*>(ws + pl.logits), C, labels, loss, g, C,
                        ws + pl.scratch, pl.scratch_bytes, stream);
  if (rc != RAD_OK) return rc;
  // ---- backward: linear layers ----
  for (int l = pl.nf - 1; l >= 0; --l) {
    const int idx = pl.nc + l;
    const int64_t D = pl.fdim[l], H = pl.fdim[l + 1];
    rc = rad_linear_weight_grad(&st[idx], g, H, H, dfc_W[l], H, ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    void* g_prev = ws + pl.grad[(idx - 1) & 1];
    // the first linear layer reads the pooled map, which is not a ReLU output: no mask there
    rc = rad_linear_input_grad(d->dtype, B, D, H, g, H, fc_W[l], H,
                               l > 0 ? reinterpret_cast<const uint32_t*>(ws + pl.relubits[idx]) : nullptr, nullptr, 0,
                               g_prev, D, dfc_b[l], ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
    if (rc != RAD_OK) return rc;
    g = g_prev;
  }
  // ---- backward: conv blocks (g = gradient of the pooled output of block l) ----
  void* dz = ws + pl.dz;
  for (int l = pl.nc - 1; l >= 0; --l) {
    rc = conv_dz(d->dtype, B, pl.H[l], pl.W[l], pl.Cout[l], g, reinterpret_cast<const uint32_t*>(ws + pl.relubits[l]), dz, s);
    if (rc != RAD_OK) return rc;
    if (conv_tc_ok(d->dtype, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, conv_W[l]))
      rc = conv_tc_weight_grad(&st[l], pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, dconv_W[l], ws + pl.scratch,
                               pl.scratch_bytes, dev_status, s);
    else
      rc = conv_weight_grad(&st[l], pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, dconv_W[l], ws + pl.scratch,
                            pl.scratch_bytes, s);
    if (rc != RAD_OK) return rc;
    rc = column_sums(d->dtype, B * pl.H[l] * pl.W[l], pl.Cout[l], dz, pl.Cout[l], dconv_b[l], ws + pl.scratch,
                     pl.scratch_bytes, s);
    if (rc != RAD_OK) return rc;
    if (l > 0) {
      void* g_prev = ws + pl.grad[(l - 1) & 1];
      if (conv_tc_dx_ok(d->dtype, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, conv_W[l], g_prev))
        rc = conv_tc_input_grad(B, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, conv_W[l], g_prev, dev_status, s);
      else
        rc = conv_input_grad(d->dtype, B, pl.H[l], pl.W[l], pl.Cin[l], pl.Cout[l], dz, conv_W[l], g_prev, s);
      if (rc != RAD_OK) return rc;
      g = g_prev;
    }
  }
  return RAD_OK;
}
