// Random-projection variant (Sec. 3.2 after Eq. 5; App. A "Random Projections for RAD"): P = R R^T with
// R a D x k matrix of independent Rademacher signs scaled by 1 / sqrt(k), k = ceil(fraction D).
// Forward: the store is S = A R' (B x k, R' the unscaled signs), one dense GEMM.  Backward:
// dW_hat = R' ((S^T dZ) / k), two dense GEMMs.  All three run on the library's GEMM entry points (tcgen05
// for bf16 shapes TMA can take, CUDA cores otherwise); R' is never kept between the passes: it is a
// function of (seed, layer, step) and is drawn again from Philox where it is needed.
#include <algorithm>

#include "common.cuh"

namespace rad {
namespace {

constexpr uint32_t kProjectStream = 6;

struct SignParams {
  void* out;            // D x ld, row-major
  int64_t D, k, ld;
  uint32_t c2, c3;
};

// One thread per (row d, 32 columns): entry (d, j) reads bit j % 32 of word (j % 128) / 32 of the Philox
// output for counter (j / 128, d, c2, c3); set means -1.  Columns k .. ld-1 are zero.
template <typename T>
__global__ void __launch_bounds__(256) rademacher_kernel(const SignParams p, const PhiloxKeys ks) {
  const int64_t groups = p.ld / 32 + (p.ld % 32 != 0 ? 1 : 0);
  const int64_t n = p.D * groups;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t d = i / groups, g = i % groups;
    uint32_t w[4];
    philox4x32_10((uint32_t)(g >> 2), (uint32_t)d, p.c2, p.c3, ks, w);
    const uint32_t bits = (g & 3) == 0 ? w[0] : (g & 3) == 1 ? w[1] : (g & 3) == 2 ? w[2] : w[3];
    T* out = static_cast<T*>(p.out) + d * p.ld + g * 32;
#pragma unroll 8
    for (int j = 0; j < 32; ++j) {
      const int64_t col = g * 32 + j;
      if (col < p.ld) out[j] = from_float<T>(col < p.k ? (((bits >> j) & 1u) ? -1.0f : 1.0f) : 0.0f);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) scale_convert_kernel(const float* in, T* out, int64_t n, float scale) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    out[i] = from_float<T>(__fmul_rn(in[i], scale));
}

// idx: the identity list of ld columns; bits: bit j set for j < k (the columns of S that hold data)
__global__ void project_meta_kernel(uint32_t* idx, uint32_t* bits, int64_t ld, int64_t* nnz, int64_t k, int64_t B) {
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < ld; j += (int64_t)gridDim.x * blockDim.x) {
    if (idx != nullptr) idx[j] = (uint32_t)j;
    if (bits != nullptr && (j & 31) == 0) {
      const int64_t nv = k - j;
      bits[j >> 5] = nv >= 32 ? 0xffffffffu : nv <= 0 ? 0u : (1u << nv) - 1u;
    }
  }
  if (nnz != nullptr && blockIdx.x == 0 && threadIdx.x == 0) { nnz[0] = k; nnz[1] = k * B; }
}

int64_t esz(int dtype) { return dtype == RAD_BF16 ? 2 : 4; }

int draw_signs(int dtype, void* out, int64_t D, int64_t k, int64_t ld, uint64_t seed, uint32_t layer, uint32_t step,
               cudaStream_t s) {
  SignParams p;
  p.out = out; p.D = D; p.k = k; p.ld = ld;
  p.c2 = (layer & 0xffffffu) | (kProjectStream << 24); p.c3 = step;
  const PhiloxKeys ks = philox_expand_key(seed);
  const int64_t n = D * ceil_div(ld, 32);
  const int grid = (int)std::min<int64_t>(ceil_div(n, 256), 148 * 16);
  count_launch();
  if (dtype == RAD_BF16)
    rademacher_kernel<bf16><<<grid, 256, 0, s>>>(p, ks);
  else
    rademacher_kernel<float><<<grid, 256, 0, s>>>(p, ks);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// the stand-in the same-sample weight-gradient path takes: a B x ld block with all of its columns kept
rad_store as_dense_block(const rad_store* st, uint32_t* idx, uint32_t* bits) {
  rad_store t = {};
  t.variant = RAD_SAME_SAMPLE; t.dtype = st->dtype; t.B = st->B; t.D = st->values_ld; t.p = 1.0f;
  t.values = st->values; t.values_capacity = st->values_capacity; t.values_ld = st->values_ld;
  t.keepbits = bits; t.offsets = idx; t.nnz = st->nnz;
  return t;
}

}  // namespace

int64_t project_ld(int64_t k) { return round_up(k, 64); }

bool project_store_ok(const rad_store* st) {
  const int64_t k = draws_per_row_host(st->p, st->D);
  return k > 0 && st->values != nullptr && st->nnz != nullptr && st->values_ld >= k && st->values_ld % 8 == 0 &&
         st->values_capacity >= st->B * st->values_ld;
}

int64_t project_store_workspace(int dtype, int64_t D, int64_t ld) { return round_up(D * ld * esz(dtype), 256); }

int64_t project_weight_grad_workspace(const rad_store* st, int64_t H) {
  const int64_t ld = st->values_ld, es = esz(st->dtype);
  rad_store t = as_dense_block(st, nullptr, nullptr);
  return round_up(st->D * ld * es, 256) + round_up(ld * 4, 256) + round_up(ceil_div(ld, 32) * 4, 256) + round_up(ld * H * 4, 256) + round_up(ld * H * es, 256) +
         round_up(tc_weight_grad_workspace(&t, H), 256);
}

int project_forward_store(const void* A, int64_t lda, const rad_store* st, void* workspace, int64_t workspace_bytes,
                          int32_t* dev_status, void* stream) {
  if (!project_store_ok(st)) return RAD_EINVAL;
  const int64_t k = draws_per_row_host(st->p, st->D), ld = st->values_ld;
  if (workspace == nullptr || workspace_bytes < project_store_workspace(st->dtype, st->D, ld)) return RAD_EWORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int rc = draw_signs(st->dtype, workspace, st->D, k, ld, st->seed, st->layer, st->step, s);
  if (rc != RAD_OK) return rc;
  count_launch();
  project_meta_kernel<<<1, 32, 0, s>>>(nullptr, nullptr, 0, st->nnz, k, st->B);
  // S = A R': B x D times D x ld, stored in the working type
  rc = rad_linear_forward(st->dtype, RAD_ACT_NONE, st->B, st->D, ld, A, lda, workspace, ld, nullptr, st->values, ld,
                          nullptr, 0, nullptr, 0, nullptr, dev_status, stream);
  if (rc != RAD_OK) return rc;
  if (st->relubits != nullptr) return launch_relu_bits(st->dtype, A, lda, st->B, st->D, st->relubits, s);
  return RAD_OK;
}

int project_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW, int64_t ldw,
                        void* workspace, int64_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (!project_store_ok(st)) return RAD_EINVAL;
  if (workspace == nullptr || workspace_bytes < project_weight_grad_workspace(st, H)) return RAD_EWORKSPACE;
  const int64_t k = draws_per_row_host(st->p, st->D), ld = st->values_ld, es = esz(st->dtype);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  void* R = ws;                                   ws += round_up(st->D * ld * es, 256);
  uint32_t* idx = reinterpret_cast<uint32_t*>(ws);  ws += round_up(ld * 4, 256);
  uint32_t* bits = reinterpret_cast<uint32_t*>(ws); ws += round_up(ceil_div(ld, 32) * 4, 256);
  float* G32 = reinterpret_cast<float*>(ws);      ws += round_up(ld * H * 4, 256);
  void* G = ws;                                   ws += round_up(ld * H * es, 256);
  const int64_t inner = workspace_bytes - (ws - static_cast<char*>(workspace));
  int rc = draw_signs(st->dtype, R, st->D, k, ld, st->seed, st->layer, st->step, s);
  if (rc != RAD_OK) return rc;
  count_launch();
  project_meta_kernel<<<(unsigned)std::min<int64_t>(ceil_div(ld, 256), 1024), 256, 0, s>>>(idx, bits, ld, nullptr, k, 0);
  // G32 = S^T dZ (ld x H): the dense block of S goes through the same-sample contraction with every column kept
  const rad_store t = as_dense_block(st, idx, bits);
  rc = rad_linear_weight_grad(&t, dZ, ldz, H, G32, H, ws, inner, dev_status, stream);
  if (rc != RAD_OK) return rc;
  // G = (S^T dZ) / k in the working type
  const int64_t n = ld * H;
  const int grid = (int)std::min<int64_t>(ceil_div(n, 256), 148 * 16);
  count_launch();
  if (st->dtype == RAD_BF16)
    scale_convert_kernel<bf16><<<grid, 256, 0, s>>>(G32, static_cast<bf16*>(G), n, 1.0f / (float)k);
  else
    scale_convert_kernel<float><<<grid, 256, 0, s>>>(G32, static_cast<float*>(G), n, 1.0f / (float)k);
  if (cudaGetLastError() != cudaSuccess) return RAD_ECUDA;
  // dW_hat = R' G: D x ld times ld x H, float32 out
  return rad_linear_forward(st->dtype, RAD_ACT_NONE, st->D, ld, H, R, ld, G, H, nullptr, nullptr, 0, dW, ldw, nullptr, 0,
                            nullptr, dev_status, stream);
}

}  // namespace rad

using namespace rad;

extern "C" int rad_rademacher(int32_t dtype, int64_t D, float fraction, int64_t ld, uint64_t seed, uint32_t layer,
                              uint32_t step, void* out, void* stream) {
  if ((dtype != RAD_F32 && dtype != RAD_BF16) || D <= 0 || out == nullptr) return RAD_EINVAL;
  const int64_t k = draws_per_row_host(fraction, D);
  if (k == 0 || ld < k) return RAD_EINVAL;
  const int rc = check_device();
  if (rc != RAD_OK) return rc;
  return draw_signs(dtype, out, D, k, ld, seed, layer, step, static_cast<cudaStream_t>(stream));
}
