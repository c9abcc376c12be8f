// Softmax cross-entropy and its Jacobian (exact; Sec. 4.2: the loss Jacobian is never sampled).
#include "common.cuh"

namespace rad {
namespace {

// One warp per row: loss_b = logsumexp(z_b) - z_b[label]; dZ = (softmax - onehot) / B.
template <typename T>
__global__ void __launch_bounds__(256) xent_rows_kernel(const float* logits, int64_t ldl, const int32_t* labels,
                                                        int64_t B, int64_t C, T* dZ, int64_t ldz,
                                                        float* row_loss) {
  const int lane = threadIdx.x & 31;
  const int64_t b = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;
  const float* z = logits + b * ldl;
  float mx = -INFINITY;
  for (int64_t c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.0f;
  for (int64_t c = lane; c < C; c += 32) sum += expf(z[c] - mx);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const int32_t y = labels[b];
  const float inv = 1.0f / sum, invB = 1.0f / (float)B;
  for (int64_t c = lane; c < C; c += 32) {
    float g = expf(z[c] - mx) * inv;
    if (c == y) g -= 1.0f;
    dZ[b * ldz + c] = from_float<T>(g * invB);
  }
  if (lane == 0) row_loss[b] = (y >= 0 && y < C) ? (logf(sum) + mx - z[y]) : 0.0f;
}

// Rows and mean in one launch for small batches (the small nets are bound by their launch count): one CTA, a
// warp takes rows w, w + 32, ..., then the same fixed-order mean as below over the row losses in shared memory.
constexpr int kXentSmallRows = 2048;
template <typename T>
__global__ void __launch_bounds__(1024) xent_small_kernel(const float* logits, int64_t ldl, const int32_t* labels, int64_t B,
                                                          int64_t C, T* dZ, int64_t ldz, float* loss) {
  __shared__ float s_row[kXentSmallRows];
  __shared__ float s[1024];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t b = warp; b < B; b += 32) {
    const float* z = logits + b * ldl;
    float mx = -INFINITY;
    for (int64_t c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.0f;
    for (int64_t c = lane; c < C; c += 32) sum += expf(z[c] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const int32_t y = labels[b];
    const float inv = 1.0f / sum, invB = 1.0f / (float)B;
    for (int64_t c = lane; c < C; c += 32) {
      float g = expf(z[c] - mx) * inv;
      if (c == y) g -= 1.0f;
      dZ[b * ldz + c] = from_float<T>(g * invB);
    }
    if (lane == 0) s_row[b] = (y >= 0 && y < C) ? (logf(sum) + mx - z[y]) : 0.0f;
  }
  __syncthreads();
  float acc = 0.0f;
  for (int64_t i = threadIdx.x; i < B; i += 1024) acc += s_row[i];
  s[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *loss = s[0] / (float)B;
}

// Fixed-order mean of the per-row losses (one CTA).
__global__ void __launch_bounds__(1024) mean_kernel(const float* row_loss, int64_t B, float* loss) {
  __shared__ float s[1024];
  float acc = 0.0f;
  for (int64_t i = threadIdx.x; i < B; i += 1024) acc += row_loss[i];
  s[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *loss = s[0] / (float)B;
}

}  // namespace
}  // namespace rad

using namespace rad;

extern "C" int rad_softmax_xent(int32_t dtype, int64_t B, int64_t C, const float* logits, int64_t ldl,
                                const int32_t* labels, float* loss, void* dZ, int64_t ldz, void* workspace,
                                int64_t workspace_bytes, void* stream) {
  if (B <= 0 || C <= 0 || logits == nullptr || labels == nullptr || loss == nullptr || dZ == nullptr)
    return RAD_EINVAL;
  if (ldl < C || ldz < C) return RAD_EINVAL;
  if (dtype != RAD_F32 && dtype != RAD_BF16) return RAD_EINVAL;
  if (workspace == nullptr || workspace_bytes < B * 4) return RAD_EWORKSPACE;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (B <= kXentSmallRows) {
    count_launch();
    if (dtype == RAD_BF16)
      xent_small_kernel<bf16><<<1, 1024, 0, s>>>(logits, ldl, labels, B, C, static_cast<bf16*>(dZ), ldz, loss);
    else
      xent_small_kernel<float><<<1, 1024, 0, s>>>(logits, ldl, labels, B, C, static_cast<float*>(dZ), ldz, loss);
    RAD_CUDA_TRY(cudaGetLastError());
    return RAD_OK;
  }
  float* rows = static_cast<float*>(workspace);
  const unsigned grid = (unsigned)ceil_div(B, 8);
  count_launch(2);
  if (dtype == RAD_BF16)
    xent_rows_kernel<bf16><<<grid, 256, 0, s>>>(logits, ldl, labels, B, C, static_cast<bf16*>(dZ), ldz, rows);
  else
    xent_rows_kernel<float><<<grid, 256, 0, s>>>(logits, ldl, labels, B, C, static_cast<float*>(dZ), ldz, rows);
  mean_kernel<<<1, 1024, 0, s>>>(rows, B, loss);
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}
