// 3x3 convolution layers with activation sampling (paper, Fig. "Convnet activation sampling",
// Sec. 4.2): the conv input is stored through the same compact store as a linear layer's input
// (one keep decision per input entry, shared by every filter tap that reads it), the ReLU
// derivative of the conv output takes one bit per entry, average pooling needs nothing, and the
// filter gradient is evaluated on the kept entries only.  NHWC, zero padding 1, stride 1, ReLU and
// 2x2 average pooling fused behind each convolution.
//
// The whole net of this configuration is about 2 GFLOP per step, so these kernels are CUDA-core
// kernels tuned for few launches and fixed summation order, not tensor-core kernels:
//   conv_forward_pool   one thread per pooled output: four conv outputs, ReLU, 4 derivative bits
//                       (a nibble; eight neighbouring channels make one word), rounded average
//   conv_dz             dZ = 0.25 * dP * bit, the conv-output gradient in the working type
//   conv_input_grad     direct transposed convolution, one thread per input entry
//   conv_weight_grad    one CTA per minibatch row: the row's kept entries are listed in shared
//                       memory from keep bits, row offsets and packed values, then every thread
//                       (filter tap, output channel) walks the list in order
#include <algorithm>
#include <cmath>

#include "common.cuh"

namespace rad {
namespace {

struct ConvShape {
  int64_t B;
  int32_t H, W, Cin, Cout;      // H, W: conv input = conv output size (padding 1)
};

// filters arrive as 3 x 3 x Cin x Cout in the working type; shared memory keeps them as float
template <typename T>
__device__ __forceinline__ void load_filters(const T* Wt, float* s_w, int n, int stride_in, int stride_out, int cout) {
  for (int i = threadIdx.x; i < n; i += blockDim.x) s_w[(i / cout) * stride_out + (i % cout)] = to_float(Wt[i]);
  (void)stride_in;
}

template <typename T>
__global__ void __launch_bounds__(256) conv_forward_pool_kernel(const ConvShape s, const T* X, const T* Wt,
                                                                const float* bias, T* P, uint32_t* relubits) {
  extern __shared__ float s_w[];                     // 9 * Cin x Cout
  load_filters(Wt, s_w, 9 * s.Cin * s.Cout, 0, s.Cout, s.Cout);
  __syncthreads();
  const int Hp = s.H / 2, Wp = s.W / 2;
  const int64_t total = s.B * Hp * Wp * s.Cout;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t nib = 0;
  if (i < total) {
    const int co = (int)(i % s.Cout);
    const int64_t pix = i / s.Cout;
    const int xp = (int)(pix % Wp), yp = (int)((pix / Wp) % Hp);
    const int64_t b = pix / ((int64_t)Wp * Hp);
    const T* Xb = X + b * s.H * s.W * s.Cin;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    // the 4 x 4 input patch around the 2 x 2 outputs
    for (int py = 0; py < 4; ++py) {
      const int yi = 2 * yp - 1 + py;
      if (yi < 0 || yi >= s.H) continue;
      for (int px = 0; px < 4; ++px) {
        const int xi = 2 * xp - 1 + px;
        if (xi < 0 || xi >= s.W) continue;
        const T* xin = Xb + ((int64_t)yi * s.W + xi) * s.Cin;
        for (int ci = 0; ci < s.Cin; ++ci) {
          const float v = to_float(xin[ci]);
#pragma unroll
          for (int o = 0; o < 4; ++o) {
            const int ky = py - (o >> 1), kx = px - (o & 1);       // tap that maps this input to output o
            if (ky >= 0 && ky < 3 && kx >= 0 && kx < 3)
              acc[o] = fmaf(v, s_w[((ky * 3 + kx) * s.Cin + ci) * s.Cout + co], acc[o]);
          }
        }
      }
    }
    const float bco = bias != nullptr ? bias[co] : 0.0f;
    float sum = 0.0f;
#pragma unroll
    for (int o = 0; o < 4; ++o) {
      const float r = to_float(from_float<T>(fmaxf(acc[o] + bco, 0.0f)));     // the activation as the device would hold it
      nib |= (r > 0.0f ? 1u : 0u) << o;
      sum += r;
    }
    P[i] = from_float<T>(0.25f * sum);
  }
  // eight neighbouring channels share one word of derivative bits: nibble k = channel co0 + k
  uint32_t word = nib << (4 * (threadIdx.x & 7));
  word |= __shfl_xor_sync(0xffffffffu, word, 1);
  word |= __shfl_xor_sync(0xffffffffu, word, 2);
  word |= __shfl_xor_sync(0xffffffffu, word, 4);
  if ((threadIdx.x & 7) == 0 && i < total) relubits[i >> 3] = word;
}

template <typename T>
__global__ void __launch_bounds__(256) conv_dz_kernel(const ConvShape s, const T* dP, const uint32_t* relubits, T* dZ) {
  const int Hp = s.H / 2, Wp = s.W / 2;
  const int64_t total = s.B * Hp * Wp * s.Cout;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int co = (int)(i % s.Cout);
  const int64_t pix = i / s.Cout;
  const int xp = (int)(pix % Wp), yp = (int)((pix / Wp) % Hp);
  const int64_t b = pix / ((int64_t)Wp * Hp);
  const uint32_t nib = (relubits[i >> 3] >> (4 * (i & 7))) & 0xfu;
  const float g = 0.25f * to_float(dP[i]);
#pragma unroll
  for (int o = 0; o < 4; ++o) {
    const int y = 2 * yp + (o >> 1), x = 2 * xp + (o & 1);
    dZ[((b * s.H + y) * s.W + x) * s.Cout + co] = from_float<T>(((nib >> o) & 1u) ? g : 0.0f);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) conv_input_grad_kernel(const ConvShape s, const T* dZ, const T* Wt, T* dX) {
  extern __shared__ float s_w[];                     // 9 * Cin rows of Cout + 1 floats (odd stride)
  const int stride = s.Cout + 1;
  for (int i = threadIdx.x; i < 9 * s.Cin * s.Cout; i += blockDim.x)
    s_w[(i / s.Cout) * stride + (i % s.Cout)] = to_float(Wt[i]);
  __syncthreads();
  const int64_t total = s.B * s.H * s.W * s.Cin;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int ci = (int)(i % s.Cin);
  const int64_t pix = i / s.Cin;
  const int xi = (int)(pix % s.W), yi = (int)((pix / s.W) % s.H);
  const int64_t b = pix / ((int64_t)s.W * s.H);
  float acc = 0.0f;
  for (int ky = 0; ky < 3; ++ky) {
    const int yo = yi - ky + 1;
    if (yo < 0 || yo >= s.H) continue;
    for (int kx = 0; kx < 3; ++kx) {
      const int xo = xi - kx + 1;
      if (xo < 0 || xo >= s.W) continue;
      const T* dz = dZ + ((b * s.H + yo) * s.W + xo) * s.Cout;
      const float* w = s_w + ((ky * 3 + kx) * s.Cin + ci) * stride;
      for (int co = 0; co < s.Cout; ++co) acc = fmaf(to_float(dz[co]), w[co], acc);
    }
  }
  dX[i] = from_float<T>(acc);
}

struct ConvDwParams {
  ConvShape s;
  int32_t variant;
  const void* values; const uint32_t* keepbits; const uint32_t* offsets; const int64_t* nnz;
  int64_t values_capacity, values_ld;
  int32_t ncb;
  const void* dZ;
  float* partial;               // B x (9 * Cin * Cout)
  int32_t list_cap;
};

// One CTA per minibatch row b; blockDim = 9 * Cout threads (tap, co).
template <typename T>
__global__ void conv_weight_grad_kernel(const ConvDwParams p) {
  extern __shared__ float sm[];
  const ConvShape& s = p.s;
  const int ncell = 9 * s.Cin * s.Cout;
  float* s_dw = sm;                                               // 9 * Cin x Cout partial of this row
  uint32_t* s_pos = reinterpret_cast<uint32_t*>(s_dw + ncell);    // kept entries: yi << 20 | xi << 10 | ci
  float* s_val = reinterpret_cast<float*>(s_pos + p.list_cap);
  __shared__ uint32_t s_scan[32];
  __shared__ uint32_t s_count;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = (blockDim.x + 31) >> 5;
  const int64_t b = blockIdx.x;
  const int64_t D = (int64_t)s.H * s.W * s.Cin;
  for (int i = tid; i < ncell; i += blockDim.x) s_dw[i] = 0.0f;
  if (tid == 0) s_count = 0;
  __syncthreads();
  const T* vals = static_cast<const T*>(p.values);
  auto put = [&](uint32_t at, int64_t col, float v) {
    if (at < (uint32_t)p.list_cap) {
      const int ci = (int)(col % s.Cin);
      const int64_t pix = col / s.Cin;
      s_pos[at] = ((uint32_t)(pix / s.W) << 20) | ((uint32_t)(pix % s.W) << 10) | (uint32_t)ci;
      s_val[at] = v;
    }
  };
  if (p.variant == RAD_SAME_SAMPLE) {
    const int64_t k = min(p.nnz[0], p.values_ld);
    for (int64_t j = tid; j < k; j += blockDim.x) put((uint32_t)j, p.offsets[j], to_float(vals[b * p.values_ld + j]));
    if (tid == 0) s_count = (uint32_t)min(k, (int64_t)p.list_cap);
  } else {
    // row b of the tile-major store: slab b / 64, row r inside it; one keep-bit word per thread and pass
    const int64_t slab = b / kTileRows;
    const int r = (int)(b % kTileRows);
    const int nwords = p.ncb * 4;
    for (int w0 = 0; w0 < nwords; w0 += blockDim.x) {
      const int wi = w0 + tid;
      uint32_t word = 0, inrow = 0;
      int64_t tile = 0;
      if (wi < nwords) {
        tile = slab * p.ncb + (wi >> 2);
        const uint32_t* tb = p.keepbits + tile * kTileWords;
        word = tb[r * 4 + (wi & 3)];
        for (int q = 0; q < (wi & 3); ++q) inrow += __popc(tb[r * 4 + q]);
        inrow += (tb[kBitWords + (r >> 1)] >> (16 * (r & 1))) & 0xffffu;          // row offset inside the tile
      }
      const uint32_t c = __popc(word);
      uint32_t incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (lane == 31) s_scan[warp] = incl;
      __syncthreads();
      uint32_t base = s_count;
      for (int q = 0; q < warp; ++q) base += s_scan[q];
      uint32_t at = base + incl - c;
      int64_t vpos = (int64_t)p.offsets[tile] + inrow;
      uint32_t rest = word;
      while (rest != 0) {
        const int bit = __ffs(rest) - 1;
        rest &= rest - 1;
        const float v = vpos < p.values_capacity ? to_float(vals[vpos]) : 0.0f;
        put(at, (int64_t)(wi >> 2) * kTileCols + (wi & 3) * 32 + bit, v);
        ++at; ++vpos;
      }
      __syncthreads();
      if (tid == 0) {
        uint32_t tot = s_count;
        for (int q = 0; q < nwarps; ++q) tot += s_scan[q];
        s_count = min(tot, (uint32_t)p.list_cap);
      }
      __syncthreads();
    }
  }
  __syncthreads();
  // thread (tap, co) adds every kept entry's contribution to its own cells, in list order
  const int co = tid % s.Cout, tap = tid / s.Cout;
  if (tap < 9) {
    const int ky = tap / 3, kx = tap % 3;
    const T* dZb = static_cast<const T*>(p.dZ) + b * s.H * s.W * s.Cout;
    float* mine = s_dw + (int64_t)tap * s.Cin * s.Cout + co;
    const uint32_t n = s_count;
    for (uint32_t e = 0; e < n; ++e) {
      const uint32_t pe = s_pos[e];
      const int yo = (int)(pe >> 20) - ky + 1, xo = (int)((pe >> 10) & 0x3ffu) - kx + 1;
      if (yo < 0 || yo >= s.H || xo < 0 || xo >= s.W) continue;
      const int ci = (int)(pe & 0x3ffu);
      mine[ci * s.Cout] = fmaf(s_val[e], to_float(dZb[((int64_t)yo * s.W + xo) * s.Cout + co]), mine[ci * s.Cout]);
    }
  }
  __syncthreads();
  for (int i = tid; i < ncell; i += blockDim.x) p.partial[b * ncell + i] = s_dw[i];
  (void)D;
}

// out[i] = sum over rows of part[b][i], in row order
__global__ void __launch_bounds__(256) conv_sum_rows_kernel(const float* part, int64_t B, int64_t n, float* out) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float acc = 0.0f;
  for (int64_t b = 0; b < B; ++b) acc += part[b * n + i];
  out[i] = acc;
}

}  // namespace

// ---- launchers used by the whole-net step ---------------------------------------------------------------
int conv_forward_pool(int dtype, int64_t B, int H, int W, int Cin, int Cout, const void* X, const void* Wt,
                      const float* bias, void* P, uint32_t* relubits, cudaStream_t st) {
  ConvShape s = {B, H, W, Cin, Cout};
  const int64_t total = B * (H / 2) * (W / 2) * Cout;
  const size_t smem = (size_t)9 * Cin * Cout * 4;
  const unsigned grid = (unsigned)ceil_div(total, 256);
  count_launch();
  if (dtype == RAD_BF16) {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_forward_pool_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_forward_pool_kernel<bf16><<<grid, 256, smem, st>>>(s, static_cast<const bf16*>(X), static_cast<const bf16*>(Wt), bias,
                                                           static_cast<bf16*>(P), relubits);
  } else {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_forward_pool_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_forward_pool_kernel<float><<<grid, 256, smem, st>>>(s, static_cast<const float*>(X), static_cast<const float*>(Wt), bias,
                                                            static_cast<float*>(P), relubits);
  }
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

int conv_dz(int dtype, int64_t B, int H, int W, int Cout, const void* dP, const uint32_t* relubits, void* dZ,
            cudaStream_t st) {
  ConvShape s = {B, H, W, 0, Cout};
  const unsigned grid = (unsigned)ceil_div(B * (H / 2) * (W / 2) * Cout, 256);
  count_launch();
  if (dtype == RAD_BF16)
    conv_dz_kernel<bf16><<<grid, 256, 0, st>>>(s, static_cast<const bf16*>(dP), relubits, static_cast<bf16*>(dZ));
  else
    conv_dz_kernel<float><<<grid, 256, 0, st>>>(s, static_cast<const float*>(dP), relubits, static_cast<float*>(dZ));
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

int conv_input_grad(int dtype, int64_t B, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, void* dX,
                    cudaStream_t st) {
  ConvShape s = {B, H, W, Cin, Cout};
  const size_t smem = (size_t)9 * Cin * (Cout + 1) * 4;
  const unsigned grid = (unsigned)ceil_div(B * H * W * Cin, 256);
  count_launch();
  if (dtype == RAD_BF16) {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_input_grad_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_input_grad_kernel<bf16><<<grid, 256, smem, st>>>(s, static_cast<const bf16*>(dZ), static_cast<const bf16*>(Wt),
                                                         static_cast<bf16*>(dX));
  } else {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_input_grad_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_input_grad_kernel<float><<<grid, 256, smem, st>>>(s, static_cast<const float*>(dZ), static_cast<const float*>(Wt),
                                                          static_cast<float*>(dX));
  }
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

int64_t conv_weight_grad_workspace(int64_t B, int Cin, int Cout) { return round_up(B * 9 * Cin * Cout * 4, 256); }

int conv_weight_grad(const rad_store* store, int H, int W, int Cin, int Cout, const void* dZ, float* dW, void* workspace,
                     int64_t workspace_bytes, cudaStream_t st) {
  if (workspace == nullptr || workspace_bytes < conv_weight_grad_workspace(store->B, Cin, Cout)) return RAD_EWORKSPACE;
  if (9 * Cout > 1024 || H >= 1024 || W >= 1024 || Cin >= 1024) return RAD_ELIMIT;
  ConvDwParams p;
  p.s = {store->B, H, W, Cin, Cout};
  p.variant = store->variant;
  p.values = store->values; p.keepbits = store->keepbits; p.offsets = store->offsets; p.nnz = store->nnz;
  p.values_capacity = store->values_capacity; p.values_ld = store->values_ld;
  p.ncb = (int32_t)ceil_div(store->D, kTileCols);
  p.dZ = dZ; p.partial = static_cast<float*>(workspace);
  p.list_cap = (int32_t)store->D;
  const int64_t ncell = (int64_t)9 * Cin * Cout;
  const size_t smem = (size_t)ncell * 4 + (size_t)p.list_cap * 8;
  if (smem > 200 * 1024) return RAD_ELIMIT;
  const int threads = (int)round_up(9 * Cout, 32);
  count_launch(2);
  if (store->dtype == RAD_BF16) {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_weight_grad_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_weight_grad_kernel<bf16><<<(unsigned)store->B, threads, smem, st>>>(p);
  } else {
    RAD_CUDA_TRY(cudaFuncSetAttribute(conv_weight_grad_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    conv_weight_grad_kernel<float><<<(unsigned)store->B, threads, smem, st>>>(p);
  }
  conv_sum_rows_kernel<<<(unsigned)ceil_div(ncell, 256), 256, 0, st>>>(p.partial, store->B, ncell, dW);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad
