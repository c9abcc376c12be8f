// CUDA-core (FFMA) kernels: the float32 nets, whose 1e-5 tolerance rules out tensor-core input
// rounding, and bf16 problems whose shapes the TMA path cannot take.  These problems are small
// and latency-bound; the kernels favour exact float32 accumulation in a fixed order over speed.
#include <algorithm>
#include <cmath>

#include "common.cuh"

namespace rad {
namespace {

constexpr int kBM = 64, kBN = 64;      // the larger of the two tiles

enum Epilogue { kEpiForward = 0, kEpiInputGrad = 1, kEpiScatterRows = 2 };

struct GemmParams {
  // C(m, n) = sum_k A(m, k) * Bm(k, n); element (m, k) of A at A[m * sam + k * sak], etc.
  const void* A; int64_t sam, sak;
  const void* Bm; int64_t sbk, sbn;
  int64_t M, N, K;
  const int64_t* M_dev;        // optional: M read from device memory (clamped to M)
  // forward epilogue
  const float* bias; int act;
  void* out_act; int64_t ld_act;
  float* out_z; int64_t ld_z;
  void* out_zlow; int64_t ld_zlow;
  // input-grad epilogue
  const uint32_t* relubits; int64_t w32;
  const void* z_prev; int64_t ld_zprev;
  void* out_low; int64_t ld_low;
  // scatter-rows epilogue (same-sample dW): row m goes to row idx[m] of out_f32
  const uint32_t* row_idx;
  float* out_f32; int64_t ld_f32;
  float* db;                   // or NULL: column sums of Bm over k (the bias gradient), from the CTAs of tile row 0
  int tile;                    // 64 or 32: rows and columns of C per CTA
};

// One TS x TS tile of C (TS = 64, or 32 where 64 would leave most SMs without a CTA) by one CTA of 256 threads,
// TS/16 x TS/16 outputs per thread; (bx, by) = tile column and row.  The K loop is double
// buffered: the next 16 rows of K travel from global memory to registers while the current ones are
// multiplied out of shared memory, one barrier per step (these GEMMs serve the small nets, where a CTA's time
// is the latency of its loads).  Every output is one chain of fused multiply-adds over k in ascending order.
// K rows per step: the small tile takes four times as many, so that its steps, which are bound by the latency
// of their loads, are a quarter as many.
constexpr int gemm_bk(int ts) { return ts == 32 ? 64 : 16; }
constexpr int kGemmSmemFloats = 4 * gemm_bk(32) * (32 + 4) > 4 * gemm_bk(64) * (64 + 4) ? 4 * gemm_bk(32) * (32 + 4)
                                                                                         : 4 * gemm_bk(64) * (64 + 4);
static_assert(kBM == kBN, "both operands share the staging layout");
template <typename T, int EPI, int TS>
__device__ __forceinline__ void gemm_body(const GemmParams& p, int64_t bx, int64_t by, float* smem) {
  constexpr int kBM = TS, kBN = TS, TM = TS / 16, kBK = gemm_bk(TS), NF = TS * kBK / 256;
  constexpr int kLdS = TS + 4;                       // floats per k row of a staged operand (16-byte multiples)
  static_assert((kLdS * 4) % 16 == 0 && (TM == 4 || TM == 2), "vector reads of the staged operands");
  int64_t M = p.M;
  if (p.M_dev != nullptr) M = min(M, *p.M_dev);
  const int64_t m0 = by * kBM, n0 = bx * kBN;
  const bool sums = EPI == kEpiScatterRows && p.db != nullptr && by == 0;
  if (m0 >= M && !sums) return;
  const int tid = threadIdx.x;
  float colsum = 0.0f;
  const int tm = (tid >> 4) * TM, tn = (tid & 15) * TM;
  const T* A = static_cast<const T*>(p.A);
  const T* Bm = static_cast<const T*>(p.Bm);
  float acc[TM][TM] = {};
  // TS x kBK elements of each operand per step; whichever index is contiguous in memory is made
  // the fast thread index
  float ra[NF], rb[NF];
  auto fetch = [&](int64_t k0) {
#pragma unroll
    for (int j = 0; j < NF; ++j) {
      const int i = tid + j * 256;
      int mm, kk;
      if (p.sak == 1) { kk = i % kBK; mm = i / kBK; } else { mm = i % kBM; kk = i / kBM; }
      const int64_t m = m0 + mm, k = k0 + kk;
      ra[j] = (m < M && k < p.K) ? to_float(A[m * p.sam + k * p.sak]) : 0.0f;
      int nn;
      if (p.sbk == 1) { kk = i % kBK; nn = i / kBK; } else { nn = i % kBN; kk = i / kBN; }
      const int64_t n = n0 + nn, kb = k0 + kk;
      rb[j] = (n < p.N && kb < p.K) ? to_float(Bm[kb * p.sbk + n * p.sbn]) : 0.0f;
    }
  };
  auto stash = [&](int buf) {
    float* sA = smem + buf * 2 * kBK * kLdS;
    float* sB = sA + kBK * kLdS;
#pragma unroll
    for (int j = 0; j < NF; ++j) {
      const int i = tid + j * 256;
      if (p.sak == 1) sA[(i % kBK) * kLdS + i / kBK] = ra[j]; else sA[(i / kBM) * kLdS + i % kBM] = ra[j];
      if (p.sbk == 1) sB[(i % kBK) * kLdS + i / kBK] = rb[j]; else sB[(i / kBN) * kLdS + i % kBN] = rb[j];
    }
  };
  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int64_t k0 = 0; k0 < p.K; k0 += kBK) {
    const bool more = k0 + kBK < p.K;
    if (more) fetch(k0 + kBK);
    const float* sA = smem + buf * 2 * kBK * kLdS;
    const float* sB = sA + kBK * kLdS;
    if (sums && tid < kBN) {
      // the block of Bm is in shared memory anyway: its column sums, row after row (rows past K hold zeros)
#pragma unroll
      for (int kk = 0; kk < kBK; ++kk) colsum += sB[kk * kLdS + tid];
    }
#pragma unroll
    for (int kk = 0; kk < kBK; ++kk) {
      float a[TM], b[TM];
      if (TM == 4) {
        const float4 a4 = *reinterpret_cast<const float4*>(sA + kk * kLdS + tm);
        const float4 b4 = *reinterpret_cast<const float4*>(sB + kk * kLdS + tn);
        a[0] = a4.x; a[1] = a4.y; a[TM - 2] = a4.z; a[TM - 1] = a4.w;
        b[0] = b4.x; b[1] = b4.y; b[TM - 2] = b4.z; b[TM - 1] = b4.w;
      } else {
        const float2 a2 = *reinterpret_cast<const float2*>(sA + kk * kLdS + tm);
        const float2 b2 = *reinterpret_cast<const float2*>(sB + kk * kLdS + tn);
        a[0] = a2.x; a[1] = a2.y;
        b[0] = b2.x; b[1] = b2.y;
      }
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TM; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) stash(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
  if (sums && tid < kBN && n0 + tid < p.N) p.db[n0 + tid] = colsum;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int64_t m = m0 + tm + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < TM; ++j) {
      const int64_t n = n0 + tn + j;
      if (n >= p.N) continue;
      float v = acc[i][j];
      if (EPI == kEpiForward) {
        if (p.bias != nullptr) v += p.bias[n];
        if (p.out_z != nullptr) p.out_z[m * p.ld_z + n] = v;
        if (p.out_zlow != nullptr) static_cast<T*>(p.out_zlow)[m * p.ld_zlow + n] = from_float<T>(v);
        if (p.out_act != nullptr) {
          const float a = p.act == RAD_ACT_RELU ? fmaxf(v, 0.0f) : p.act == RAD_ACT_GELU ? gelu_f(v) : v;
          static_cast<T*>(p.out_act)[m * p.ld_act + n] = from_float<T>(a);
        }
      } else if (EPI == kEpiInputGrad) {
        if (p.relubits != nullptr) {
          if (((p.relubits[m * p.w32 + (n >> 5)] >> (n & 31)) & 1u) == 0) v = 0.0f;
        } else if (p.z_prev != nullptr) {
          v *= gelu_grad_f(to_float(static_cast<const T*>(p.z_prev)[m * p.ld_zprev + n]));
        }
        static_cast<T*>(p.out_low)[m * p.ld_low + n] = from_float<T>(v);
      } else {
        p.out_f32[(int64_t)p.row_idx[m] * p.ld_f32 + n] = v;
      }
    }
  }
}

// The tile a GEMM of M x N outputs runs with, and the body for it.
inline int pick_tile(int64_t M, int64_t N) { return ceil_div(M, 64) * ceil_div(N, 64) < 64 ? 32 : 64; }
template <typename T, int EPI>
__device__ __forceinline__ void gemm_tile(const GemmParams& p, int64_t bx, int64_t by, float* smem) {
  if (p.tile == 32) gemm_body<T, EPI, 32>(p, bx, by, smem);
  else gemm_body<T, EPI, 64>(p, bx, by, smem);
}

template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_kernel(const GemmParams p) {
  __shared__ __align__(16) float smem[kGemmSmemFloats];
  gemm_tile<T, EPI>(p, blockIdx.x, blockIdx.y, smem);
}

template <int EPI>
int launch_gemm(int dtype, const GemmParams& p0, int64_t Mgrid, cudaStream_t s) {
  GemmParams p = p0;
  p.tile = pick_tile(Mgrid, p.N);
  dim3 grid((unsigned)ceil_div(p.N, p.tile), (unsigned)ceil_div(Mgrid, p.tile));
  if (grid.x == 0 || grid.y == 0) return RAD_OK;
  count_launch();
  if (dtype == RAD_BF16)
    gemm_kernel<bf16, EPI><<<grid, 256, 0, s>>>(p);
  else
    gemm_kernel<float, EPI><<<grid, 256, 0, s>>>(p);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// relubits[b, w] = bits of (X[b, 32w..] > 0)
template <typename T>
__global__ void __launch_bounds__(256) relu_bits_rows_kernel(const T* X, int64_t ld, int64_t B, int64_t H,
                                                             int64_t w32, uint32_t* out) {
  const int64_t n = B * w32;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = i / w32, w = i % w32;
    const T* rowp = X + b * ld + w * 32;
    const int nv = (int)min((int64_t)32, H - w * 32);
    uint32_t m = 0;
    for (int c = 0; c < nv; ++c) m |= (to_float(rowp[c]) > 0.0f ? 1u : 0u) << c;
    out[i] = m;
  }
}

// ---- different-sample dW on CUDA cores ----------------------------------------------------------
// One CTA owns 128 columns d of the layer input (one column block) and 32 outputs h.  Per row slab
// it rebuilds the 64 x 128 tile of A_hat in shared memory from keep bits and packed values
// (per-word popcount prefix), then accumulates A_hat^T dZ.
constexpr int kSparseBN = 32;
struct SparseDwParams {
  const void* values; const uint32_t* keepbits; const uint32_t* offsets;
  int64_t capacity;
  int64_t B, D, H; int32_t ncb, nslabs;
  const void* dZ; int64_t ldz;
  float* dW; int64_t ldw;
  float* db;                 // or NULL: column sums of dZ (the bias gradient), from the CTAs of column block 0
};

template <typename T>
__device__ __forceinline__ void sparse_dw_body(const SparseDwParams& p, int cb, int64_t by, float (*sAh)[kTileCols + 1],
                                               float (*sZ)[kSparseBN + 1], uint32_t* s_scan) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t h0 = by * kSparseBN;
  const T* vals = static_cast<const T*>(p.values);
  const T* dZ = static_cast<const T*>(p.dZ);
  // 128 x 32 outputs over 256 threads: 4 columns d x 4 outputs h each
  const int td = (tid >> 3) * 4, th = (tid & 7) * 4;
  float acc[4][4] = {};
  float db_acc = 0.0f;
  for (int slab = 0; slab < p.nslabs; ++slab) {
    const int64_t tile = (int64_t)slab * p.ncb + cb;
    const uint32_t word = p.keepbits[tile * kTileWords + tid];    // row tid/4, word tid%4
    const uint32_t cnt = __popc(word);
    // exclusive scan of the 256 per-word counts
    uint32_t incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    uint32_t wbase = 0;
    for (int w = 0; w < warp; ++w) wbase += s_scan[w];
    const int64_t base = p.offsets[tile] + (wbase + incl - cnt);
    const int r = tid >> 2, c0 = (tid & 3) * 32;
    // every kept entry's place follows from the word alone, so the loads do not wait for one another
#pragma unroll 16
    for (int b = 0; b < 32; ++b) {
      const int64_t at = base + __popc(word & ((1u << b) - 1u));
      float v = 0.0f;
      if (((word >> b) & 1u) != 0 && at < p.capacity) v = to_float(vals[at]);   // a store that overflowed is never read past
      sAh[r][c0 + b] = v;
    }
    for (int i = tid; i < kTileRows * kSparseBN; i += 256) {
      const int rr = i / kSparseBN, hh = i % kSparseBN;
      const int64_t row = (int64_t)slab * kTileRows + rr, h = h0 + hh;
      sZ[rr][hh] = (row < p.B && h < p.H) ? to_float(dZ[row * p.ldz + h]) : 0.0f;
    }
    __syncthreads();
    if (p.db != nullptr && cb == 0 && tid < kSparseBN) {
      // the dZ block is in shared memory anyway: its column sums, slab after slab in row order
      float sum = 0.0f;
      for (int rr = 0; rr < kTileRows; ++rr) sum += sZ[rr][tid];
      db_acc += sum;
    }
#pragma unroll 4
    for (int rr = 0; rr < kTileRows; ++rr) {
      float a[4], z[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = sAh[rr][td + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) z[j] = sZ[rr][th + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], z[j], acc[i][j]);
    }
    __syncthreads();
  }
  if (p.db != nullptr && cb == 0 && tid < kSparseBN && h0 + tid < p.H) p.db[h0 + tid] = db_acc;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t d = (int64_t)cb * kTileCols + td + i;
    if (d >= p.D) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t h = h0 + th + j;
      if (h < p.H) p.dW[d * p.ldw + h] = acc[i][j];
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) sparse_dw_kernel(const SparseDwParams p) {
  __shared__ float sAh[kTileRows][kTileCols + 1];
  __shared__ float sZ[kTileRows][kSparseBN + 1];
  __shared__ uint32_t s_scan[256];
  sparse_dw_body<T>(p, (int)blockIdx.x, blockIdx.y, sAh, sZ, s_scan);
}

// dW of a layer and the gradient of its input in one launch: both read the same dZ and neither reads the
// other's result, so the first `dw_blocks` CTAs are those of sparse_dw_kernel and the rest those of the
// input-gradient GEMM, each doing exactly what it does in a launch of its own (the nets that run on CUDA
// cores are bound by their launch count).
constexpr int kDwDxSmemA = kTileRows * (kTileCols + 1) * 4, kDwDxSmemZ = kTileRows * (kSparseBN + 1) * 4;
static_assert(kDwDxSmemA + kDwDxSmemZ + 1024 >= kGemmSmemFloats * 4, "the GEMM's tiles fit the same buffer");
template <typename T>
__global__ void __launch_bounds__(256) dw_dx_kernel(const SparseDwParams d, const GemmParams g, int dw_blocks, int gx) {
  __shared__ __align__(16) unsigned char raw[kDwDxSmemA + kDwDxSmemZ + 1024];
  if ((int)blockIdx.x < dw_blocks) {
    sparse_dw_body<T>(d, (int)(blockIdx.x % d.ncb), blockIdx.x / d.ncb, reinterpret_cast<float(*)[kTileCols + 1]>(raw),
                      reinterpret_cast<float(*)[kSparseBN + 1]>(raw + kDwDxSmemA),
                      reinterpret_cast<uint32_t*>(raw + kDwDxSmemA + kDwDxSmemZ));
  } else {
    const int b = (int)blockIdx.x - dw_blocks;
    gemm_tile<T, kEpiInputGrad>(g, b % gx, b / gx, reinterpret_cast<float*>(raw));
  }
}

__global__ void zero_rows_kernel(float* dW, int64_t ldw, int64_t D, int64_t H) {
  const int64_t n = D * H;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x)
    dW[(i / H) * ldw + (i % H)] = 0.0f;
}

// ---- column sums (bias gradient), two fixed-order stages ------------------------------------------
constexpr int kColChunkRows = 128;
template <typename T>
__global__ void __launch_bounds__(256) colsum_partial_kernel(const T* dZ, int64_t ldz, int64_t B, int64_t H,
                                                             float* partial) {
  const int64_t h = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (h >= H) return;
  const int64_t b0 = (int64_t)blockIdx.y * kColChunkRows, b1 = min(B, b0 + kColChunkRows);
  float s = 0.0f;
#pragma unroll 8
  for (int64_t b = b0; b < b1; ++b) s += to_float(dZ[b * ldz + h]);
  partial[(int64_t)blockIdx.y * H + h] = s;
}
// The same chunk sums with 16-byte loads: a thread owns eight neighbouring bf16 columns (two bytes per load and
// lane leave most of the memory system idle); rows in the same order, so the sums are the same numbers.
__global__ void __launch_bounds__(256) colsum_partial_vec8_kernel(const bf16* dZ, int64_t ldz, int64_t B, int64_t H,
                                                                  float* partial) {
  const int64_t h = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 8;
  if (h >= H) return;
  const int64_t b0 = (int64_t)blockIdx.y * kColChunkRows, b1 = min(B, b0 + kColChunkRows);
  float s[8] = {};
#pragma unroll 8
  for (int64_t b = b0; b < b1; ++b) {
    const uint4 v = *reinterpret_cast<const uint4*>(dZ + b * ldz + h);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      s[2 * i] += __uint_as_float(w[i] << 16);
      s[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  float4* out = reinterpret_cast<float4*>(partial + (int64_t)blockIdx.y * H + h);
  out[0] = make_float4(s[0], s[1], s[2], s[3]);
  out[1] = make_float4(s[4], s[5], s[6], s[7]);
}
__global__ void __launch_bounds__(256) colsum_final_kernel(const float* partial, int64_t chunks, int64_t H,
                                                           float* db) {
  const int64_t h = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (h >= H) return;
  float s = 0.0f;
#pragma unroll 8
  for (int64_t c = 0; c < chunks; ++c) s += partial[c * H + h];      // loads in flight together, added in order
  db[h] = s;
}
// First stage for a narrow matrix (at most 64 columns, e.g. the bias gradient of a convolution: B H W rows, 16
// columns), where one thread per column would leave most of a CTA idle: the CTA's threads are R row lanes x HP
// columns (HP the power of two that holds H); a lane sums every R-th row of the CTA's slab, then the column's
// lanes are added in lane order.  Second stage as above.
template <typename T>
__global__ void __launch_bounds__(256) colsum_narrow_partial_kernel(const T* dZ, int64_t ldz, int64_t B, int H, int HP,
                                                                    int64_t rows_per_block, float* partial) {
  __shared__ float s[256];
  const int c = threadIdx.x & (HP - 1), r = threadIdx.x / HP, R = 256 / HP;
  const int64_t b0 = (int64_t)blockIdx.x * rows_per_block, b1 = min(B, b0 + rows_per_block);
  float sum = 0.0f;
  if (c < H)
#pragma unroll 8
    for (int64_t b = b0 + r; b < b1; b += R) sum += to_float(dZ[b * ldz + c]);
  s[threadIdx.x] = sum;
  __syncthreads();
  if (r == 0 && c < H) {
    float t = 0.0f;
    for (int i = 0; i < R; ++i) t += s[i * HP + c];
    partial[(int64_t)blockIdx.x * H + c] = t;
  }
}
// Both stages in one launch for few rows (the small nets are bound by their launch count): the same chunk sums,
// added in the same order, by the thread that owns the column.
constexpr int kColSmallChunks = 2;
template <typename T>
__global__ void __launch_bounds__(256) colsum_small_kernel(const T* dZ, int64_t ldz, int64_t B, int64_t H, float* db) {
  const int64_t h = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (h >= H) return;
  float total = 0.0f;
  for (int64_t b0 = 0; b0 < B; b0 += kColChunkRows) {
    const int64_t b1 = min(B, b0 + kColChunkRows);
    float s = 0.0f;
#pragma unroll 8
    for (int64_t b = b0; b < b1; ++b) s += to_float(dZ[b * ldz + h]);
    total += s;
  }
  db[h] = total;
}

}  // namespace

// The same for a same-sample store (Sec. 4.3): the first CTAs scatter A_c^T dZ into the kept rows of dW (and
// leave the bias gradient), the next ones make the input gradient, the last ones write zeros to the rows of dW
// whose column was not kept (bit d of keep_cols clear), which the scatter never touches.
template <typename T>
__global__ void __launch_bounds__(256) same_dw_dx_kernel(const GemmParams w, const GemmParams g, int dw_blocks, int gxw,
                                                         int dx_blocks, int gxg, const uint32_t* keep_cols, int64_t D, int64_t H) {
  __shared__ __align__(16) float smem[kGemmSmemFloats];
  const int b = (int)blockIdx.x;
  if (b < dw_blocks) {
    gemm_tile<T, kEpiScatterRows>(w, b % gxw, b / gxw, smem);
  } else if (b < dw_blocks + dx_blocks) {
    gemm_tile<T, kEpiInputGrad>(g, (b - dw_blocks) % gxg, (b - dw_blocks) / gxg, smem);
  } else {
    const int nz = (int)gridDim.x - dw_blocks - dx_blocks;
    for (int64_t d = b - dw_blocks - dx_blocks; d < D; d += nz) {
      if ((keep_cols[d >> 5] >> (d & 31)) & 1u) continue;
      for (int64_t h = threadIdx.x; h < H; h += 256) w.out_f32[d * w.ld_f32 + h] = 0.0f;
    }
  }
}

int simt_forward(int dtype, int act, int64_t B, int64_t D, int64_t H, const void* A, int64_t lda,
                 const void* W, int64_t ldw, const float* bias, void* out_act, int64_t ld_act,
                 float* out_z, int64_t ld_z, void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
                 cudaStream_t s) {
  GemmParams p = {};
  p.A = A; p.sam = lda; p.sak = 1;
  p.Bm = W; p.sbk = ldw; p.sbn = 1;
  p.M = B; p.N = H; p.K = D;
  p.bias = bias; p.act = act;
  p.out_act = out_act; p.ld_act = ld_act; p.out_z = out_z; p.ld_z = ld_z;
  p.out_zlow = out_zlow; p.ld_zlow = ld_zlow;
  int rc = launch_gemm<kEpiForward>(dtype, p, B, s);
  if (rc != RAD_OK) return rc;
  if (relubits != nullptr) {
    if (out_act == nullptr) return RAD_EINVAL;
    const int64_t w32 = ceil_div(H, 32), n = B * w32;
    const int g = (int)std::min<int64_t>(ceil_div(n, 256), 148 * 16);
    count_launch();
    if (dtype == RAD_BF16)
      relu_bits_rows_kernel<bf16><<<g, 256, 0, s>>>(static_cast<const bf16*>(out_act), ld_act, B, H, w32, relubits);
    else
      relu_bits_rows_kernel<float><<<g, 256, 0, s>>>(static_cast<const float*>(out_act), ld_act, B, H, w32, relubits);
    if (cudaGetLastError() != cudaSuccess) return RAD_ECUDA;
  }
  return RAD_OK;
}

namespace {
GemmParams input_grad_params(int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz, const SimtInputGrad& ig) {
  GemmParams p = {};
  p.A = dZ; p.sam = ldz; p.sak = 1;          // (b, h)
  p.Bm = ig.W; p.sbk = 1; p.sbn = ig.ldw;    // Bm(h, d) = W[d, h]
  p.M = B; p.N = D; p.K = H;
  p.relubits = ig.relubits_prev; p.w32 = ceil_div(D, 32);
  p.z_prev = ig.z_prev; p.ld_zprev = ig.ld_zprev;
  p.out_low = ig.dZ_prev; p.ld_low = ig.ldp;
  return p;
}
}  // namespace

int simt_input_grad(int dtype, int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz,
                    const void* W, int64_t ldw, const uint32_t* relubits_prev, const void* z_prev,
                    int64_t ld_zprev, void* dZ_prev, int64_t ldp, cudaStream_t s) {
  const SimtInputGrad ig = {W, ldw, relubits_prev, z_prev, ld_zprev, dZ_prev, ldp};
  return launch_gemm<kEpiInputGrad>(dtype, input_grad_params(B, D, H, dZ, ldz, ig), B, s);
}

int simt_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW,
                     int64_t ldw, int32_t* dev_status, cudaStream_t s, float* db, bool* db_written,
                     const SimtInputGrad* ig, bool* ig_done) {
  (void)dev_status;
  if (db_written != nullptr) *db_written = false;
  if (ig_done != nullptr) *ig_done = false;
  if (st->variant == RAD_SAME_SAMPLE) {
    GemmParams p = {};
    p.A = st->values; p.sam = 1; p.sak = st->values_ld;     // A(j, b) = values[b, j]
    p.Bm = dZ; p.sbk = ldz; p.sbn = 1;
    p.M = min(st->values_ld, st->D); p.N = H; p.K = st->B;
    p.M_dev = st->nnz;
    p.row_idx = st->offsets; p.out_f32 = dW; p.ld_f32 = ldw;
    p.db = db;
    if (db_written != nullptr) *db_written = db != nullptr;
    p.tile = pick_tile(p.M, p.N);
    const int64_t gxw = ceil_div(p.N, p.tile), dw_blocks = gxw * std::max<int64_t>(1, ceil_div(p.M, p.tile));
    if (st->keepbits != nullptr) {
      // one launch: scatter, zeros for the rows not kept and, where asked for, the input gradient
      const bool with_dx = ig != nullptr && ig_done != nullptr;
      GemmParams g = with_dx ? input_grad_params(st->B, st->D, H, dZ, ldz, *ig) : GemmParams{};
      g.tile = with_dx ? pick_tile(g.M, g.N) : 64;
      const int64_t gxg = with_dx ? ceil_div(g.N, g.tile) : 1, dx_blocks = with_dx ? gxg * ceil_div(g.M, g.tile) : 0;
      const int64_t nz = std::min<int64_t>(st->D, 148 * 4);
      if (dw_blocks + dx_blocks + nz <= 0x7fffffff) {
        count_launch();
        if (st->dtype == RAD_BF16)
          same_dw_dx_kernel<bf16><<<(unsigned)(dw_blocks + dx_blocks + nz), 256, 0, s>>>(p, g, (int)dw_blocks, (int)gxw, (int)dx_blocks,
                                                                                          (int)gxg, st->keepbits, st->D, H);
        else
          same_dw_dx_kernel<float><<<(unsigned)(dw_blocks + dx_blocks + nz), 256, 0, s>>>(p, g, (int)dw_blocks, (int)gxw, (int)dx_blocks,
                                                                                           (int)gxg, st->keepbits, st->D, H);
        if (with_dx) *ig_done = true;
        return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
      }
    }
    const int g = (int)std::min<int64_t>(ceil_div(st->D * H, 256), 148 * 16);
    count_launch();
    zero_rows_kernel<<<g, 256, 0, s>>>(dW, ldw, st->D, H);
    return launch_gemm<kEpiScatterRows>(st->dtype, p, std::max<int64_t>(p.M, 1), s);
  }
  SparseDwParams p;
  p.values = st->values; p.keepbits = st->keepbits; p.offsets = st->offsets;
  p.capacity = st->values_capacity;
  p.B = st->B; p.D = st->D; p.H = H;
  p.ncb = (int32_t)ceil_div(st->D, kTileCols); p.nslabs = (int32_t)ceil_div(st->B, kTileRows);
  p.dZ = dZ; p.ldz = ldz; p.dW = dW; p.ldw = ldw;
  p.db = db;
  if (db_written != nullptr) *db_written = db != nullptr;
  dim3 grid((unsigned)p.ncb, (unsigned)ceil_div(H, kSparseBN));
  count_launch();
  if (ig != nullptr && ig_done != nullptr) {
    GemmParams g = input_grad_params(st->B, st->D, H, dZ, ldz, *ig);
    g.tile = pick_tile(g.M, g.N);
    const int64_t gx = ceil_div(g.N, g.tile), gy = ceil_div(g.M, g.tile), dw_blocks = (int64_t)grid.x * grid.y;
    if (dw_blocks + gx * gy <= 0x7fffffff) {
      if (st->dtype == RAD_BF16)
        dw_dx_kernel<bf16><<<(unsigned)(dw_blocks + gx * gy), 256, 0, s>>>(p, g, (int)dw_blocks, (int)gx);
      else
        dw_dx_kernel<float><<<(unsigned)(dw_blocks + gx * gy), 256, 0, s>>>(p, g, (int)dw_blocks, (int)gx);
      *ig_done = true;
      return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
    }
  }
  if (st->dtype == RAD_BF16)
    sparse_dw_kernel<bf16><<<grid, 256, 0, s>>>(p);
  else
    sparse_dw_kernel<float><<<grid, 256, 0, s>>>(p);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

int64_t column_sums_workspace(int64_t B, int64_t H) {
  return round_up(ceil_div(B, kColChunkRows) * H * 4, 256);
}

int column_sums(int dtype, int64_t B, int64_t H, const void* dZ, int64_t ldz, float* db, void* workspace,
                int64_t workspace_bytes, cudaStream_t s) {
  if (workspace == nullptr || workspace_bytes < column_sums_workspace(B, H)) return RAD_EWORKSPACE;
  const int64_t chunks = ceil_div(B, kColChunkRows);
  if (chunks <= kColSmallChunks) {
    count_launch();
    if (dtype == RAD_BF16)
      colsum_small_kernel<bf16><<<(unsigned)ceil_div(H, 256), 256, 0, s>>>(static_cast<const bf16*>(dZ), ldz, B, H, db);
    else
      colsum_small_kernel<float><<<(unsigned)ceil_div(H, 256), 256, 0, s>>>(static_cast<const float*>(dZ), ldz, B, H, db);
    return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
  }
  float* partial = static_cast<float*>(workspace);
  count_launch(2);
  if (H <= 64) {
    // no more slabs than the chunk count the workspace was sized for
    const int64_t slabs = std::min<int64_t>(chunks, 2 * 148);
    const int64_t rows_per_block = ceil_div(B, slabs), nblocks = ceil_div(B, rows_per_block);
    const int HP = H <= 16 ? 16 : H <= 32 ? 32 : 64;
    if (dtype == RAD_BF16)
      colsum_narrow_partial_kernel<bf16><<<(unsigned)nblocks, 256, 0, s>>>(static_cast<const bf16*>(dZ), ldz, B, (int)H, HP,
                                                                          rows_per_block, partial);
    else
      colsum_narrow_partial_kernel<float><<<(unsigned)nblocks, 256, 0, s>>>(static_cast<const float*>(dZ), ldz, B, (int)H, HP,
                                                                           rows_per_block, partial);
    colsum_final_kernel<<<1, 256, 0, s>>>(partial, nblocks, H, db);
    return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
  }
  dim3 grid((unsigned)ceil_div(H, 256), (unsigned)chunks);
  if (dtype == RAD_BF16 && H % 8 == 0 && ldz % 8 == 0 && ((uintptr_t)dZ & 15) == 0 && ((uintptr_t)partial & 15) == 0)
    colsum_partial_vec8_kernel<<<dim3((unsigned)ceil_div(H, 2048), (unsigned)chunks), 256, 0, s>>>(static_cast<const bf16*>(dZ), ldz, B,
                                                                                                   H, partial);
  else if (dtype == RAD_BF16)
    colsum_partial_kernel<bf16><<<grid, 256, 0, s>>>(static_cast<const bf16*>(dZ), ldz, B, H, partial);
  else
    colsum_partial_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(dZ), ldz, B, H, partial);
  colsum_final_kernel<<<(unsigned)ceil_div(H, 256), 256, 0, s>>>(partial, chunks, H, db);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad
