// 3x3 convolutions as implicit GEMMs on the tcgen05 tensor cores (paper, Fig. "Convnet activation sampling",
// Sec. 4.2: the conv input is what is sampled; the filter gradient is formed from the sample).  bf16 in,
// float32 accumulation in tensor memory, NHWC, zero padding 1, stride 1.
//
//   forward          M = output pixels (a tile of 128: 32 pooling windows, the four pixels of a window in four
//                    neighbouring accumulator rows), N = Cout (padded to 64), K = 9 Cin taken 64 at a time.  The A
//                    tile is the im2col patch matrix, written K-major into shared memory by the CTA's threads
//                    (no patch matrix ever exists in global memory); B is the filter block.  The epilogue adds the
//                    bias, applies ReLU, packs the four derivative bits of a window and writes the 2x2 average.
//   filter gradient  dW[(tap, ci), co] = sum over pixels of A_hat[pixel + tap, ci] dZ[pixel, co]: M = (tap, ci) in
//                    tiles of 128, N = Cout (padded to 64), K = pixels, split over CTAs; both operands are
//                    MN-major (the contraction index is the slow index of both tensors).  A_hat is the sampled
//                    conv input, expanded from its compact store into a zero-filled NHWC buffer of one layer
//                    (held only while this layer's gradient is formed).  Partial tiles are summed in split order.
//   input gradient   dX[pixel, ci] = sum over (tap, co) of dZ[pixel - tap, co] W[tap, ci, co] (the transposed
//                    convolution, exact): M = input pixels in raster order, N = Cin (padded to 64), K = 9 Cout taken
//                    64 at a time; the A tile is the patch matrix of dZ with the taps mirrored, K-major as in the
//                    forward pass; B is K-major too (for a tap and an input channel the output channels are
//                    contiguous in the filter tensor); the epilogue rounds and writes 64 bytes per row and chunk.
//
// One CTA (no cluster), eight warps: all of them write operand tiles with the 128-byte swizzle the tensor core
// expects (16-byte chunk c of row r lands at chunk c ^ (r & 7)), thread 0 issues tcgen05.mma.cta_group::1
// (M128 N64 K16), two shared-memory stages alternate, the 128 x 64 accumulator takes 64 columns of tensor
// memory.  Every wait is bounded; on expiry the CTA raises RAD_DEV_ETIMEOUT, frees its tensor memory and returns.
#include <algorithm>

#include "common.cuh"

namespace rad {
namespace {

constexpr int kCvM = 128, kCvN = 64, kCvK = 64;
constexpr int kCvThreads = 256;
constexpr int kCvABytes = kCvM * kCvK * 2;       // 16 KB either way round
constexpr int kCvBBytes = kCvK * kCvN * 2;       // 8 KB
constexpr int kCvStageBytes = kCvABytes + kCvBBytes;

struct ConvTcParams {
  int64_t B;
  int32_t H, W, Cin, Cout;
  const bf16* X;            // forward: conv input; filter gradient: A_hat (zero where dropped), both NHWC dense
  const bf16* Wt;           // 3 x 3 x Cin x Cout
  const float* bias;
  bf16* P;                  // pooled output; input gradient: dX, B x H x W x Cin
  uint32_t* relubits;
  const bf16* dZ;           // B x H x W x Cout
  float* partial;           // splits x (9 Cin) x Cout
  int32_t kblocks_per_split;
  int32_t* dev_status;
  uint64_t wait_limit_ns;
};

__device__ __forceinline__ uint32_t cv_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t cv_timer() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool cv_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// false: the wait ran out (or another one did): the caller stops issuing work
__device__ __forceinline__ bool cv_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint64_t limit_ns) {
  if (cv_try_wait(bar, parity)) return true;
  const uint64_t t0 = cv_timer();
  while (true) {
    for (int i = 0; i < 32; ++i) {
      if (cv_try_wait(bar, parity)) return true;
      __nanosleep(40);
    }
    if (*abort_flag != 0) return false;
    if (cv_timer() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}
// 128-byte-swizzle descriptor (K-major: SBO 1024; MN-major: LBO 8192 between 64-wide blocks, SBO 1024)
__device__ __forceinline__ uint64_t cv_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// D = f32, A = B = bf16, M = 128, N = 64, one CTA
__host__ __device__ constexpr uint32_t cv_idesc(bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(kCvN >> 3) << 17) | ((uint32_t)(kCvM >> 4) << 24);
}
__device__ __forceinline__ void cv_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void cv_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cv_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct CvCtl {
  uint64_t done[2];        // the MMAs that read stage s have retired
  uint32_t tmem_base;
  int abort_flag;
};

// 16 bytes of a dense NHWC tensor at pixel (b, y, x), channel c0 .. c0 + 7, zero outside the image
__device__ __forceinline__ uint4 cv_load_pixel(const bf16* T, int64_t b, int y, int x, int H, int W, int C, int c0) {
  if (y < 0 || y >= H || x < 0 || x >= W) return make_uint4(0u, 0u, 0u, 0u);
  return __ldg(reinterpret_cast<const uint4*>(T + ((b * H + y) * W + x) * C + c0));
}

// kCvFwd: forward tile `blockIdx.x` (128 output pixels); kCvDw: filter-gradient unit (m tile, split) = blockIdx;
// kCvDx: input-gradient tile `blockIdx.x` (128 input pixels in raster order)
enum { kCvFwd = 0, kCvDw = 1, kCvDx = 2 };
template <int kMode>
__global__ void __launch_bounds__(kCvThreads) conv_tc_kernel(const ConvTcParams p) {
  constexpr bool kDw = kMode == kCvDw, kDx = kMode == kCvDx;
  extern __shared__ uint8_t cv_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(cv_raw) + 1023) & ~(uintptr_t)1023);
  CvCtl* ctl = reinterpret_cast<CvCtl*>(smem + 2 * kCvStageBytes);
  volatile int* abort_flag = &ctl->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int H = p.H, W = p.W, Cin = p.Cin, Cout = p.Cout;
  const int64_t npix = p.B * H * W;
  const int ktaps = 9 * Cin;                          // rows of the filter matrix
  if (tid == 0) {
    for (int s = 0; s < 2; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(cv_smem(&ctl->done[s])), "r"(1u) : "memory");
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(cv_smem(&ctl->tmem_base)), "r"(64u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = ctl->tmem_base;

  // what this CTA contracts over
  const int mtile = kDw ? (int)blockIdx.x : 0, split = kDw ? (int)blockIdx.y : 0;
  const int64_t tile = kDw ? 0 : blockIdx.x;
  const int nkb = kDw ? p.kblocks_per_split : ((kDx ? 9 * Cout : ktaps) + kCvK - 1) / kCvK;
  const int64_t kb0 = kDw ? (int64_t)split * p.kblocks_per_split : 0;
  bool ok = true;
  for (int kb = 0; kb < nkb; ++kb) {
    const int s = kb & 1;
    uint8_t* sA = smem + s * kCvStageBytes;
    uint8_t* sB = sA + kCvABytes;
    // the MMAs of two K blocks ago have read this stage
    if (kb >= 2) ok = cv_wait(cv_smem(&ctl->done[s]), ((kb >> 1) - 1) & 1, abort_flag, p.wait_limit_ns);
    if (!__syncthreads_and(ok ? 1 : 0)) { ok = false; break; }
    if (kDx) {
      // A: K-major patch tile of dZ, row m = input pixel tile * 128 + m, k = (tap, co): the output pixel that
      // reached this input pixel through tap (ty, tx) lies at (y - ty + 1, x - tx + 1)
      for (int c = tid; c < kCvM * 8; c += kCvThreads) {
        const int m = c >> 3, cc = c & 7;
        const int k0 = kb * kCvK + cc * 8, tap = k0 / Cout, co0 = k0 - tap * Cout;
        const int64_t pix = tile * kCvM + m;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (tap < 9 && pix < npix) {
          const int x = (int)(pix % W), y = (int)((pix / W) % H);
          const int64_t b = pix / ((int64_t)W * H);
          v = cv_load_pixel(p.dZ, b, y - tap / 3 + 1, x - tap % 3 + 1, H, W, Cout, co0);
        }
        *reinterpret_cast<uint4*>(sA + m * 128 + ((cc ^ (m & 7)) << 4)) = v;
      }
      // B: K-major, row n = input channel, k = (tap, co): W[tap, n, co0 .. co0 + 7] is contiguous
      for (int c = tid; c < kCvN * 8; c += kCvThreads) {
        const int n = c >> 3, cc = c & 7;
        const int k0 = kb * kCvK + cc * 8, tap = k0 / Cout, co0 = k0 - tap * Cout;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (tap < 9 && n < Cin) v = __ldg(reinterpret_cast<const uint4*>(p.Wt + ((int64_t)tap * Cin + n) * Cout + co0));
        *reinterpret_cast<uint4*>(sB + n * 128 + ((cc ^ (n & 7)) << 4)) = v;
      }
    } else if (!kDw) {
      // A: K-major patch tile, row m = window (tile * 32 + m / 4), pixel m % 4 of it; 8 chunks of 8 k per row
      for (int c = tid; c < kCvM * 8; c += kCvThreads) {
        const int m = c >> 3, cc = c & 7;
        const int k0 = kb * kCvK + cc * 8, tap = k0 / Cin, ci0 = k0 - tap * Cin;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        const int64_t q = tile * 32 + (m >> 2);
        if (tap < 9 && q < npix / 4) {
          const int Wp = W >> 1, Hp = H >> 1;
          const int xp = (int)(q % Wp), yp = (int)((q / Wp) % Hp);
          const int64_t b = q / ((int64_t)Wp * Hp);
          const int y = 2 * yp + ((m >> 1) & 1), x = 2 * xp + (m & 1);
          v = cv_load_pixel(p.X, b, y + tap / 3 - 1, x + tap % 3 - 1, H, W, Cin, ci0);
        }
        *reinterpret_cast<uint4*>(sA + m * 128 + ((cc ^ (m & 7)) << 4)) = v;
      }
      // B: filter rows k (MN-major: Cout contiguous), 8 chunks of 8 channels per row
      for (int c = tid; c < kCvK * 8; c += kCvThreads) {
        const int k = c >> 3, cc = c & 7;
        const int kg = kb * kCvK + k;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (kg < ktaps && cc * 8 < Cout) v = __ldg(reinterpret_cast<const uint4*>(p.Wt + (int64_t)kg * Cout + cc * 8));
        *reinterpret_cast<uint4*>(sB + k * 128 + ((cc ^ (k & 7)) << 4)) = v;
      }
    } else {
      // A: MN-major, row k = pixel, 16 chunks of 8 (tap, ci) indices in two blocks of 64; B: dZ of the pixel
      for (int c = tid; c < kCvK * 16; c += kCvThreads) {
        const int k = c >> 4, cc = c & 15;
        const int m0 = mtile * kCvM + cc * 8, tap = m0 / Cin, ci0 = m0 - tap * Cin;
        const int64_t pix = (kb0 + kb) * kCvK + k;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (tap < 9 && pix < npix) {
          const int x = (int)(pix % W), y = (int)((pix / W) % H);
          const int64_t b = pix / ((int64_t)W * H);
          v = cv_load_pixel(p.X, b, y + tap / 3 - 1, x + tap % 3 - 1, H, W, Cin, ci0);
        }
        *reinterpret_cast<uint4*>(sA + (cc >> 3) * 8192 + k * 128 + (((cc & 7) ^ (k & 7)) << 4)) = v;
      }
      for (int c = tid; c < kCvK * 8; c += kCvThreads) {
        const int k = c >> 3, cc = c & 7;
        const int64_t pix = (kb0 + kb) * kCvK + k;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (pix < npix && cc * 8 < Cout) v = __ldg(reinterpret_cast<const uint4*>(p.dZ + pix * Cout + cc * 8));
        *reinterpret_cast<uint4*>(sB + k * 128 + ((cc ^ (k & 7)) << 4)) = v;
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      constexpr uint32_t idesc = cv_idesc(kDw, !kDx);
      const uint32_t a0 = cv_smem(sA), b0 = cv_smem(sB);
#pragma unroll
      for (int k = 0; k < kCvK / 16; ++k) {
        const uint64_t adesc = kDw ? cv_desc(a0 + k * 2048, 8192, 1024) : cv_desc(a0 + k * 32, 16, 1024);
        const uint64_t bdesc = kDx ? cv_desc(b0 + k * 32, 16, 1024) : cv_desc(b0 + k * 2048, 8192, 1024);
        cv_mma(tmem, adesc, bdesc, idesc, (kb > 0 || k > 0) ? 1u : 0u);
      }
      cv_commit(cv_smem(&ctl->done[s]));
    }
  }
  // the last commit covers every MMA before it
  if (ok && nkb > 0) ok = cv_wait(cv_smem(&ctl->done[(nkb - 1) & 1]), ((nkb - 1) >> 1) & 1, abort_flag, p.wait_limit_ns);
  ok = __syncthreads_and(ok ? 1 : 0) != 0;
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (ok) {
    const int q = warp & 3, chunk = warp >> 2;       // accumulator rows 32 q .. 32 q + 31, columns 32 chunk .. + 31
    const int m = q * 32 + lane;
    uint32_t r[32];
    cv_tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(chunk * 32), r);
    if (kDx) {
      // row m = input pixel, columns = input channels: rounded once, 64 bytes per row and chunk
      const int64_t pix = tile * kCvM + m;
      if (pix < npix) {
        bf16* dst = p.P + pix * Cin + chunk * 32;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          if (chunk * 32 + j < Cin) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[j + 2 * e]), __uint_as_float(r[j + 2 * e + 1]));
              w[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    } else if (!kDw) {
      // rows 4 w .. 4 w + 3 are the 2 x 2 window w: bias, ReLU, derivative bits, rounded average
      const int64_t win = tile * 32 + (m >> 2);
      const bool win_ok = win < npix / 4;
      const int quad = lane & ~3;
      uint32_t word = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const int co = chunk * 32 + j;
        float a = 0.0f;
        if (co < Cout) {
          const float z = __uint_as_float(r[j]) + (p.bias != nullptr ? __ldg(p.bias + co) : 0.0f);
          a = __bfloat162float(__float2bfloat16_rn(fmaxf(z, 0.0f)));       // the activation as the device would hold it
        }
        const uint32_t pos = __ballot_sync(0xffffffffu, a > 0.0f);
        const float a0 = __shfl_sync(0xffffffffu, a, quad), a1 = __shfl_sync(0xffffffffu, a, quad + 1);
        const float a2 = __shfl_sync(0xffffffffu, a, quad + 2), a3 = __shfl_sync(0xffffffffu, a, quad + 3);
        word |= ((pos >> quad) & 0xfu) << (4 * (j & 7));
        if ((lane & 3) == 0 && win_ok && co < Cout) {
          p.P[win * Cout + co] = __float2bfloat16_rn(0.25f * (((a0 + a1) + a2) + a3));
          if ((j & 7) == 7) p.relubits[(win * Cout + co) >> 3] = word;      // eight channels make one word
        }
        if ((j & 7) == 7) word = 0;
      }
    } else {
      const int mg = mtile * kCvM + m;
      if (mg < ktaps) {
        float* dst = p.partial + ((int64_t)split * ktaps + mg) * Cout + chunk * 32;
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          if (chunk * 32 + j < Cout)
            *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                              __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0 && ctl->abort_flag != 0) raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(64u) : "memory");
  }
}

// dW[i] = sum over splits of partial[s][i], in split order
__global__ void __launch_bounds__(256) conv_tc_reduce_kernel(const float* partial, int splits, int64_t n, float* out) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float acc = 0.0f;
  for (int s = 0; s < splits; ++s) acc += partial[(int64_t)s * n + i];
  out[i] = acc;
}

// A_hat (B x D, zero where dropped) from a compact store: the buffer is cleared first, then the kept values
// are dropped in place.  different-sample: a thread per keep-bit word; same-sample: a thread per kept entry.
__global__ void __launch_bounds__(256) densify_different_kernel(const bf16* values, const uint32_t* keepbits, const uint32_t* offsets,
                                                                int64_t B, int64_t D, int32_t ncb, int64_t capacity, bf16* out) {
  const int64_t nwords = ((B + kTileRows - 1) / kTileRows) * ncb * kBitWords;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nwords; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t tile = i / kBitWords;
    const int t = (int)(i - tile * kBitWords), r = t >> 2, w = t & 3;
    const uint32_t* tw = keepbits + tile * kTileWords;
    uint32_t word = tw[t];
    if (word == 0) continue;
    int64_t pos = (int64_t)offsets[tile] + ((tw[kBitWords + (r >> 1)] >> (16 * (r & 1))) & 0xffffu);
    for (int q = 0; q < w; ++q) pos += __popc(tw[r * 4 + q]);
    const int64_t row = (tile / ncb) * kTileRows + r, col0 = (tile % ncb) * kTileCols + 32 * w;
    while (word != 0) {
      const int b = __ffs(word) - 1;
      word &= word - 1;
      if (row < B && col0 + b < D && pos < capacity) out[row * D + col0 + b] = values[pos];
      ++pos;
    }
  }
}
__global__ void __launch_bounds__(256) densify_same_kernel(const bf16* values, const uint32_t* idx, const int64_t* nnz, int64_t B,
                                                           int64_t D, int64_t ld, bf16* out) {
  const int64_t k = min(nnz[0], ld);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < B * k; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = i / k, j = i - b * k;
    const uint32_t col = idx[j];
    if (col < (uint32_t)D) out[b * D + col] = values[b * ld + j];
  }
}

constexpr size_t kCvSmem = 2 * kCvStageBytes + sizeof(CvCtl) + 1024;
int g_conv_kernel = RAD_CONV_KERNEL_AUTO;

}  // namespace

// Shapes the tensor-core kernels take: bf16, Cin 16, 32 or 64 (a 64-deep K block is a whole number of taps),
// Cout a multiple of 8 up to 64, even H and W.
bool conv_tc_ok(int dtype, int H, int W, int Cin, int Cout, const void* X, const void* Wt) {
  if (g_conv_kernel == RAD_CONV_KERNEL_SIMT) return false;
  return dtype == RAD_BF16 && (Cin == 16 || Cin == 32 || Cin == 64) && Cout % 8 == 0 && Cout >= 8 && Cout <= kCvN && H % 2 == 0 &&
         W % 2 == 0 && ((uintptr_t)X & 15) == 0 && ((uintptr_t)Wt & 15) == 0;
}

int conv_tc_forward_pool(int64_t B, int H, int W, int Cin, int Cout, const void* X, const void* Wt, const float* bias, void* P,
                         uint32_t* relubits, int32_t* dev_status, cudaStream_t st) {
  ConvTcParams p = {};
  p.B = B; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout;
  p.X = static_cast<const bf16*>(X); p.Wt = static_cast<const bf16*>(Wt); p.bias = bias;
  p.P = static_cast<bf16*>(P); p.relubits = relubits; p.dev_status = dev_status; p.wait_limit_ns = wait_limit_ns();
  RAD_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<kCvFwd>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCvSmem));
  const int64_t windows = B * (H / 2) * (W / 2);
  count_launch();
  conv_tc_kernel<kCvFwd><<<(unsigned)ceil_div(windows, 32), kCvThreads, kCvSmem, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// Shapes the input-gradient kernel takes: as above with the channel counts in each other's roles (K runs over
// (tap, co) in chunks of eight output channels, N over the input channels).
bool conv_tc_dx_ok(int dtype, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, const void* dX) {
  (void)H; (void)W;
  if (g_conv_kernel == RAD_CONV_KERNEL_SIMT) return false;
  return dtype == RAD_BF16 && (Cout == 16 || Cout == 32 || Cout == 64) && Cin % 8 == 0 && Cin >= 8 && Cin <= kCvN &&
         ((uintptr_t)dZ & 15) == 0 && ((uintptr_t)Wt & 15) == 0 && ((uintptr_t)dX & 15) == 0;
}

int conv_tc_input_grad(int64_t B, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, void* dX, int32_t* dev_status,
                       cudaStream_t st) {
  ConvTcParams p = {};
  p.B = B; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout;
  p.dZ = static_cast<const bf16*>(dZ); p.Wt = static_cast<const bf16*>(Wt); p.P = static_cast<bf16*>(dX);
  p.dev_status = dev_status; p.wait_limit_ns = wait_limit_ns();
  RAD_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<kCvDx>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCvSmem));
  count_launch();
  conv_tc_kernel<kCvDx><<<(unsigned)ceil_div(B * H * W, kCvM), kCvThreads, kCvSmem, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// K blocks of 64 pixels per CTA of the filter-gradient kernel, and the splits that follow from it
static int conv_tc_splits(int64_t npix, int* kblocks_per_split) {
  const int64_t kblocks = ceil_div(npix, kCvK);
  int64_t per = std::max<int64_t>(4, ceil_div(kblocks, 96));      // about one wave of CTAs per M tile pair
  *kblocks_per_split = (int)per;
  return (int)ceil_div(kblocks, per);
}

int64_t conv_tc_weight_grad_workspace(int64_t B, int H, int W, int Cin, int Cout) {
  int per = 0;
  const int splits = conv_tc_splits(B * H * W, &per);
  return round_up(B * H * W * Cin * 2, 256) + round_up((int64_t)splits * 9 * Cin * Cout * 4, 256);
}

int conv_tc_weight_grad(const rad_store* store, int H, int W, int Cin, int Cout, const void* dZ, float* dW, void* workspace,
                        int64_t workspace_bytes, int32_t* dev_status, cudaStream_t st) {
  const int64_t B = store->B, D = store->D;
  if (workspace == nullptr || workspace_bytes < conv_tc_weight_grad_workspace(B, H, W, Cin, Cout)) return RAD_EWORKSPACE;
  bf16* dense = static_cast<bf16*>(workspace);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + round_up(B * D * 2, 256));
  RAD_CUDA_TRY(cudaMemsetAsync(dense, 0, (size_t)(B * D * 2), st));
  count_launch();
  if (store->variant == RAD_SAME_SAMPLE) {
    densify_same_kernel<<<(unsigned)std::min<int64_t>(ceil_div(B * store->values_ld, 256), 148 * 16), 256, 0, st>>>(
        static_cast<const bf16*>(store->values), store->offsets, store->nnz, B, D, store->values_ld, dense);
  } else {
    const int32_t ncb = (int32_t)ceil_div(D, kTileCols);
    const int64_t nwords = ceil_div(B, kTileRows) * ncb * kBitWords;
    densify_different_kernel<<<(unsigned)std::min<int64_t>(ceil_div(nwords, 256), 148 * 16), 256, 0, st>>>(
        static_cast<const bf16*>(store->values), store->keepbits, store->offsets, B, D, ncb, store->values_capacity, dense);
  }
  ConvTcParams p = {};
  p.B = B; p.H = H; p.W = W; p.Cin = Cin; p.Cout = Cout;
  p.X = dense; p.dZ = static_cast<const bf16*>(dZ); p.partial = partial; p.dev_status = dev_status;
  p.wait_limit_ns = wait_limit_ns();
  const int splits = conv_tc_splits(B * H * W, &p.kblocks_per_split);
  RAD_CUDA_TRY(cudaFuncSetAttribute(conv_tc_kernel<kCvDw>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCvSmem));
  count_launch(2);
  conv_tc_kernel<kCvDw><<<dim3((unsigned)ceil_div(9 * Cin, kCvM), (unsigned)splits), kCvThreads, kCvSmem, st>>>(p);
  const int64_t n = (int64_t)9 * Cin * Cout;
  conv_tc_reduce_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, st>>>(partial, splits, n, dW);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad

extern "C" int rad_set_conv_kernel(int32_t which) {
  if (which != RAD_CONV_KERNEL_AUTO && which != RAD_CONV_KERNEL_SIMT && which != RAD_CONV_KERNEL_TENSOR) return RAD_EINVAL;
  const int prev = rad::g_conv_kernel;
  rad::g_conv_kernel = which;
  return prev;
}
