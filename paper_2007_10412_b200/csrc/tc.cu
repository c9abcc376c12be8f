// tcgen05 GEMM engine (bf16 in, float32 accumulate in tensor memory) for the four contractions of
// a RAD step on large aligned layers:
//   forward      Z = A W + b                 (exact; Sec. 3: the forward pass is the original graph)
//   input grad   dA = dZ W^T                 (exact; Sec. 4.2)
//   dW, same     dW[idx, :] = A_c^T dZ       (column-compacted dense GEMM; Sec. 4.3 "same sample")
//   dW, diff.    dW = A_hat^T dZ             (A_hat tiles rebuilt in shared memory from keep bits
//                                             and packed values; Sec. 4.2 / 4.3 "different sample")
//
// Every kernel here runs on SM pairs: a cluster of two CTAs, one per SM, persistent, with one
// thread of the even CTA issuing tcgen05.mma.cta_group::2 on operands that both CTAs stage in their
// own shared memory (TMA, 128-byte swizzle, no multicast) through an mbarrier ring.
//   dense kernels    256 x 256 tile per pair; each CTA keeps two alternating 128 x 256 float32
//                    accumulators in tensor memory, so the epilogue of a tile (bias, activation,
//                    ReLU bits, GELU', stores) runs under the MMAs of the next one.
//   sparse-A kernel  512 x 256 tile per pair; sixteen "expander" warps per CTA write the A_hat
//                    tile of each K block into shared memory instead of TMA.
// Long dW contractions can be split along K; partial tiles are summed in split order by a second
// kernel, so results are reproducible.
// Every mbarrier wait is bounded: on expiry both CTAs of the pair raise their abort flags, all
// roles leave their loops, the pair meets at a cluster barrier, tensor memory is released, the
// kernel returns and the launch reports RAD_DEV_ETIMEOUT.
#include <cuda.h>

#include <algorithm>
#include <cmath>

#include "common.cuh"

namespace rad {
namespace {

constexpr int BM = 256, BN = 256, BK = 64;
constexpr int kHalfM = 128;
constexpr int kNumSMsDefault = 148;
constexpr int kMaxSplits = 16;
constexpr int kRasterGroup = 16;               // m-tiles per raster group (16 x 4 MB of A panels stay in L2 beside the B panels in flight)

enum AKind { kAK = 0, kAMN = 1, kASparse = 2 };
enum BKind { kBK_ = 0, kBMN = 1 };
enum EpiKind { kFwd = 0, kDx = 1, kDw = 2, kDwT = 3 };

struct TcParams {
  int64_t M, N, K;
  const int64_t* N_dev;      // same-sample dW: N = number of kept columns, read on the device
  const uint32_t* keep_cols; // same-sample dW: bit d set = column d of the layer input was kept
  int32_t splits;            // K splits (1: epilogue writes final results)
  int32_t num_stages;
  int32_t comp_depth;        // sparse A: depth of the ring of compressed (index + values) buffers
  // sparse A (different-sample store)
  const bf16* values; const uint32_t* keepbits; const uint32_t* offsets;
  int64_t values_capacity; int32_t ncb; int32_t comp_cap;   // comp_cap: value bytes per half-stage
  // forward epilogue
  const float* bias; int32_t act;
  bf16* out_act; int64_t ld_act; float* out_z; int64_t ld_z; bf16* out_zlow; int64_t ld_zlow;
  uint32_t* relubits; int64_t w32;
  // forward epilogue that also fills the next layer's store (index part already in place)
  bf16* st_values; const uint32_t* st_keepbits; const uint32_t* st_offsets; int64_t st_capacity; int32_t st_ncb; float st_scale;
  // input-grad epilogue
  const uint32_t* relubits_prev; const bf16* z_prev; int64_t ld_zprev; bf16* out_dx; int64_t ld_dx;
  // dW epilogue
  float* out_dw; int64_t ld_dw; int64_t dw_rows; const uint32_t* row_idx; float* partial; int64_t partial_rows;
  int32_t* dev_status;
  uint64_t wait_limit_ns;    // every device-side wait of the launch gives up after this long
};

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major: rows of 64 elements (128 B), eight
// rows form a 1024 B swizzle atom, SBO = 1024 B between atoms along M/N.  MN-major: rows of 64
// M/N elements (one per K index), SBO = 1024 B between groups of eight K rows, LBO = distance to
// the next 64 M/N elements.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// ---- work decomposition ---------------------------------------------------------------------------
struct Unit {
  int64_t m0, n0;
  int32_t kb0, kb1;    // K blocks [kb0, kb1)
  int32_t split;
};

struct Schedule {
  int64_t M, m_tiles, n_tiles, ntiles, units;
  int32_t kblocks, splits, bm, bn;
  __device__ Schedule(int64_t M_, int64_t N_, int64_t K_, int32_t splits_, int32_t bm_ = BM, int32_t bn_ = BN) {
    M = M_;
    bm = bm_;
    bn = bn_;
    m_tiles = (M + bm - 1) / bm;
    n_tiles = (N_ + bn - 1) / bn;
    ntiles = m_tiles * n_tiles;
    kblocks = (int32_t)((K_ + BK - 1) / BK);
    splits = splits_;
    units = ntiles * splits;
  }
  // split-major order: CTAs of one wave work on the same K range, so operand panels shared by
  // tiles of a row or column of the grid are read from L2 at about the same time.
  __device__ Unit unit(int64_t u) const {
    Unit w;
    const int64_t s = u / ntiles, t = u % ntiles;
    const int64_t per_group = kRasterGroup * n_tiles;
    const int64_t g = t / per_group, r = t % per_group;
    const int64_t first_m = g * kRasterGroup;
    const int64_t gm = min((int64_t)kRasterGroup, m_tiles - first_m);
    w.m0 = (first_m + r % gm) * bm;
    w.n0 = (r / gm) * bn;
    w.split = (int32_t)s;
    w.kb0 = (int32_t)(s * kblocks / splits);
    w.kb1 = (int32_t)((s + 1) * kblocks / splits);
    return w;
  }
};

// ---- epilogue of one 32-column chunk of one accumulator row ------------------------------------------
// r: the 32 float32 accumulators of row m, columns n .. n+31 (as bit patterns).
template <int EPI>
__device__ __forceinline__ void epilogue_chunk(const TcParams& p, uint32_t (&r)[32], int64_t m, int64_t n, bool row_ok,
                                               int32_t split) {
  const int nvalid = (int)min((int64_t)32, p.N - n);      // multiple of 8
  if (EPI == kFwd) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
    if (p.bias != nullptr) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        if (j < nvalid) {
          const float4 b4 = __ldg(reinterpret_cast<const float4*>(p.bias + n + j));
          v[j] += b4.x; v[j + 1] += b4.y; v[j + 2] += b4.z; v[j + 3] += b4.w;
        }
      }
    }
    if (row_ok) {
      if (p.out_z != nullptr) {
        float4* dst = reinterpret_cast<float4*>(p.out_z + m * p.ld_z + n);
#pragma unroll
        for (int j = 0; j < 32; j += 4)
          if (j < nvalid) dst[j >> 2] = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      }
      if (p.out_zlow != nullptr) {
        uint4* dst = reinterpret_cast<uint4*>(p.out_zlow + m * p.ld_zlow + n);
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          if (j < nvalid) {
            __nv_bfloat162 a = __floats2bfloat162_rn(v[j], v[j + 1]), b = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
            __nv_bfloat162 c = __floats2bfloat162_rn(v[j + 4], v[j + 5]), d = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
            dst[j >> 3] = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                                     *reinterpret_cast<uint32_t*>(&c), *reinterpret_cast<uint32_t*>(&d));
          }
        }
      }
      if (p.out_act != nullptr) {
        uint32_t bits = 0;
        uint32_t ab[16];                          // the rounded activations, two to a word
        uint4* dst = reinterpret_cast<uint4*>(p.out_act + m * p.ld_act + n);
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
#pragma unroll
          for (int e = 0; e < 8; e += 2) ab[(j + e) >> 1] = 0u;
          if (j < nvalid) {
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              float a0 = v[j + e], a1 = v[j + e + 1];
              if (p.act == RAD_ACT_RELU) { a0 = fmaxf(a0, 0.0f); a1 = fmaxf(a1, 0.0f); }
              else if (p.act == RAD_ACT_GELU) { a0 = gelu_f(a0); a1 = gelu_f(a1); }
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(a0, a1);
              ab[(j + e) >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
              // the bit is taken from the rounded activation, the tensor the backward sees
              bits |= (__bfloat162float(h2.x) > 0.0f ? 1u : 0u) << (j + e);
              bits |= (__bfloat162float(h2.y) > 0.0f ? 1u : 0u) << (j + e + 1);
            }
            dst[j >> 3] = make_uint4(ab[j >> 1], ab[(j >> 1) + 1], ab[(j >> 1) + 2], ab[(j >> 1) + 3]);
          }
        }
        if (p.relubits != nullptr) p.relubits[m * p.w32 + (n >> 5)] = bits;
        if (p.st_values != nullptr) {
          // This row's 32 activations are one keep-bit word of the next layer's store (Sec. 4.2: the
          // layer input is what is sampled), whose index part (drawn from the key alone) is in place:
          // tile offset + row offset + kept entries of the row's earlier words say where they go.
          const int64_t tile = (m >> 6) * p.st_ncb + (n >> 7);
          const int rr = (int)(m & 63), wq = (int)((n >> 5) & 3);
          const uint32_t* tw = p.st_keepbits + tile * kTileWords;
          const uint4 rowbits = __ldg(reinterpret_cast<const uint4*>(tw + rr * 4));
          const uint32_t word = wq == 0 ? rowbits.x : wq == 1 ? rowbits.y : wq == 2 ? rowbits.z : rowbits.w;
          const uint32_t first = __ldg(p.st_offsets + tile);
          uint64_t pos = (uint64_t)first + __ldg(reinterpret_cast<const unsigned short*>(tw + kBitWords) + rr);
          if (wq > 0) pos += __popc(rowbits.x);
          if (wq > 1) pos += __popc(rowbits.y);
          if (wq > 2) pos += __popc(rowbits.z);
          const uint64_t cap = (uint64_t)p.st_capacity;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if ((word >> j) & 1u) {
              const float a = __uint_as_float((j & 1) ? (ab[j >> 1] & 0xffff0000u) : (ab[j >> 1] << 16));
              if (pos < cap) p.st_values[pos] = __float2bfloat16_rn(__fmul_rn(a, p.st_scale));
              ++pos;
            }
          }
          if (rr == 0 && wq == 0) {
            // zeros between the tile's last value and its padded end
            const uint4 last = __ldg(reinterpret_cast<const uint4*>(tw + 63 * 4));
            const uint32_t exact = __ldg(reinterpret_cast<const unsigned short*>(tw + kBitWords) + 63) + __popc(last.x) +
                                   __popc(last.y) + __popc(last.z) + __popc(last.w);
            const uint64_t end = min((uint64_t)__ldg(p.st_offsets + tile + 1), cap);
            for (uint64_t q = (uint64_t)first + exact; q < end; ++q) p.st_values[q] = __float2bfloat16_rn(0.0f);
          }
        }
      }
    }
  } else if (EPI == kDx) {
    if (row_ok) {
      uint32_t bits = 0xffffffffu;
      if (p.relubits_prev != nullptr) bits = __ldg(p.relubits_prev + m * ((p.N + 31) / 32) + (n >> 5));
      uint4* dst = reinterpret_cast<uint4*>(p.out_dx + m * p.ld_dx + n);
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        if (j < nvalid) {
          float g[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) g[e] = ((bits >> (j + e)) & 1u) ? __uint_as_float(r[j + e]) : 0.0f;
          if (p.z_prev != nullptr) {
            const uint4 zq = __ldg(reinterpret_cast<const uint4*>(p.z_prev + m * p.ld_zprev + n + j));
            const uint32_t zw[4] = {zq.x, zq.y, zq.z, zq.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float z = __uint_as_float((e & 1) ? (zw[e >> 1] & 0xffff0000u) : (zw[e >> 1] << 16));
              g[e] *= gelu_grad_f(z);
            }
          }
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(g[e], g[e + 1]);
            pk[e >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          dst[j >> 3] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
  } else {
    if (row_ok) {
      float* dst;
      if (p.splits > 1) {
        dst = p.partial + ((int64_t)split * p.partial_rows + m) * p.N + n;
      } else {
        const int64_t row = (p.row_idx != nullptr) ? (int64_t)__ldg(p.row_idx + m) : m;
        if (row >= p.dw_rows) { raise_status(p.dev_status, RAD_DEV_EINTERNAL); return; }
        dst = p.out_dw + row * p.ld_dw + n;
      }
      float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        if (j < nvalid)
          d4[j >> 2] = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                   __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
    }
  }
}

// Same-sample dW, transposed tile: the accumulator row is output column h of dW, the accumulator column is
// kept column j; r holds dW[idx[n + jj], h] for jj < 32.  For a fixed jj the 32 lanes of a warp write 32
// consecutive floats of one row of dW (or of the split's partial block, row n + jj).
__device__ __forceinline__ void epilogue_chunk_dwt(const TcParams& p, const uint32_t (&r)[32], int64_t h, int64_t n,
                                                   int nvalid, bool row_ok, int32_t split) {
  if (!row_ok) return;
  if (p.splits > 1) {
    float* dst = p.partial + ((int64_t)split * p.partial_rows + n) * p.M + h;
#pragma unroll
    for (int jj = 0; jj < 32; ++jj)
      if (jj < nvalid) dst[(int64_t)jj * p.M] = __uint_as_float(r[jj]);
  } else {
#pragma unroll
    for (int jj = 0; jj < 32; ++jj) {
      if (jj < nvalid) {
        const int64_t row = (int64_t)__ldg(p.row_idx + n + jj);
        if (row < p.dw_rows) p.out_dw[row * p.ld_dw + h] = __uint_as_float(r[jj]);
        else raise_status(p.dev_status, RAD_DEV_EINTERNAL);
      }
    }
  }
}

// ---- shared memory layout -------------------------------------------------------------------------
constexpr int kIndexBytes = kTileWords * 4;   // keep bits + row offsets of one store tile (1152 B)
constexpr int kExpanderWarps = 16;            // one thread per keep-bit word of the two halves
constexpr int kFirstExpanderWarp = 7;        // warp 6 feeds the compressed ring
// ---- expansion of one keep-bit word into the A_hat tile -------------------------------------------
// sA: the stage's A tile (four 8 KB blocks of 64 columns, 128-byte rows per K index, 128-byte
// swizzle); sC: keep bits, row offsets and packed values of store tile h of this K block; the thread
// owns row r, columns 32 wq .. 32 wq + 31 of that store tile.  limit: staged values per tile.
__device__ __forceinline__ void expand_word(uint8_t* sA, const uint8_t* sC, int h, int r, int wq, uint32_t limit) {
  const uint32_t* bits = reinterpret_cast<const uint32_t*>(sC);
  const unsigned short* rowoff = reinterpret_cast<const unsigned short*>(sC + kBitWords * 4);
  const unsigned short* vals = reinterpret_cast<const unsigned short*>(sC + kIndexBytes);
  const uint4 rowbits = *reinterpret_cast<const uint4*>(bits + r * 4);
  const uint32_t word = wq == 0 ? rowbits.x : wq == 1 ? rowbits.y : wq == 2 ? rowbits.z : rowbits.w;
  uint32_t pos = rowoff[r];
  if (wq > 0) pos += __popc(rowbits.x);
  if (wq > 1) pos += __popc(rowbits.y);
  if (wq > 2) pos += __popc(rowbits.z);
  uint8_t* rowp = sA + h * 16384 + (wq >> 1) * 8192 + r * 128;
  const int j0 = (wq & 1) * 4;
  const uint32_t cnt = __popc(word);
  // one path per warp: the dense form is right for any word
  if (__all_sync(0xffffffffu, cnt + (pos & 3u) <= 12u && cnt <= 10u)) {
    // sparse word: zero this thread's 32 columns, then drop the kept values in place.  The
    // values are consecutive from `pos`: three aligned 8-byte loads cover them (a word whose
    // values would pass the end of the staged tile places nothing: the producer has flagged it).
    // Byte address of column c of this word in the swizzled row: base ^ (c << 1), because the
    // 16-byte chunk index (j0 + (c >> 3)) ^ (r & 7) equals (c >> 3) ^ (j0 ^ (r & 7)) for j0 in {0, 4}
    // and rows are 128-byte aligned.
    const uint32_t base = smem_u32(rowp) ^ ((uint32_t)(j0 ^ (r & 7)) << 4);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
      asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base ^ (uint32_t)(jj << 4)), "r"(0u) : "memory");
    const uint32_t rest = (pos + cnt <= limit) ? word : 0u;
    const uint32_t e0 = pos & 3u;
    const uint2* win = reinterpret_cast<const uint2*>(vals + (min(pos, limit) & ~3u));   // stays inside the ring
    const uint2 q0 = win[0], q1 = win[1];
    uint2 q2 = make_uint2(0u, 0u);
    if (e0 + cnt > 8u) q2 = win[2];
    // bring the first kept value to bit 0 of s0: drop whole words, then a half word
    const bool drop = (e0 & 2u) != 0u;
    const uint32_t w0 = drop ? q0.y : q0.x, w1 = drop ? q1.x : q0.y, w2 = drop ? q1.y : q1.x;
    const uint32_t w3 = drop ? q2.x : q1.y, w4 = drop ? q2.y : q2.x, w5 = drop ? 0u : q2.y;
    const uint32_t sh = (e0 & 1u) << 4;
    const uint32_t sv[5] = {__funnelshift_r(w0, w1, sh), __funnelshift_r(w1, w2, sh), __funnelshift_r(w2, w3, sh),
                            __funnelshift_r(w3, w4, sh), __funnelshift_r(w4, w5, sh)};
    // every lane runs the warp's longest word; a lane that has run out stores nothing.  The word is
    // bit-reversed so that the next kept column is a leading-zero count away.
    const uint32_t steps = __reduce_max_sync(0xffffffffu, rest != 0u ? cnt : 0u);
    uint32_t rw = __brev(rest);
#pragma unroll
    for (int i = 0; i < 10; ++i) {
      if ((uint32_t)i >= steps) break;                  // warp-uniform
      const uint32_t c = (uint32_t)__clz((int)rw);      // 32 once the word is used up
      const uint32_t v = sv[i >> 1] >> (16 * (i & 1));
      asm volatile("{\n\t.reg .pred k;\n\tsetp.ne.u32 k, %2, 0;\n\t@k st.shared.b16 [%0], %1;\n\t}"
                   ::"r"(base ^ (c << 1)), "h"((unsigned short)v), "r"(rw) : "memory");
      rw &= ~(0x80000000u >> (c & 31u));
    }
  } else {
    // dense word: every column's value position follows from a popcount of the bits below
    // it, so the 32 loads are independent; each 16-byte chunk is written once
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 8; e += 2) {
        const int b0 = jj * 8 + e;
        const uint32_t p0 = pos + __popc(word & ((1u << b0) - 1u));
        const uint32_t p1 = pos + __popc(word & ((2u << b0) - 1u));
        const uint32_t v0 = ((word >> b0) & 1u) && p0 < limit ? vals[p0] : 0u;
        const uint32_t v1 = ((word >> (b0 + 1)) & 1u) && p1 < limit ? vals[p1] : 0u;
        pk[e >> 1] = v0 | (v1 << 16);
      }
      *reinterpret_cast<uint4*>(rowp + (((j0 + jj) ^ (r & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
  }
}

// ---- two-CTA engine (dense operands) -----------------------------------------------------------------
// A cluster of two CTAs (one SM pair) owns a 256 x 256 output tile.  Each CTA stages 128 rows of
// the A tile and 128 rows (N) of the B tile per K block and keeps 128 accumulator rows in its own
// tensor memory; one thread of the even CTA issues tcgen05.mma.cta_group::2, which reads both
// CTAs' shared memory.  Against the one-CTA tile this halves the operand bytes each SM's shared
// memory has to deliver per MMA, and a 128 x 256 accumulator takes 256 tensor-memory columns, so
// two of them alternate: the epilogue of one tile runs under the MMAs of the next.
// Barriers: full[s] (even CTA; its producer arrives once with the byte count of both CTAs, and
// both CTAs' TMA complete on it: the odd CTA reloads a stage only after the commit that follows the
// even CTA's wait on the previous phase, so its bytes never reach an older phase), empty[s] and tmem_full[b] (one per CTA, signalled by the MMA thread's commit to
// both CTAs), tmem_empty[b] (even CTA; every epilogue warp of the pair arrives).
constexpr int kStage2Bytes = 2 * 128 * BK * 2;   // 16 KB of A + 16 KB of B per CTA and stage
constexpr int kStages2 = 6;
constexpr int kEpiWarps2 = 8;
constexpr int kThreads2 = 32 * (2 + kEpiWarps2);

struct SmemCtl2 {
  uint64_t full[kStages2], empty[kStages2], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {   // shared::cluster address
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrival on a barrier of either CTA of the pair (default semantics, as for a local arrival: what
// the waiter goes on to touch is ordered by tcgen05 or proxy fences issued before the arrival; a
// cluster-scope release here would drain the SM's outstanding stores every time).
__device__ __forceinline__ void mbar_arrive_remote(uint32_t caddr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(caddr) : "memory");
}
// What a bounded wait of the pair needs: this CTA's abort flag, the peer's (shared::cluster address) and
// the time limit of the launch (a kernel argument; rad_set_wait_limit_ns).
struct PairWait {
  volatile int* abort_flag;
  uint32_t peer_abort;
  uint64_t limit_ns;
};
// Bounded wait of the pair: on expiry both CTAs' abort flags are raised.  sleep_ns > 0: a long wait
// off the critical path (an epilogue warp waiting for a whole tile) leaves the issue slots to others.
__device__ __forceinline__ bool mbar_wait2(uint32_t bar, uint32_t parity, const PairWait& wc, uint32_t sleep_ns = 0) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 32; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      if (sleep_ns != 0) __nanosleep(sleep_ns);
    }
    if (*wc.abort_flag != 0) return false;
    if (global_timer_ns() - t0 > wc.limit_ns) {
      *wc.abort_flag = 1;
      asm volatile("st.relaxed.cluster.shared::cluster.u32 [%0], %1;" ::"r"(wc.peer_abort), "r"(1u) : "memory");
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t cbar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(cbar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {   // the barrier at this offset in both CTAs
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D = f32, A = B = bf16, M = 256 over the pair, N = n (a multiple of 16, at most 256).
__host__ __device__ constexpr uint32_t make_idesc_pair(bool a_mn, bool b_mn, uint32_t n = 256u) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((n >> 3) << 17) | ((256u >> 4) << 24);
}

template <int AK, int BKIND, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads2, 1)
tc_gemm_pair_kernel(const TcParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  SmemCtl2* ctl = reinterpret_cast<SmemCtl2*>(smem + (size_t)kStages2 * kStage2Bytes);
  volatile int* abort_flag = &ctl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();         // 0: issues the MMAs; both stage operands and run epilogues
  const uint32_t peer_abort = map_to_cta(smem_u32(&ctl->abort_flag), rank ^ 1u);
  const PairWait wc = {abort_flag, peer_abort, p.wait_limit_ns};
  // Same-sample dW (kDwT): the tile is dW^T, M = H, N = kept columns (known on the device only).  The kept
  // columns are cut into the fewest tiles of at most 256 and the tile width bn is what one of them needs,
  // rounded up to the MMA's granule of 16: 105 kept columns cost one tile of 112, not one of 256.
  int64_t n_cols = p.N;
  int bn = BN;
  if (EPI == kDwT) {
    int64_t nd;
    asm volatile("ld.global.cg.s64 %0, [%1];" : "=l"(nd) : "l"(p.N_dev) : "memory");
    n_cols = nd < n_cols ? nd : n_cols;
    const int64_t nt = max((int64_t)1, (n_cols + BN - 1) / BN);
    bn = max(16, (int)(((n_cols + nt - 1) / nt + 15) / 16 * 16));
  }
  const Schedule sched(p.M, n_cols, p.K, p.splits, BM, bn);
  const int boxes_b = (EPI == kDwT) ? (bn / 2 + 63) / 64 : 2;     // 64-column boxes of B this CTA stages per K block
  const uint32_t stage_tx = 2u * (uint32_t)(kStage2Bytes / 2 + boxes_b * 8192);
  const int64_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  if (tid == 0) {
    for (int s = 0; s < kStages2; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[b]), 2 * kEpiWarps2);
    }
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // the same warp of both CTAs allocates for the pair: two 128 x 256 accumulators per CTA
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&ctl->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();        // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  const uint32_t smem_base = smem_u32(smem);

  if (warp == 0) {
    // ===== TMA producer: this CTA's 128 rows of A and 128 rows (N) of B, completing on the even CTA's barrier =====
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      const int m_own = (int)w.m0 + 128 * (int)rank, n_own = (int)w.n0 + (bn / 2) * (int)rank;
      for (int kb = w.kb0; kb < w.kb1; ++kb) {
        if (lane == 0) {
          ok = mbar_wait2(smem_u32(&ctl->empty[stage]), phase ^ 1u, wc);
          if (ok) {
            const uint32_t sA = smem_base + stage * kStage2Bytes;
            const uint32_t sB = sA + kStage2Bytes / 2;
            const uint32_t full = map_to_cta(smem_u32(&ctl->full[stage]), 0u);
            const int k0 = kb * BK;
            if (rank == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[stage]), stage_tx);   // both CTAs' bytes
            if (AK == kAK) {
              tma_load_2d_pair(sA, &tmA, k0, m_own, full);                         // 64 (K) x 128 rows
            } else {
#pragma unroll
              for (int c = 0; c < 2; ++c) tma_load_2d_pair(sA + c * 8192, &tmA, m_own + c * 64, k0, full);
            }
            if (BKIND == kBK_) {
              tma_load_2d_pair(sB, &tmB, k0, n_own, full);
            } else {
#pragma unroll
              for (int c = 0; c < 2; ++c)
                if (c < boxes_b) tma_load_2d_pair(sB + c * 8192, &tmB, n_own + c * 64, k0, full);
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (++stage == kStages2) { stage = 0; phase ^= 1u; }
      }
    }
    // tail: every commit aimed at this CTA's stage barriers has landed before the CTA may leave
    if (lane == 0) {
      for (int i = 0; i < kStages2 && ok; ++i) {
        ok = mbar_wait2(smem_u32(&ctl->empty[stage]), phase ^ 1u, wc);
        if (++stage == kStages2) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer: one thread of the even CTA drives both tensor cores =====
    if (rank == 0) {
      const uint32_t idesc = make_idesc_pair(AK != kAK, BKIND == kBMN, (uint32_t)bn);
      int stage = 0, buf = 0;
      uint32_t phase = 0, buf_phases = 0;          // bit b: phase of accumulator b
      bool ok = true;
      for (int64_t u = pair; u < sched.units && ok; u += npairs) {
        const Unit w = sched.unit(u);
        if (lane == 0)
          ok = mbar_wait2(smem_u32(&ctl->tmem_empty[0]) + 8u * buf, ((buf_phases >> buf) & 1u) ^ 1u, wc);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        tc_fence_after();
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (lane == 0) {
            ok = mbar_wait2(smem_u32(&ctl->full[stage]), phase, wc);
            if (ok) {
              tc_fence_after();
              const uint32_t sA = smem_base + stage * kStage2Bytes;
              const uint32_t sB = sA + kStage2Bytes / 2;
#pragma unroll
              for (int k = 0; k < BK / 16; ++k) {
                const uint64_t adesc = (AK == kAK) ? make_desc(sA + k * 32, 16, 1024) : make_desc(sA + k * 2048, 8192, 1024);
                const uint64_t bdesc = (BKIND == kBK_) ? make_desc(sB + k * 32, 16, 1024) : make_desc(sB + k * 2048, 8192, 1024);
                tc_mma_pair(tmem_base + buf * 256, adesc, bdesc, idesc, (kb > w.kb0 || k > 0) ? 1u : 0u);
              }
              tc_commit_pair(smem_u32(&ctl->empty[stage]));          // frees the stage in both CTAs
              if (kb == w.kb1 - 1) tc_commit_pair(smem_u32(&ctl->tmem_full[0]) + 8u * buf);
            }
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
          if (++stage == kStages2) { stage = 0; phase ^= 1u; }
        }
        buf_phases ^= 1u << buf;
        buf ^= 1;
      }
    }
  } else {
    // ===== epilogue: thread = one accumulator row of this CTA, 128 columns per warp =====
    const int q = warp & 3;
    // the two warps of a lane quarter split the tile's 32-column chunks between them
    const int chunks = (bn + 31) / 32, half_chunks = (chunks + 1) / 2;
    const int c_first = ((warp - 2) >> 2) * half_chunks * 32;
    const int c_last = min(c_first + half_chunks * 32, chunks * 32);
    const uint32_t empty_bar = map_to_cta(smem_u32(&ctl->tmem_empty[0]), 0u);     // [b] is 8 bytes further
    int buf = 0;
    uint32_t buf_phases = 0;
    bool ok = true;
    if (EPI == kDwT && p.keep_cols != nullptr) {
      // Rows of dW whose column was not kept are zero (Sec. 4.3: only the sampled part of the weight matrix
      // gets a gradient).  The epilogue warps have nothing to do until the first tile's MMAs retire, so they
      // write those rows now: row d belongs to CTA d mod grid, a thread writes 16 bytes at a time.
      const int et = tid - 64;                       // 0 .. 255
      const int64_t h4 = p.M / 4;
      for (int64_t d = blockIdx.x; d < p.dw_rows; d += gridDim.x) {
        if ((__ldg(p.keep_cols + (d >> 5)) >> (d & 31)) & 1u) continue;
        float4* rowp = reinterpret_cast<float4*>(p.out_dw + d * p.ld_dw);
        for (int64_t i = et; i < h4; i += 32 * kEpiWarps2) rowp[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      if (lane == 0) ok = mbar_wait2(smem_u32(&ctl->tmem_full[0]) + 8u * buf, (buf_phases >> buf) & 1u, wc, 200u);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      tc_fence_after();
      const int64_t m = w.m0 + 128 * (int64_t)rank + q * 32 + lane;
      const bool row_ok = m < sched.M;
#pragma unroll 1
      for (int c0 = c_first; c0 < c_last; c0 += 32) {
        const int64_t n = w.n0 + c0;
        if (n >= n_cols) break;               // warp-uniform
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256 + c0), r);
        tmem_ld_wait();
        // a chunk may reach past the tile's width (bn is a multiple of 16) and past the last kept column
        if (EPI == kDwT) epilogue_chunk_dwt(p, r, m, n, (int)min((int64_t)min(32, bn - c0), n_cols - n), row_ok, w.split);
        else epilogue_chunk<(EPI == kDwT ? kDw : EPI)>(p, r, m, n, row_ok, w.split);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(empty_bar + 8u * buf);
      buf_phases ^= 1u << buf;
      buf ^= 1;
    }
  }

  // ===== teardown: neither CTA leaves (or frees tensor memory) while the other may still use it =====
  tc_fence_before();
  cluster_sync_all();
  if (tid == 0 && ctl->abort_flag != 0) raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---- two-CTA engine, sparse A (different-sample dW) --------------------------------------------------
// The pair owns a 256 x 512 tile of dW.  Each CTA rebuilds 128 columns of A_hat (one store tile per
// K block) in shared memory and loads its half of the dZ tile (two blocks of 128 columns); per 16
// rows of K two MMAs (M256 N256), one per 256-column half of the tile; the two 128 x 256
// accumulators of a CTA fill its tensor memory.  A store tile is expanded once per 512 output
// columns: the wide tile halves the expansion work per flop against a 256-column tile and brings the
// shared-memory traffic per K block and CTA from about 1540 to about 1200 wavefronts.
// Roles per CTA: 0 dZ producer, 1 MMA issuer (even CTA) and tensor-memory owner, 2-5 epilogue,
// 6 producer of the compressed ring, 7-22 expanders (two groups on alternate K blocks).  full[s] lives in the even CTA: one arrival
// with the dZ bytes of both CTAs plus one per expander warp of either CTA.
constexpr int kSpBM = 256, kSpBN = 512;
constexpr int kSpAStageBytes = 128 * BK * 2;           // 16 KB: this CTA's 128 columns of A_hat
constexpr int kSpBStageBytes = 256 * BK * 2;           // 32 KB: this CTA's 2 x 128 columns of dZ
constexpr int kSpStageBytes = kSpAStageBytes + kSpBStageBytes;
constexpr int kSpMaxStages = 4;
constexpr int kSpExpanderWarps = 8;                    // per K block: one thread per keep-bit word of the store tile
constexpr int kSpExpanderGroups = 2;                   // groups of eight warps take alternate K blocks
constexpr int kSpThreads = 32 * (kFirstExpanderWarp + kSpExpanderGroups * kSpExpanderWarps);

struct SmemCtlSp {
  uint64_t full[kSpMaxStages], empty[kSpMaxStages], comp_full[8], comp_empty[8], tmem_full, tmem_empty;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kSpThreads, 1)
tc_sparse_pair_kernel(const TcParams p, const __grid_constant__ CUtensorMap tmB) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stages = p.num_stages;
  const int comp_slot = kIndexBytes + p.comp_cap;               // index data + values of this CTA's store tile of one K block
  uint8_t* comp_base = smem + (size_t)stages * kSpStageBytes;
  SmemCtlSp* ctl = reinterpret_cast<SmemCtlSp*>(comp_base + (size_t)p.comp_depth * comp_slot);
  volatile int* abort_flag = &ctl->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t peer_abort = map_to_cta(smem_u32(&ctl->abort_flag), rank ^ 1u);
  const PairWait wc = {abort_flag, peer_abort, p.wait_limit_ns};
  const Schedule sched(p.M, p.N, p.K, p.splits, kSpBM, kSpBN);
  const int64_t pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1 + 2 * kSpExpanderWarps);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int c = 0; c < p.comp_depth; ++c) {
      mbar_init(smem_u32(&ctl->comp_full[c]), 1);
      mbar_init(smem_u32(&ctl->comp_empty[c]), kSpExpanderWarps);
    }
    mbar_init(smem_u32(&ctl->tmem_full), 1);
    mbar_init(smem_u32(&ctl->tmem_empty), 8);          // four epilogue warps in each CTA
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&ctl->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  const uint32_t smem_base = smem_u32(smem);
  // this CTA's store tile column (128 columns of the layer input) of a unit, and whether it exists
  auto tile_col_of = [&](const Unit& w) -> int64_t { return (w.m0 + 128 * (int64_t)rank) / kTileCols; };

  if (warp == 0) {
    // ===== dZ producer: this CTA's 128 columns of each 256-column half of the dZ tile =====
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      const int n_own = (int)w.n0 + 128 * (int)rank;       // + 256 for the second half
      for (int kb = w.kb0; kb < w.kb1; ++kb) {
        if (lane == 0) {
          ok = mbar_wait2(smem_u32(&ctl->empty[stage]), phase ^ 1u, wc);
          if (ok) {
            const uint32_t sB = smem_base + stage * kSpStageBytes + kSpAStageBytes;
            if (rank == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[stage]), 2 * kSpBStageBytes);   // both CTAs' bytes
            const uint32_t full = map_to_cta(smem_u32(&ctl->full[stage]), 0u);
#pragma unroll
            for (int c = 0; c < 4; ++c)
              tma_load_2d_pair(sB + c * 8192, &tmB, n_own + (c >> 1) * 256 + (c & 1) * 64, kb * BK, full);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
    if (lane == 0) {   // every commit aimed at this CTA's stage barriers has landed before the CTA may leave
      for (int i = 0; i < stages && ok; ++i) {
        ok = mbar_wait2(smem_u32(&ctl->empty[stage]), phase ^ 1u, wc);
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer (even CTA) =====
    if (rank == 0) {
      constexpr uint32_t idesc = make_idesc_pair(true, true);
      int stage = 0;
      uint32_t phase = 0, unit_phase = 0;
      bool ok = true;
      for (int64_t u = pair; u < sched.units && ok; u += npairs) {
        const Unit w = sched.unit(u);
        if (lane == 0) ok = mbar_wait2(smem_u32(&ctl->tmem_empty), unit_phase ^ 1u, wc);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        tc_fence_after();
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (lane == 0) {
            ok = mbar_wait2(smem_u32(&ctl->full[stage]), phase, wc);
            if (ok) {
              tc_fence_after();
              const uint32_t sA = smem_base + stage * kSpStageBytes;
              const uint32_t sB = sA + kSpAStageBytes;
#pragma unroll
              for (int k = 0; k < BK / 16; ++k) {
                const uint64_t adesc = make_desc(sA + k * 2048, 8192, 1024);
#pragma unroll
                for (int j = 0; j < 2; ++j)
                  tc_mma_pair(tmem_base + j * 256, adesc, make_desc(sB + j * 16384 + k * 2048, 8192, 1024), idesc,
                              (kb > w.kb0 || k > 0) ? 1u : 0u);
              }
              tc_commit_pair(smem_u32(&ctl->empty[stage]));
              if (kb == w.kb1 - 1) tc_commit_pair(smem_u32(&ctl->tmem_full));
            }
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
        unit_phase ^= 1u;
      }
    }
  } else if (warp < 6) {
    // ===== epilogue: thread = one accumulator row (512 columns) =====
    const int q = warp & 3;
    const uint32_t empty_bar = map_to_cta(smem_u32(&ctl->tmem_empty), 0u);
    uint32_t unit_phase = 0;
    bool ok = true;
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      if (lane == 0) ok = mbar_wait2(smem_u32(&ctl->tmem_full), unit_phase, wc, 1000u);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      tc_fence_after();
      const int64_t m = w.m0 + 128 * (int64_t)rank + q * 32 + lane;
      const bool row_ok = m < sched.M;
#pragma unroll 1
      for (int c0 = 0; c0 < kSpBN; c0 += 32) {
        const int64_t n = w.n0 + c0;
        if (n >= p.N) break;                  // warp-uniform
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
        tmem_ld_wait();
        epilogue_chunk<kDw>(p, r, m, n, row_ok, w.split);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(empty_bar);
      unit_phase ^= 1u;
    }
  } else if (warp == 6) {
    // ===== producer of the compressed ring: keep bits + row offsets (1152 B) and packed values of
    // this CTA's store tile of each K block.  It runs ahead of the A/B ring: a slot is free as soon
    // as the expanders have read it, long before the MMAs of that K block retire. =====
    int slot = 0;
    uint32_t cphase = 0;
    bool ok = true;
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      const int64_t tile_col = tile_col_of(w);
      const bool have = tile_col < p.ncb;
      uint32_t off_lo = 0, off_hi = 0;                // tile offsets of K block (base + lane)
      for (int kb = w.kb0; kb < w.kb1; ++kb) {
        if (((kb - w.kb0) & 31) == 0 && have) {
          const int kbl = kb + lane;
          if (kbl < w.kb1) {
            const int64_t t0 = (int64_t)kbl * p.ncb + tile_col;
            off_lo = __ldg(p.offsets + t0);
            off_hi = __ldg(p.offsets + t0 + 1);
          }
        }
        const int src = (kb - w.kb0) & 31;
        const uint32_t o0 = __shfl_sync(0xffffffffu, off_lo, src);
        const uint32_t o1 = __shfl_sync(0xffffffffu, off_hi, src);
        if (lane == 0) {
          ok = mbar_wait2(smem_u32(&ctl->comp_empty[slot]), cphase ^ 1u, wc);
          if (ok) {
            const uint32_t cfull = smem_u32(&ctl->comp_full[slot]);
            const uint32_t sC = smem_u32(comp_base) + slot * comp_slot;
            uint32_t vb = have ? (o1 - o0) * 2u : 0u;
            if (vb > (uint32_t)p.comp_cap || (int64_t)o1 > p.values_capacity) {
              vb = 0;
              raise_status(p.dev_status, RAD_DEV_ECAPACITY);
            }
            mbar_arrive_expect_tx(cfull, (have ? (uint32_t)kIndexBytes : 0u) + vb);
            if (have) {
              bulk_load(sC, p.keepbits + ((int64_t)kb * p.ncb + tile_col) * kTileWords, kIndexBytes, cfull);
              if (vb != 0) bulk_load(sC + kIndexBytes, p.values + o0, vb, cfull);
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (++slot == p.comp_depth) { slot = 0; cphase ^= 1u; }
      }
    }
  } else {
    // ===== expanders: rebuild this CTA's A_hat tile (64 K rows x 128 columns, M-major, swizzled) =====
    // One thread per keep-bit word: row r of the slab, columns 32*wq..32*wq+31 of the store tile.
    // The row's first value is given by the stored row offset; the words before this one in the row
    // are counted with popc.  Eight consecutive lanes take eight consecutive rows of the same word
    // column: with the 128-byte swizzle their 16-byte zero stores then fall on eight different bank
    // groups.
    // Two groups of eight warps take alternate K blocks, so the waits, loads and fence of one K
    // block overlap the stores of the next.
    const int et = tid - 32 * kFirstExpanderWarp;            // 0..511
    const uint32_t group = (uint32_t)(et >> 8);
    const int wi = et & 255;
    const int r = (wi & 7) + ((wi >> 5) << 3), wq = (wi >> 3) & 3;
    int stage = 0, slot = 0;
    uint32_t phase = 0, cphase = 0, turn = 0;
    bool ok = true;
    for (int64_t u = pair; u < sched.units && ok; u += npairs) {
      const Unit w = sched.unit(u);
      const bool have = tile_col_of(w) < p.ncb;
      for (int kb = w.kb0; kb < w.kb1; ++kb, turn ^= 1u) {
        if (turn == group) {
          ok = mbar_wait2(smem_u32(&ctl->comp_full[slot]), cphase, wc) &&
               mbar_wait2(smem_u32(&ctl->empty[stage]), phase ^ 1u, wc);     // A tile of this stage is free
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          // columns past the layer's width keep whatever the buffer held: their accumulator rows are never written
          if (have) {
            uint8_t* sA = smem + (size_t)stage * kSpStageBytes;
            const uint8_t* sC = comp_base + (size_t)slot * comp_slot;
            expand_word(sA, sC, 0, r, wq, (uint32_t)p.comp_cap >> 1);
            fence_proxy_async();
          }
          __syncwarp();
          if (lane == 0) {
            mbar_arrive_remote(map_to_cta(smem_u32(&ctl->full[stage]), 0u));
            mbar_arrive(smem_u32(&ctl->comp_empty[slot]));
          }
        }
        if (++stage == stages) { stage = 0; phase ^= 1u; }
        if (++slot == p.comp_depth) { slot = 0; cphase ^= 1u; }
      }
    }
  }

  // ===== teardown: neither CTA leaves (or frees tensor memory) while the other may still use it =====
  tc_fence_before();
  cluster_sync_all();
  if (tid == 0 && ctl->abort_flag != 0) raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// The pair kernels' bounded wait on a barrier nobody arrives at, in a cluster of two CTAs that owns no tensor
// memory and has no loads in flight: both waits run out, both abort flags go up, the pair meets at the
// cluster barrier as the real kernels do on their way out, and the status word reports the timeout.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(64, 1) wait_probe_pair_kernel(uint64_t limit_ns, int32_t* dev_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  const uint32_t rank = cluster_ctarank();
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_sync_all();
  const PairWait wc = {&abort_flag, map_to_cta(smem_u32(&abort_flag), rank ^ 1u), limit_ns};
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait2(smem_u32(&bar), 0u, wc, 100u);
  cluster_sync_all();
  if (threadIdx.x == 0 && (!ok || abort_flag != 0)) raise_status(dev_status, RAD_DEV_ETIMEOUT);
}

// Sum of the K-split partial tiles in split order; rows may be scattered (same-sample).
__global__ void __launch_bounds__(256) dw_reduce_kernel(const float* partial, int64_t partial_rows, int splits,
                                                        int64_t M, const int64_t* M_dev, int64_t N,
                                                        const uint32_t* row_idx, float* out, int64_t ldw) {
  if (M_dev != nullptr) M = min(M, *M_dev);
  const int64_t n4 = N / 4, total = M * n4;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t m = i / n4, c = i % n4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < splits; ++s) {
      const float4 v = __ldcs(reinterpret_cast<const float4*>(partial + ((int64_t)s * partial_rows + m) * N) + c);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    const int64_t row = row_idx != nullptr ? (int64_t)row_idx[m] : m;
    reinterpret_cast<float4*>(out + row * ldw)[c] = acc;
  }
}

// ---- host side -------------------------------------------------------------------------------------
}  // namespace

// cuTensorMapEncodeTiled through the runtime's driver entry point table (no link against libcuda).
void* tensor_map_encoder() {
  static void* fn = nullptr;
  if (fn == nullptr) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = sym;
  }
  return fn;
}

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() { return reinterpret_cast<EncodeTiledFn>(tensor_map_encoder()); }

// bf16 matrix, `inner` contiguous elements per row, `outer` rows of `ld` elements; box = 64 x box_outer.
int make_map(CUtensorMap* map, const void* ptr, int64_t inner, int64_t outer, int64_t ld, int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return RAD_ECUDA;
  const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_outer};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? RAD_OK : RAD_ECUDA;
}

int num_sms() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = kNumSMsDefault;
  }
  return n;
}

// K splits for a dW contraction.  Cost model in units of one CTA working through one K block
// (about 1024 tensor-pipe clocks): waves x K blocks per unit, plus what writing and re-reading the
// float32 partial tiles costs at HBM speed.  Pure function of the shapes, so the workspace query
// and the launch agree.
int choose_splits(int64_t m_tiles, int64_t n_tiles, int64_t kblocks, int64_t bm = BM, int64_t sms = kNumSMsDefault,
                  int64_t bn = BN, double kblock_scale = 1.0) {
  const double kblock_us = 0.55 * kblock_scale;                             // 1024 clk at ~1.9 GHz for a 256-wide tile
  const double partial_us = (double)(m_tiles * bm) * (double)(n_tiles * bn) * 8.0 / 6.5e6;   // per split
  int best = 1;
  double best_cost = 1e300;
  for (int s = 1; s <= kMaxSplits && s <= kblocks; ++s) {
    const int64_t units = m_tiles * n_tiles * s;
    const double cost = (double)ceil_div(units, sms) * (double)ceil_div(kblocks, s) * kblock_us +
                        (s > 1 ? partial_us * s + 5.0 : 0.0);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return best;
}

struct DwPlan { int splits; int64_t partial_rows; int64_t bytes; int comp_cap; int stages; int comp_depth; };

// Clusters of two CTAs of `kernel` that can be resident at once.
template <typename K>
int resident_pairs_of(K kernel, int threads, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (num_sms() / 2));
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    n = num_sms() / 2;
  }
  return std::min(n, num_sms() / 2);
}

// SM pairs the K splits of a dW contraction are planned for: what the device can really keep resident (a part
// whose SM count per GPC is odd somewhere hosts fewer two-CTA clusters than half its SMs, and a plan for 74
// pairs on 72 runs an extra wave), or half the default SM count where there is no device to ask (size queries
// on a host without one).  Found once, so that workspace queries and launches agree.
int planning_pairs() {
  static int pairs = 0;
  if (pairs == 0) {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10 &&
        cudaFuncSetAttribute(tc_sparse_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) == cudaSuccess) {
      pairs = resident_pairs_of(tc_sparse_pair_kernel, kSpThreads, 227 * 1024);
    } else {
      (void)cudaGetLastError();
      pairs = kNumSMsDefault / 2;
    }
  }
  return pairs;
}

DwPlan plan_dw(const rad_store* st, int64_t H) {
  DwPlan d;
  const int64_t kblocks = ceil_div(st->B, BK);
  int64_t m_expect;
  if (st->variant == RAD_SAME_SAMPLE) {
    // transposed tile: M = H, N = kept columns in tiles of at most 256 (the kernel fits the width to the count)
    m_expect = std::max<int64_t>(1, (int64_t)std::llround((double)st->D * store_keep_fraction(st)));
    d.partial_rows = round_up(std::min(st->values_ld, round_up(st->D, 8)), 16);
    d.comp_cap = 0;
    d.stages = 3;
    d.comp_depth = 0;
    const int64_t n_tiles = ceil_div(m_expect, BN);
    const int64_t bn = round_up(ceil_div(m_expect, n_tiles), 16);
    d.splits = choose_splits(ceil_div(H, BM), n_tiles, kblocks, BM, planning_pairs(), bn, (double)bn / BN);
    d.bytes = d.splits > 1 ? (int64_t)d.splits * d.partial_rows * H * 4 : 0;
    return d;
  } else {
    m_expect = st->D;
    d.partial_rows = round_up(st->D, BM);
    // per-tile value staging: mean + 8 sigma of Binomial(8192, p_eff), padded, in bytes
    const double pe = store_keep_fraction(st), n = (double)kTileRows * kTileCols;
    int64_t cap = (int64_t)(n * pe + 8.0 * std::sqrt(n * pe * (1.0 - pe)) + 16.0);
    cap = std::min<int64_t>(round_up(cap, 8), (int64_t)n) * 2;
    d.comp_cap = (int)round_up(cap, 128);
    // shared memory: 48 KB per A/B stage plus a ring of compressed slots
    const int64_t budget = 227 * 1024 - 2048 - (int64_t)sizeof(SmemCtlSp);
    const int64_t slot = kIndexBytes + d.comp_cap;
    d.stages = (4 * kSpStageBytes + 3 * slot <= budget) ? 4 : (3 * kSpStageBytes + 2 * slot <= budget) ? 3 : 2;
    d.comp_depth = (int)std::max<int64_t>(2, std::min<int64_t>(8, (budget - d.stages * kSpStageBytes) / slot));
    d.splits = choose_splits(ceil_div(m_expect, kSpBM), ceil_div(H, kSpBN), kblocks, kSpBM, planning_pairs(), kSpBN);
    d.bytes = d.splits > 1 ? (int64_t)d.splits * d.partial_rows * H * 4 : 0;
    return d;
  }
}

template <int AK, int BKIND, int EPI>
int launch_pair(const TcParams& p, const CUtensorMap& ta, const CUtensorMap& tb, int64_t max_units, cudaStream_t s) {
  constexpr size_t smem = (size_t)kStages2 * kStage2Bytes + sizeof(SmemCtl2) + 1024;
  static_assert(smem <= 227 * 1024, "stage ring too deep");
  auto kernel = tc_gemm_pair_kernel<AK, BKIND, EPI>;
  // The kernel is persistent: the grid must not exceed the clusters that can be resident at once
  // (SM pairs that can host a cluster; fewer than half the SM count on some parts).
  static int resident_pairs = 0;
  if (resident_pairs == 0) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return RAD_ECUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (num_sms() / 2));
    cfg.blockDim = dim3(kThreads2);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = num_sms() / 2;
    }
    resident_pairs = std::min(n, num_sms() / 2);
  }
  const int pairs = (int)std::max<int64_t>(1, std::min<int64_t>(max_units, resident_pairs));
  count_launch();
  kernel<<<2 * pairs, kThreads2, smem, s>>>(p, ta, tb);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

int launch_sparse_pair(const TcParams& p, const CUtensorMap& tb, int64_t max_units, cudaStream_t s) {
  const size_t smem = (size_t)p.num_stages * kSpStageBytes + (size_t)p.comp_depth * (kIndexBytes + p.comp_cap) +
                      sizeof(SmemCtlSp) + 1024;
  if (smem > 227 * 1024 || p.num_stages > kSpMaxStages || p.comp_depth > 8) return RAD_EUNSUPPORTED;
  static int resident_pairs = 0;
  if (resident_pairs == 0) {
    if (cudaFuncSetAttribute(tc_sparse_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return RAD_ECUDA;
    resident_pairs = resident_pairs_of(tc_sparse_pair_kernel, kSpThreads, 227 * 1024);
  }
  const int pairs = (int)std::max<int64_t>(1, std::min<int64_t>(max_units, resident_pairs));
  count_launch();
  tc_sparse_pair_kernel<<<2 * pairs, kSpThreads, smem, s>>>(p, tb);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

int launch_wait_probe_pair(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s) {
  count_launch();
  wait_probe_pair_kernel<<<2, 64, 0, s>>>(limit_ns, dev_status);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

bool tc_shape_ok(int64_t B, int64_t D, int64_t H, const void* p0, int64_t ld0, const void* p1, int64_t ld1) {
  if (B < 64 || D < 64 || H < 64) return false;                    // tiny layers stay on CUDA cores
  if (D % 8 != 0 || H % 8 != 0) return false;
  if (!aligned16(p0) || !aligned16(p1) || ld0 % 8 != 0 || ld1 % 8 != 0) return false;
  if (B >= (1ll << 31) || D >= (1ll << 31) || H >= (1ll << 31)) return false;
  return encode_fn() != nullptr;
}

int tc_forward(int act, int64_t B, int64_t D, int64_t H, const void* A, int64_t lda, const void* W, int64_t ldw,
               const float* bias, void* out_act, int64_t ld_act, float* out_z, int64_t ld_z, void* out_zlow,
               int64_t ld_zlow, uint32_t* relubits, int32_t* dev_status, cudaStream_t s, const rad_store* next) {
  CUtensorMap ta, tb;
  int rc = make_map(&ta, A, D, B, lda, 128);          // K-major A: box 64 (K) x 128 rows (one CTA of the pair)
  if (rc != RAD_OK) return rc;
  rc = make_map(&tb, W, H, D, ldw, 64);               // MN-major B: box 64 (N) x 64 K rows
  if (rc != RAD_OK) return rc;
  TcParams p = {};
  p.M = B; p.N = H; p.K = D; p.splits = 1; p.num_stages = 3;
  p.bias = bias; p.act = act;
  p.out_act = static_cast<bf16*>(out_act); p.ld_act = ld_act; p.out_z = out_z; p.ld_z = ld_z;
  p.out_zlow = static_cast<bf16*>(out_zlow); p.ld_zlow = ld_zlow; p.relubits = relubits; p.w32 = ceil_div(H, 32);
  p.dev_status = dev_status;
  p.wait_limit_ns = wait_limit_ns();
  if (next != nullptr) {
    // the store of this layer's output (B x H) as the next layer's input; its index part is in place
    if (out_act == nullptr || next->B != B || next->D != H || next->dtype != RAD_BF16 || !aligned16(next->keepbits))
      return RAD_EINVAL;
    p.st_values = static_cast<bf16*>(next->values); p.st_keepbits = next->keepbits; p.st_offsets = next->offsets;
    p.st_capacity = next->values_capacity; p.st_ncb = (int32_t)ceil_div(H, kTileCols);
    p.st_scale = next->law == RAD_LAW_FIXED ? (float)H / (float)draws_per_row_host(next->p, H)
                                            : (float)kLaneRange / (float)keep_threshold_host(next->p);
  }
  return launch_pair<kAK, kBMN, kFwd>(p, ta, tb, ceil_div(B, BM) * ceil_div(H, BN), s);
}

int tc_input_grad(int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz, const void* W, int64_t ldw,
                  const uint32_t* relubits_prev, const void* z_prev, int64_t ld_zprev, void* dZ_prev, int64_t ldp,
                  int32_t* dev_status, cudaStream_t s) {
  CUtensorMap ta, tb;
  int rc = make_map(&ta, dZ, H, B, ldz, 128);         // K-major A (K = H)
  if (rc != RAD_OK) return rc;
  rc = make_map(&tb, W, H, D, ldw, 128);              // K-major B: rows d (N), K = H contiguous
  if (rc != RAD_OK) return rc;
  TcParams p = {};
  p.M = B; p.N = D; p.K = H; p.splits = 1; p.num_stages = 3;
  p.relubits_prev = relubits_prev; p.z_prev = static_cast<const bf16*>(z_prev); p.ld_zprev = ld_zprev;
  p.out_dx = static_cast<bf16*>(dZ_prev); p.ld_dx = ldp;
  p.dev_status = dev_status;
  p.wait_limit_ns = wait_limit_ns();
  return launch_pair<kAK, kBK_, kDx>(p, ta, tb, ceil_div(B, BM) * ceil_div(D, BN), s);
}

int sm_pairs() { return planning_pairs(); }

int64_t tc_weight_grad_workspace(const rad_store* st, int64_t H) {
  if (st->dtype != RAD_BF16 || st->D % 8 != 0 || H % 8 != 0 || st->B < 64 || st->D < 64 || H < 64) return 0;
  return plan_dw(st, H).bytes;
}

int tc_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW, int64_t ldw,
                   void* workspace, int64_t workspace_bytes, int32_t* dev_status, cudaStream_t s) {
  const DwPlan d = plan_dw(st, H);
  if (d.bytes > 0 && (workspace == nullptr || workspace_bytes < d.bytes || !aligned16(workspace))) return RAD_EWORKSPACE;
  if (!aligned16(st->keepbits) || !aligned16(st->values)) return RAD_EUNSUPPORTED;
  CUtensorMap ta, tb;
  int rc = make_map(&tb, dZ, H, st->B, ldz, 64);      // MN-major B: box 64 (N = h) x 64 K rows (b)
  if (rc != RAD_OK) return rc;
  TcParams p = {};
  p.N = H; p.K = st->B; p.splits = d.splits; p.num_stages = d.stages; p.comp_depth = d.comp_depth;
  p.out_dw = dW; p.ld_dw = ldw; p.dw_rows = st->D; p.partial = static_cast<float*>(workspace); p.partial_rows = d.partial_rows;
  p.dev_status = dev_status;
  p.wait_limit_ns = wait_limit_ns();
  if (st->variant == RAD_SAME_SAMPLE) {
    // dW[idx, :]^T = dZ^T A_c: A operand dZ (M = h, MN-major), B operand the gathered block A_c (N = kept
    // column, MN-major), K = minibatch rows; the tile lands transposed and is scattered by kept column
    const int64_t nmax = std::min(st->values_ld, round_up(st->D, 8));
    ta = tb;                                           // dZ: box 64 (h) x 64 K rows
    rc = make_map(&tb, st->values, st->values_ld, st->B, st->values_ld, 64);
    if (rc != RAD_OK) return rc;
    p.M = H; p.N = nmax; p.N_dev = st->nnz; p.row_idx = st->offsets; p.keep_cols = st->keepbits;
    const int64_t n_expect = std::max<int64_t>(1, (int64_t)std::llround((double)st->D * store_keep_fraction(st)));
    rc = launch_pair<kAMN, kBMN, kDwT>(p, ta, tb, ceil_div(H, BM) * ceil_div(std::min(n_expect, nmax), BN) * d.splits, s);
  } else {
    ta = tb;                                           // unused by the sparse-A kernel
    p.M = st->D;
    p.values = static_cast<const bf16*>(st->values); p.keepbits = st->keepbits; p.offsets = st->offsets;
    p.values_capacity = st->values_capacity; p.ncb = (int32_t)ceil_div(st->D, kTileCols); p.comp_cap = d.comp_cap;
    rc = launch_sparse_pair(p, tb, ceil_div(st->D, kSpBM) * ceil_div(H, kSpBN) * d.splits, s);
  }
  if (rc != RAD_OK) return rc;
  if (d.splits > 1) {
    const int64_t rows = st->variant == RAD_SAME_SAMPLE ? p.N : p.M;       // rows of a partial block
    const int64_t work = rows * (H / 4);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>(ceil_div(work, 256), 148 * 16));
    count_launch();
    dw_reduce_kernel<<<grid, 256, 0, s>>>(p.partial, d.partial_rows, d.splits, rows, p.N_dev, H, p.row_idx, dW, ldw);
  }
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad
