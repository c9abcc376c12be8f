// Forward-pass store kernels: Philox keep mask, scale, compaction (Sec. 3.2 / 4.2 of the paper:
// the layer input is what gets sampled, never the Jacobian itself).
//
// different-sample: one pass over A.  A CTA takes one 64 x 128 tile (ticket order), draws the
// keep bits of its entries, counts them, and learns where its values start from a decoupled
// look-back over the tiles before it (each tile publishes first its own count, then its
// inclusive prefix, in a 64-bit status word).  Kept values are staged in shared memory in
// (row, column) order and leave as 16-byte stores.  The order of tiles in `values` is fixed by the
// tile index, so the layout does not depend on scheduling.
//
// same-sample: the column mask is drawn once (one CTA), then rows are gathered.
#include <algorithm>
#include <cmath>

#include "common.cuh"
#include "store.cuh"

namespace rad {

uint32_t keep_threshold_host(float p) {
  if (!(p > 0.0f) || !(p <= 1.0f)) return 0;
  double t = rint((double)p * (double)kLaneRange);
  if (t < 1.0) t = 1.0;
  if (t > (double)kLaneRange) t = (double)kLaneRange;
  return (uint32_t)t;
}

int64_t draws_per_row_host(float fraction, int64_t D) {
  if (!(fraction > 0.0f) || !(fraction <= 1.0f) || D <= 0) return 0;
  double k = ceil((double)fraction * (double)D * (1.0 - ldexp(1.0, -22)));
  if (k < 1.0) k = 1.0;
  if (k > (double)D) k = (double)D;
  return (int64_t)k;
}

// Expected share of kept entries: p_eff for Bernoulli keeps, 1 - (1 - 1/D)^k for k draws with replacement.
double store_keep_fraction(const rad_store* st) {
  if (st->law == RAD_LAW_REPLACE) {
    const double k = (double)draws_per_row_host(st->p, st->D), D = (double)st->D;
    return D <= 1.0 ? 1.0 : 1.0 - pow(1.0 - 1.0 / D, k);
  }
  if (st->law == RAD_LAW_FIXED) return (double)draws_per_row_host(st->p, st->D) / (double)st->D;
  return keep_threshold_host(st->p) / (double)kLaneRange;
}

namespace {

template <typename T> struct Raw8;   // eight consecutive elements of one row
template <> struct Raw8<float> { float v[8]; };
template <> struct Raw8<bf16> { uint4 q; };

template <typename T>
__device__ __forceinline__ void load8(const T* rowp, int64_t col0, int nvalid, bool vec, Raw8<T>& out);

template <>
__device__ __forceinline__ void load8<float>(const float* rowp, int64_t col0, int nvalid, bool vec,
                                             Raw8<float>& out) {
  if (vec && nvalid == 8) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(rowp + col0));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(rowp + col0 + 4));
    out.v[0] = a.x; out.v[1] = a.y; out.v[2] = a.z; out.v[3] = a.w;
    out.v[4] = b.x; out.v[5] = b.y; out.v[6] = b.z; out.v[7] = b.w;
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) out.v[i] = (i < nvalid) ? rowp[col0 + i] : 0.0f;
  }
}
template <>
__device__ __forceinline__ void load8<bf16>(const bf16* rowp, int64_t col0, int nvalid, bool vec,
                                            Raw8<bf16>& out) {
  if (vec && nvalid == 8) {
    out.q = __ldcs(reinterpret_cast<const uint4*>(rowp + col0));
  } else {
    const unsigned short* p = reinterpret_cast<const unsigned short*>(rowp) + col0;
    uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (i < nvalid) w[i >> 1] |= (uint32_t)p[i] << (16 * (i & 1));
    out.q = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

__device__ __forceinline__ float elem(const Raw8<float>& r, int i) { return r.v[i]; }
__device__ __forceinline__ float elem(const Raw8<bf16>& r, int i) {
  const uint32_t w = (i < 2) ? r.q.x : (i < 4) ? r.q.y : (i < 6) ? r.q.z : r.q.w;
  return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
}

// (a > 0) for the eight entries; zero of either sign gives 0.
template <typename T> __device__ __forceinline__ uint32_t positive8(const Raw8<T>& r) {
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) m |= (elem(r, i) > 0.0f ? 1u : 0u) << i;
  return m;
}

// Four lanes each hold one byte per item (4 items); afterwards lane k of the four holds the
// 32-bit word of item k: byte j = what lane j held for item k.
__device__ __forceinline__ uint32_t transpose4x4_bytes(uint32_t v, int k) {
  uint32_t x = __shfl_xor_sync(0xffffffffu, v, 1);
  v = (k & 1) ? __byte_perm(v, x, 0x3715) : __byte_perm(v, x, 0x6240);
  x = __shfl_xor_sync(0xffffffffu, v, 2);
  v = (k & 2) ? __byte_perm(v, x, 0x3276) : __byte_perm(v, x, 0x5410);
  return v;
}

// Where the mask comes from: a Bernoulli draw in the kernel; the multiplicity matrix of the with-replacement law
// (which also gives the weights); or keep bits and tile offsets that are already in place (made from the key
// alone by an index kernel), in which case only values and ReLU bits are written and nothing waits for anything.
enum MaskSource { kMaskDraw = 0, kMaskCounts = 1, kMaskIndex = 2 };
template <typename T, int kMask>
__global__ void __launch_bounds__(256) store_different_kernel(const StoreParams p, const PhiloxKeys ks) {
  constexpr bool kReplace = kMask == kMaskCounts;
  __shared__ uint32_t s_rowcnt[kTileRows];
  __shared__ uint32_t s_rowoff[kTileRows];
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_total;
  __shared__ int64_t s_base;        // first element of this tile in `values`, or -1: do not write
  __shared__ __align__(16) T s_stage[kTileRows * kTileCols];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_tile = kMask == kMaskIndex ? blockIdx.x : atomicAdd(p.ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  if (tile >= (uint32_t)p.ntiles) return;
  const int64_t slab = tile / p.ncb;
  const int cb = tile % p.ncb;
  const int half = lane >> 4, cg = lane & 15;
  const int64_t col0 = (int64_t)cb * kTileCols + cg * 8;
  const int nvalid = (int)max((int64_t)0, min((int64_t)8, p.D - col0));
  const T* Abase = static_cast<const T*>(p.A);

  Raw8<T> raw[4];
  uint2 mult[4];                                 // kReplace: the eight multiplicities of an item, a byte each
  uint32_t masks = 0, relus = 0, counts = 0;     // one byte per item: keep bits, ReLU bits, kept count
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int64_t row = slab * kTileRows + warp * 8 + it * 2 + half;
    // four lanes share a keep-bit word and make it together (all lanes take part, valid or not)
    uint32_t word = 0;
    if (kMask == kMaskDraw) word = philox_keep32_quad((uint32_t)(col0 >> 5), (uint32_t)row, p.c2, p.c3, ks, p.T, lane);
    if (kMask == kMaskIndex) word = p.keepbits[(int64_t)tile * kTileWords + (warp * 8 + it * 2 + half) * 4 + (cg >> 2)];
    if (row < p.B && nvalid > 0) {
      load8<T>(Abase + row * p.lda, col0, nvalid, p.vec_ok != 0, raw[it]);
      uint32_t m;
      if (kReplace) {
        mult[it] = *reinterpret_cast<const uint2*>(p.counts + row * p.ldc + col0);
        m = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i)
          m |= ((((i < 4 ? mult[it].x : mult[it].y) >> (8 * (i & 3))) & 0xffu) != 0 ? 1u : 0u) << i;
        m &= (1u << nvalid) - 1u;
      } else {
        // this lane's eight columns are one byte of the word
        m = (word >> (8 * (cg & 3))) & ((1u << nvalid) - 1u);
      }
      masks |= m << (8 * it);
      counts |= __popc(m) << (8 * it);
      if (p.relubits != nullptr) relus |= (positive8(raw[it]) & ((1u << nvalid) - 1u)) << (8 * it);
    }
  }
  // exclusive prefix of the kept count inside each row (16 lanes per row); the four items scan as
  // one word, a byte each (a row holds at most 128 kept entries)
  uint32_t incl = counts;
#pragma unroll
  for (int o = 1; o < 16; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o, 16);
    if (cg >= o) incl += n;
  }
  const uint32_t pres = incl - counts;
  if (cg == 15) {
#pragma unroll
    for (int it = 0; it < 4; ++it) s_rowcnt[warp * 8 + it * 2 + half] = (incl >> (8 * it)) & 0xffu;
  }
  {
    // four lanes make one 32-bit word of keep bits (and of ReLU bits) per item
    const int k = cg & 3;
    const int r = warp * 8 + k * 2 + half;
    if (kMask != kMaskIndex) p.keepbits[(int64_t)tile * kTileWords + r * 4 + (cg >> 2)] = transpose4x4_bytes(masks, k);
    if (p.relubits != nullptr) {
      const uint32_t rw = transpose4x4_bytes(relus, k);
      const int64_t row = slab * kTileRows + r;
      const int word = cb * 4 + (cg >> 2);
      if (row < p.B && word < p.w32) p.relubits[row * p.w32 + word] = rw;
    }
  }
  __syncthreads();

  // row offsets inside the tile and the tile total (warp 0)
  if (warp == 0) {
    const uint32_t v0 = s_rowcnt[2 * lane], v1 = s_rowcnt[2 * lane + 1];
    uint32_t incl = v0 + v1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    const uint32_t ex = incl - (v0 + v1);
    s_rowoff[2 * lane] = ex;
    s_rowoff[2 * lane + 1] = ex + v0;
    // row offsets travel with the keep bits: the dW kernel finds a row's values without a scan
    if (kMask != kMaskIndex) p.keepbits[(int64_t)tile * kTileWords + kBitWords + lane] = ex | ((ex + v0) << 16);
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    if (lane == 0) {
      s_total = total;
      const uint32_t gran = (total + kValueAlign - 1) / kValueAlign;
      // the first tile knows its prefix at once; the others publish their own count first
      if (kMask != kMaskIndex)
        store_status(p.status + tile, ((tile == 0 ? kFlagPrefix : kFlagAggregate) << kFlagShift) |
                                          pack_counts(gran, total));
    }
  }
  __syncthreads();

  // stage the kept values of the tile in (row, column) order
  const uint32_t total = s_total;
  const uint32_t padded = (total + kValueAlign - 1) / kValueAlign * kValueAlign;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int r = warp * 8 + it * 2 + half;
    uint32_t pos = s_rowoff[r] + ((pres >> (8 * it)) & 0xffu);
    const uint32_t m = (masks >> (8 * it)) & 0xffu;
    if (m != 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if ((m >> i) & 1u) {
          float w = p.scale;
          if (kReplace)   // weight of an entry drawn c times: fl32(c * (D / k)), then one product with the entry
            w = __fmul_rn((float)(((i < 4 ? mult[it].x : mult[it].y) >> (8 * (i & 3))) & 0xffu), p.scale);
          s_stage[pos++] = from_float<T>(__fmul_rn(elem(raw[it], i), w));
        }
      }
    }
  }
  if (tid < (int)(padded - total)) s_stage[total + tid] = from_float<T>(0.0f);

  if (kMask == kMaskIndex) {
    // the tile's place is known: no look-back
    if (tid == 0) {
      const int64_t base = p.offsets[tile];
      if (base + padded > p.capacity) {
        raise_status(p.dev_status, RAD_DEV_ECAPACITY);
        s_base = -1;
      } else {
        s_base = base;
      }
    }
  } else if (warp == 0) {
    // look-back (warp 0): sum the counts of earlier tiles until one with a known prefix is met
    uint64_t excl = 0;
    bool failed = false;
    if (tile != 0) {
      int64_t idx = (int64_t)tile - 1;
      bool done = false;
      while (!done) {
        const int64_t j = idx - lane;
        uint64_t w = kFlagPrefix << kFlagShift;          // before the first tile: prefix 0
        if (j >= 0) w = wait_status(p.status + j, p.wait_limit_ns);
        const uint64_t flag = w >> kFlagShift;
        if (__any_sync(0xffffffffu, flag == 0 || flag == kFlagPoison)) { failed = true; break; }
        const uint32_t pm = __ballot_sync(0xffffffffu, flag == kFlagPrefix);
        uint64_t contrib = w & kValueMask;
        if (pm != 0) {
          const int first = __ffs(pm) - 1;
          if (lane > first) contrib = 0;
          done = true;
        }
        excl += warp_sum_u64(contrib);
        idx -= 32;
      }
    }
    if (lane == 0) {
      if (failed) {
        store_status(p.status + tile, kFlagPoison << kFlagShift);   // later tiles stop waiting too
        raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
        s_base = -1;
      } else {
        const uint64_t incl = excl + pack_counts(padded / kValueAlign, total);
        if (tile != 0) store_status(p.status + tile, (kFlagPrefix << kFlagShift) | incl);
        const int64_t base = (int64_t)(excl >> 32) * kValueAlign;
        p.offsets[tile] = (uint32_t)base;
        if (tile == (uint32_t)p.ntiles - 1) {
          p.offsets[p.ntiles] = (uint32_t)((incl >> 32) * kValueAlign);
          p.nnz[0] = (int64_t)(incl & 0xffffffffu);
          p.nnz[1] = (int64_t)(incl >> 32) * kValueAlign;
        }
        if (base + padded > p.capacity) {
          raise_status(p.dev_status, RAD_DEV_ECAPACITY);
          s_base = -1;
        } else {
          s_base = base;
        }
      }
    }
  }
  __syncthreads();
  const int64_t base = s_base;
  if (base < 0) return;
  // 16-byte stores: base and padded are multiples of 8 elements
  constexpr int kPerVec = 16 / (int)sizeof(T);
  uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.values) + base);
  const uint4* src = reinterpret_cast<const uint4*>(s_stage);
  for (int i = tid; i < (int)(padded / kPerVec); i += 256) dst[i] = src[i];
}

// ---- same-sample ---------------------------------------------------------------------------------
struct SameParams {
  const void* A;
  int64_t lda;
  int64_t B, D;
  KeepThreshold T;
  float scale;
  uint32_t c2, c3;
  void* values;
  int64_t ld;
  uint32_t* keepbits;
  uint32_t* idx;
  int64_t* nnz;
  int32_t* dev_status;
};

// One CTA draws the D column decisions and writes the ascending kept-column list.
__global__ void __launch_bounds__(1024) same_mask_kernel(const SameParams p, const PhiloxKeys ks) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_running = 0;
  __syncthreads();
  const int64_t groups = (p.D + 31) / 32;
  for (int64_t g0 = 0; g0 < groups; g0 += 1024) {
    const int64_t g = g0 + tid;
    uint32_t m = 0;
    if (g < groups) {
      const int nvalid = (int)min((int64_t)32, p.D - g * 32);
      m = philox_keep32((uint32_t)g, 0u, p.c2, p.c3, ks, p.T) & (0xffffffffu >> (32 - nvalid));
      p.keepbits[g] = m;
    }
    const uint32_t c = __popc(m);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const uint32_t v = s_warp[lane];
      uint32_t wi = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      s_warp[lane] = wi - v;
    }
    __syncthreads();
    uint32_t pos = s_running + s_warp[warp] + incl - c;
    for (int i = 0; i < 32; ++i)
      if ((m >> i) & 1u) p.idx[pos++] = (uint32_t)(g * 32 + i);
    __syncthreads();
    if (tid == 1023) s_running = pos;   // last thread's end position is the running total
    __syncthreads();
  }
  if (tid == 0) {
    const int64_t k = s_running;
    p.nnz[0] = k;
    p.nnz[1] = k * p.B;
    if (k > p.ld) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
  }
}

// values[b, j] = A[b, idx[j]] * scale for j < k', zero up to ld.  One warp per row at a time.
template <typename T>
__global__ void __launch_bounds__(256) same_gather_kernel(const SameParams p, const float* colscale) {
  const int64_t k = min(p.nnz[0], p.ld);
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * 8;
  const T* A = static_cast<const T*>(p.A);
  T* out = static_cast<T*>(p.values);
  for (int64_t b = warp0; b < p.B; b += nwarps) {
    const T* rowp = A + b * p.lda;
    T* orow = out + b * p.ld;
    for (int64_t j = lane; j < p.ld; j += 32) {
      float v = 0.0f;
      if (j < k) {
        const uint32_t col = __ldg(p.idx + j);
        if (col < (uint32_t)p.D) v = __fmul_rn(to_float(rowp[col]), colscale != nullptr ? colscale[j] : p.scale);
        else raise_status(p.dev_status, RAD_DEV_EINTERNAL);
      }
      orow[j] = from_float<T>(v);
    }
  }
}

// The same gather with every access 16 bytes wide, for masks dense enough that most of a row is needed
// anyway (or when the 1-bit ReLU derivatives of the row are wanted, which need all of it): a warp brings a
// whole row of A into its own shared-memory buffer with asynchronous 16-byte copies, takes the ReLU bits
// from there, and writes the gathered row eight (bf16) or four (f32) outputs per lane and store.  The kept
// columns sit in shared memory as 16-bit numbers (D <= 65536).
template <typename T>
__global__ void __launch_bounds__(256) same_gather_rows_kernel(const SameParams p, uint32_t* relubits, int64_t w32, int warps) {
  extern __shared__ __align__(16) unsigned char s_dyn[];
  constexpr int kPer = 16 / (int)sizeof(T);
  const int64_t k = min(p.nnz[0], p.ld);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint16_t* s_idx = reinterpret_cast<uint16_t*>(s_dyn);
  const int64_t idx_bytes = (p.ld * 2 + 15) / 16 * 16;
  for (int64_t j = tid; j < p.ld; j += blockDim.x) {
    uint32_t col = 0;
    if (j < k) {
      col = __ldg(p.idx + j);
      if (col >= (uint32_t)p.D) { raise_status(p.dev_status, RAD_DEV_EINTERNAL); col = 0; }
    }
    s_idx[j] = (uint16_t)col;
  }
  __syncthreads();
  if (warp >= warps) return;
  const int64_t row_bytes = p.D * (int64_t)sizeof(T);
  T* s_row = reinterpret_cast<T*>(s_dyn + idx_bytes + (int64_t)warp * row_bytes);
  const uint32_t s_row_addr = (uint32_t)__cvta_generic_to_shared(s_row);
  const T* A = static_cast<const T*>(p.A);
  T* out = static_cast<T*>(p.values);
  const int64_t chunks = p.D / kPer;
  for (int64_t b = (int64_t)blockIdx.x * warps + warp; b < p.B; b += (int64_t)gridDim.x * warps) {
    const T* rowp = A + b * p.lda;
    for (int64_t c = lane; c < chunks; c += 32)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_row_addr + (uint32_t)(c * 16)), "l"(rowp + c * kPer) : "memory");
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    if (relubits != nullptr) {
      for (int64_t w = lane; w < w32; w += 32) {
        uint32_t m = positive32(s_row + w * 32);    // D is a multiple of 32 on this path
        relubits[b * w32 + w] = m;
      }
    }
    T* orow = out + b * p.ld;
    for (int64_t j0 = (int64_t)lane * kPer; j0 < p.ld; j0 += 32 * kPer) {
      __align__(16) T v[kPer];
#pragma unroll
      for (int e = 0; e < kPer; ++e) {
        const float a = j0 + e < k ? to_float(s_row[s_idx[j0 + e]]) : 0.0f;
        v[e] = from_float<T>(__fmul_rn(a, p.scale));
      }
      *reinterpret_cast<uint4*>(orow + j0) = *reinterpret_cast<const uint4*>(v);
    }
    __syncwarp();                                   // the row buffer is overwritten by the next row's copies
  }
}

// relubits[b, w] = bits of (A[b, 32w .. 32w+31] > 0).  One thread per output word.
template <typename T>
__global__ void __launch_bounds__(256) relu_bits_kernel(const T* A, int64_t lda, int64_t B, int64_t D,
                                                        int64_t w32, uint32_t* out) {
  const int64_t n = B * w32;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = i / w32, w = i % w32;
    const T* rowp = A + b * lda + w * 32;
    const int nv = (int)min((int64_t)32, D - w * 32);
    uint32_t m = 0;
    for (int c = 0; c < nv; ++c) m |= (to_float(rowp[c]) > 0.0f ? 1u : 0u) << c;
    out[i] = m;
  }
}

// ---- with-replacement law -------------------------------------------------------------------------
struct ReplaceParams {
  int64_t B, D, k;
  uint32_t c2, c3;
  uint8_t* counts;      // different-sample: B rows of ldc bytes
  int64_t ldc;
  int32_t* dev_status;
};

// One CTA per row: the k draws of the row land in a shared-memory histogram (a byte per column, four to
// a word), which is then written out as the row of the multiplicity matrix.
__global__ void __launch_bounds__(128) replace_counts_kernel(const ReplaceParams p, const PhiloxKeys ks) {
  extern __shared__ uint32_t s_hist[];
  const int64_t row = blockIdx.x;
  const int words = (int)(p.ldc / 4);
  for (int i = threadIdx.x; i < words; i += 128) s_hist[i] = 0;
  __syncthreads();
  const int64_t calls = (p.k + 3) / 4;
  for (int64_t c = threadIdx.x; c < calls; c += 128) {
    uint32_t w[4];
    philox4x32_10((uint32_t)c, (uint32_t)row, p.c2, p.c3, ks, w);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (4 * c + j < p.k) {
        const uint32_t col = __umulhi(w[j], (uint32_t)p.D);
        const uint32_t old = atomicAdd(&s_hist[col >> 2], 1u << (8 * (col & 3)));
        if (((old >> (8 * (col & 3))) & 0xffu) == 0xffu) raise_status(p.dev_status, RAD_DEV_EINTERNAL);   // a byte ran over
      }
    }
  }
  __syncthreads();
  uint32_t* out = reinterpret_cast<uint32_t*>(p.counts + row * p.ldc);
  for (int i = threadIdx.x; i < words; i += 128) out[i] = s_hist[i];
}

// Fixed-count law: one thread per row runs Floyd's subset sampling on a bitmap of its own in shared
// memory (step i needs the outcome of the steps before it, so a row cannot be split; the rows run side
// by side); the CTA then writes the rows of the multiplicity matrix, 0 or 1 per entry.
constexpr int kFixedRows = 64;
__global__ void __launch_bounds__(128) fixed_counts_kernel(const ReplaceParams p, const PhiloxKeys ks, int rows_per_cta,
                                                           int words) {
  extern __shared__ uint32_t s_bits[];            // rows_per_cta x words
  const int tid = threadIdx.x;
  for (int i = tid; i < rows_per_cta * words; i += 128) s_bits[i] = 0;
  __syncthreads();
  const int64_t row0 = (int64_t)blockIdx.x * rows_per_cta;
  if (tid < rows_per_cta && row0 + tid < p.B) {
    uint32_t* bm = s_bits + tid * words;
    for (int64_t c = 0; 4 * c < p.k; ++c) {
      uint32_t w[4];
      philox4x32_10((uint32_t)c, (uint32_t)(row0 + tid), p.c2, p.c3, ks, w);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        const int64_t i = 4 * c + jj;
        if (i < p.k) {
          const uint32_t j = (uint32_t)(p.D - p.k + i);
          const uint32_t t = __umulhi(w[jj], j + 1u);
          const uint32_t pick = ((bm[t >> 5] >> (t & 31)) & 1u) ? j : t;
          bm[pick >> 5] |= 1u << (pick & 31);
        }
      }
    }
  }
  __syncthreads();
  const int quads = (int)(p.ldc / 4);             // four entries, a byte each, per output word
  for (int r = 0; r < rows_per_cta && row0 + r < p.B; ++r) {
    uint32_t* out = reinterpret_cast<uint32_t*>(p.counts + (row0 + r) * p.ldc);
    for (int q = tid; q < quads; q += 128) {
      const uint32_t nib = (q >> 3) < words ? (s_bits[r * words + (q >> 3)] >> (4 * (q & 7))) & 0xfu : 0u;
      out[q] = (nib & 1u) | ((nib & 2u) << 7) | ((nib & 4u) << 14) | ((nib & 8u) << 21);
    }
  }
}

constexpr int kSameFixedMaxD = 262144;   // same-sample fixed-count law: the bitmap sits in shared memory
struct SameReplaceParams {
  int64_t D, k;
  uint32_t c2, c3;
  float scale;          // D / k
  int32_t fixed;        // 1: k distinct columns by Floyd's sampling instead of k draws with replacement
  uint32_t* hist;       // D words of scratch
  float* colscale;      // weight of kept column j (D floats of scratch)
};

// Same-sample: one set of k draws for the layer.  One CTA: histogram in global scratch, then the
// ascending list of the columns that were hit, their weights and the keep-bit words.
__global__ void __launch_bounds__(1024) same_replace_mask_kernel(const SameParams p, const SameReplaceParams r,
                                                                 const PhiloxKeys ks) {
  __shared__ uint32_t s_warp[32];
  __shared__ uint32_t s_running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int64_t i = tid; i < p.D; i += 1024) r.hist[i] = 0;
  if (tid == 0) s_running = 0;
  __syncthreads();
  if (r.fixed) {
    // Floyd's subset sampling is sequential: one thread, bitmap in shared memory (D <= kSameFixedMaxD)
    __shared__ uint32_t s_bits[kSameFixedMaxD / 32];
    for (int i = tid; i < kSameFixedMaxD / 32; i += 1024) s_bits[i] = 0;
    __syncthreads();
    if (tid == 0) {
      for (int64_t c = 0; 4 * c < r.k; ++c) {
        uint32_t w[4];
        philox4x32_10((uint32_t)c, 0u, r.c2, r.c3, ks, w);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int64_t i = 4 * c + jj;
          if (i < r.k) {
            const uint32_t j = (uint32_t)(p.D - r.k + i);
            const uint32_t t = __umulhi(w[jj], j + 1u);
            const uint32_t pick = ((s_bits[t >> 5] >> (t & 31)) & 1u) ? j : t;
            s_bits[pick >> 5] |= 1u << (pick & 31);
          }
        }
      }
    }
    __syncthreads();
    for (int64_t i = tid; i < p.D; i += 1024) r.hist[i] = (s_bits[i >> 5] >> (i & 31)) & 1u;
  } else {
    const int64_t calls = (r.k + 3) / 4;
    for (int64_t c = tid; c < calls; c += 1024) {
      uint32_t w[4];
      philox4x32_10((uint32_t)c, 0u, r.c2, r.c3, ks, w);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (4 * c + j < r.k) atomicAdd(&r.hist[__umulhi(w[j], (uint32_t)p.D)], 1u);
    }
  }
  __syncthreads();
  for (int64_t d0 = 0; d0 < p.D; d0 += 1024) {
    const int64_t d = d0 + tid;
    const uint32_t c = d < p.D ? r.hist[d] : 0u;
    const uint32_t kept = c != 0 ? 1u : 0u;
    const uint32_t word = __ballot_sync(0xffffffffu, kept != 0);
    if (lane == 0 && d < p.D) p.keepbits[d >> 5] = word;
    const uint32_t before = __popc(word & ((1u << lane) - 1u));
    if (lane == 31) s_warp[warp] = before + kept;
    __syncthreads();
    if (warp == 0) {
      const uint32_t v = s_warp[lane];
      uint32_t wi = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      s_warp[lane] = wi - v;
    }
    __syncthreads();
    const uint32_t pos = s_running + s_warp[warp] + before;
    if (kept) {
      p.idx[pos] = (uint32_t)d;
      r.colscale[pos] = __fmul_rn((float)c, r.scale);
    }
    __syncthreads();
    if (tid == 1023) s_running = pos + kept;   // last thread's end position is the running total
    __syncthreads();
  }
  if (tid == 0) {
    const int64_t k = s_running;
    p.nnz[0] = k;
    p.nnz[1] = k * p.B;
    if (k > p.ld) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
  }
}

// The look-back's wait on a status word that nobody publishes (a word of the probe's own that stays zero):
// it gives up after `limit_ns` and the status word reports the timeout, as the store kernels do.
__device__ uint64_t g_probe_status_word;
__global__ void wait_probe_lookback_kernel(uint64_t limit_ns, int32_t* dev_status) {
  const uint64_t w = wait_status(&g_probe_status_word, limit_ns);
  if ((w >> kFlagShift) == 0) raise_status(dev_status, RAD_DEV_ETIMEOUT);
}

constexpr int kPipelinedMinTiles = 2048;
int g_store_kernel = RAD_STORE_KERNEL_AUTO;

// Values (and ReLU bits) into a store whose index part is in place: the persistent kernel's loader and
// compaction warps where they apply (many tiles, aligned input), else one CTA per tile.  p.ticket: 256 bytes.
int launch_store_fill(const StoreParams& p, const PhiloxKeys& ks, int dtype, double keep_fraction, cudaStream_t s) {
  if (g_store_kernel == RAD_STORE_KERNEL_PIPELINED ||
      (g_store_kernel == RAD_STORE_KERNEL_AUTO && p.ntiles >= kPipelinedMinTiles && keep_fraction <= 0.5)) {
    RAD_CUDA_TRY(cudaMemsetAsync(p.ticket, 0, 256, s));
    const int rc = launch_store_pipelined(p, ks, dtype, s, true);
    if (rc != RAD_EUNSUPPORTED) return rc;
  }
  count_launch();
  if (dtype == RAD_BF16)
    store_different_kernel<bf16, kMaskIndex><<<p.ntiles, 256, 0, s>>>(p, ks);
  else
    store_different_kernel<float, kMaskIndex><<<p.ntiles, 256, 0, s>>>(p, ks);
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}

// The persistent TMA-fed kernel where the input can be described by a tensor map, else the generic one
// (same layout, same scratch: a claim counter and one status word per tile or chunk of tiles).
int launch_store_different(const StoreParams& p, const PhiloxKeys& ks, int dtype, uint32_t T, cudaStream_t s) {
  // The pipelined kernel pays off where there are many tiles per SM and most entries are dropped: its
  // per-entry staging loop is slower than the generic kernel's for dense masks, and a CTA works
  // through a chunk of tiles one after the other, which only adds latency to a small problem.
  const bool pipelined = p.counts != nullptr ? false : g_store_kernel == RAD_STORE_KERNEL_PIPELINED ||
                         (g_store_kernel == RAD_STORE_KERNEL_AUTO && p.ntiles >= kPipelinedMinTiles && T <= kLaneRange / 2);
  const int rc = pipelined ? launch_store_pipelined(p, ks, dtype, s) : RAD_EUNSUPPORTED;
  if (rc != RAD_EUNSUPPORTED) return rc;
  count_launch();
  if (p.counts != nullptr) {
    if (dtype == RAD_BF16)
      store_different_kernel<bf16, kMaskCounts><<<p.ntiles, 256, 0, s>>>(p, ks);
    else
      store_different_kernel<float, kMaskCounts><<<p.ntiles, 256, 0, s>>>(p, ks);
  } else if (dtype == RAD_BF16) {
    store_different_kernel<bf16, kMaskDraw><<<p.ntiles, 256, 0, s>>>(p, ks);
  } else {
    store_different_kernel<float, kMaskDraw><<<p.ntiles, 256, 0, s>>>(p, ks);
  }
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}

int64_t status_bytes(int64_t B, int64_t D) {
  const int64_t ntiles = ceil_div(B, kTileRows) * ceil_div(D, kTileCols);
  return round_up(ntiles * 8 + 256, 256);
}
int64_t counts_ld(int64_t D) { return round_up(D, 16); }

// different-sample: claim counter and look-back status words, then (with-replacement law) the multiplicity
// matrix; same-sample with replacement: 256 bytes, a histogram word and a weight per column.
int64_t store_workspace_bytes(int variant, int64_t B, int64_t D, int law = RAD_LAW_BERNOULLI) {
  if (variant == RAD_SAME_SAMPLE) return law != RAD_LAW_BERNOULLI ? 256 + round_up(8 * D, 256) : 256;
  return status_bytes(B, D) + (law != RAD_LAW_BERNOULLI ? round_up(B * counts_ld(D), 256) : 0);
}

constexpr int64_t kMaxCountsRowBytes = 200 * 1024;   // a row's histogram has to fit shared memory

}  // namespace
}  // namespace rad

namespace rad {
int launch_wait_probe_lookback(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s) {
  count_launch();
  wait_probe_lookback_kernel<<<1, 32, 0, s>>>(limit_ns, dev_status);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}
int launch_relu_bits(int dtype, const void* A, int64_t lda, int64_t B, int64_t D, uint32_t* relubits, cudaStream_t s) {
  const int64_t w32 = ceil_div(D, 32), n = B * w32;
  const int g2 = (int)std::min<int64_t>(ceil_div(n, 256), 148 * 16);
  count_launch();
  if (dtype == RAD_BF16)
    relu_bits_kernel<bf16><<<g2, 256, 0, s>>>(static_cast<const bf16*>(A), lda, B, D, w32, relubits);
  else
    relu_bits_kernel<float><<<g2, 256, 0, s>>>(static_cast<const float*>(A), lda, B, D, w32, relubits);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}
}  // namespace rad

using namespace rad;

extern "C" int rad_set_store_kernel(int32_t which) {
  if (which != RAD_STORE_KERNEL_AUTO && which != RAD_STORE_KERNEL_GENERIC && which != RAD_STORE_KERNEL_PIPELINED)
    return RAD_EINVAL;
  const int prev = g_store_kernel;
  g_store_kernel = which;
  return prev;
}

extern "C" uint32_t rad_keep_threshold(float p) { return keep_threshold_host(p); }
extern "C" float rad_effective_p(float p) { return (float)keep_threshold_host(p) / (float)kLaneRange; }
extern "C" float rad_scale(float p) {
  const uint32_t T = keep_threshold_host(p);
  return T == 0 ? 0.0f : (float)kLaneRange / (float)T;
}

extern "C" int64_t rad_draws_per_row(float fraction, int64_t D) { return draws_per_row_host(fraction, D); }
extern "C" float rad_replace_scale(float fraction, int64_t D) {
  const int64_t k = draws_per_row_host(fraction, D);
  return k == 0 ? 0.0f : (float)D / (float)k;
}

extern "C" int rad_store_size_query(int32_t variant, int32_t dtype, int64_t B, int64_t D, float p,
                                    rad_store_sizes* out) {
  return rad_store_size_query_law(variant, dtype, RAD_LAW_BERNOULLI, B, D, p, out);
}

extern "C" int rad_store_size_query_law(int32_t variant, int32_t dtype, int32_t law, int64_t B, int64_t D, float p,
                                        rad_store_sizes* out) {
  if (out == nullptr || B <= 0 || D <= 0) return RAD_EINVAL;
  if (dtype != RAD_F32 && dtype != RAD_BF16) return RAD_EINVAL;
  if (variant == RAD_PROJECT) {
    // a dense B x ld block (ld: k rounded up to 64 columns, zero beyond k); no index data
    const int64_t k = draws_per_row_host(p, D);
    if (k == 0) return RAD_EINVAL;
    const int64_t ld = project_ld(k);
    out->values_ld_worst = out->values_ld_typical = ld;
    out->values_worst = out->values_typical = B * ld;
    out->keepbits_words = out->offsets_words = 0;
    out->relubits_words = B * ceil_div(D, 32);
    out->workspace_bytes = project_store_workspace(dtype, D, ld);
    return RAD_OK;
  }
  if (variant == RAD_ROWS_SAMPLE) {
    // B x ld values and B x ld 16-bit column numbers (ld: k rounded up to 8 columns); exact, whatever the key
    const int64_t k = draws_per_row_host(p, D);
    if (k == 0 || law != RAD_LAW_FIXED) return RAD_EINVAL;
    if (D > 65536) return RAD_EUNSUPPORTED;
    const int64_t ld = round_up(k, 8);
    out->values_ld_worst = out->values_ld_typical = ld;
    out->values_worst = out->values_typical = B * ld;
    out->keepbits_words = B * ld / 2;
    out->offsets_words = 0;
    out->relubits_words = B * ceil_div(D, 32);
    out->workspace_bytes = 256;
    return RAD_OK;
  }
  if (variant == RAD_REDRAWN_SAMPLE) {
    // the different-sample store without its keep bits; the index of one layer lives in the workspace
    if (law != RAD_LAW_BERNOULLI && law != RAD_LAW_FIXED) return RAD_EINVAL;
    const int rc = rad_store_size_query_law(RAD_DIFFERENT_SAMPLE, dtype, law, B, D, p, out);
    if (rc != RAD_OK) return rc;
    out->workspace_bytes = redrawn_index_bytes(B, D) + round_up(out->workspace_bytes, 256);
    out->keepbits_words = 0;
    return RAD_OK;
  }
  if (variant != RAD_DIFFERENT_SAMPLE && variant != RAD_SAME_SAMPLE) return RAD_EINVAL;
  if (law != RAD_LAW_BERNOULLI && law != RAD_LAW_REPLACE && law != RAD_LAW_FIXED) return RAD_EINVAL;
  const uint32_t T = keep_threshold_host(p);
  if (T == 0) return RAD_EINVAL;
  if ((double)B * (double)D >= 4294967296.0 * 0.75) return RAD_EINVAL;   // 32-bit tile offsets
  rad_store probe = {};
  probe.law = law; probe.p = p; probe.D = D;
  // share of kept entries; the count of distinct columns among k draws varies less than a Binomial
  // of the same mean, so the Binomial band below covers it
  const double pe = store_keep_fraction(&probe);
  const int64_t w32 = ceil_div(D, 32);
  out->relubits_words = B * w32;
  if (variant == RAD_DIFFERENT_SAMPLE) {
    const int64_t ntiles = ceil_div(B, kTileRows) * ceil_div(D, kTileCols);
    const double n = (double)B * (double)D;
    const int64_t pad = ntiles * (kValueAlign - 1);
    out->values_worst = B * D + pad;
    const double typ = n * pe + 8.0 * sqrt(n * pe * (1.0 - pe)) + 64.0;
    out->values_typical = round_up((int64_t)fmin(typ, n) + pad, kValueAlign);
    if (out->values_typical > out->values_worst) out->values_typical = out->values_worst;
    out->values_ld_worst = out->values_ld_typical = 0;
    out->keepbits_words = ntiles * kTileWords;
    out->offsets_words = ntiles + 1;
  } else {
    const double n = (double)D;
    const int64_t ldw = round_up(D, 64);
    int64_t ldt = round_up((int64_t)(n * pe + 8.0 * sqrt(n * pe * (1.0 - pe)) + 8.0), 64);
    if (ldt > ldw) ldt = ldw;
    out->values_ld_worst = ldw;
    out->values_ld_typical = ldt;
    out->values_worst = B * ldw;
    out->values_typical = B * ldt;
    out->keepbits_words = w32;
    out->offsets_words = D;
  }
  out->workspace_bytes = store_workspace_bytes(variant, B, D, law);
  return RAD_OK;
}

extern "C" int rad_linear_forward_store(const void* A, int64_t lda, const rad_store* st, void* workspace,
                                        int64_t workspace_bytes, int32_t* dev_status, void* stream) {
  if (A == nullptr || st == nullptr) return RAD_EINVAL;
  if (st->B <= 0 || st->D <= 0 || lda < st->D) return RAD_EINVAL;
  if (st->dtype != RAD_F32 && st->dtype != RAD_BF16) return RAD_EINVAL;
  if (st->variant == RAD_PROJECT) {
    const int rcp = check_device();
    return rcp != RAD_OK ? rcp : project_forward_store(A, lda, st, workspace, workspace_bytes, dev_status, stream);
  }
  if (st->variant == RAD_ROWS_SAMPLE) {
    const int rcr = check_device();
    return rcr != RAD_OK ? rcr : rows_forward_store(A, lda, st, dev_status, static_cast<cudaStream_t>(stream));
  }
  if (st->variant == RAD_REDRAWN_SAMPLE) {
    // the index part goes to the head of the workspace, the different-sample store does the rest
    if (st->law != RAD_LAW_BERNOULLI && st->law != RAD_LAW_FIXED) return RAD_EINVAL;
    const int64_t head = redrawn_index_bytes(st->B, st->D);
    if (workspace == nullptr || workspace_bytes < head) return RAD_EWORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return RAD_EINVAL;
    rad_store full = *st;
    full.variant = RAD_DIFFERENT_SAMPLE;
    full.keepbits = static_cast<uint32_t*>(workspace);
    return rad_linear_forward_store(A, lda, &full, static_cast<char*>(workspace) + head, workspace_bytes - head, dev_status,
                                    stream);
  }
  if (st->variant != RAD_DIFFERENT_SAMPLE && st->variant != RAD_SAME_SAMPLE) return RAD_EINVAL;
  if (st->values == nullptr || st->keepbits == nullptr || st->offsets == nullptr || st->nnz == nullptr)
    return RAD_EINVAL;
  const uint32_t T = keep_threshold_host(st->p);
  if (T == 0) return RAD_EINVAL;
  if (st->law != RAD_LAW_BERNOULLI && st->law != RAD_LAW_REPLACE && st->law != RAD_LAW_FIXED) return RAD_EINVAL;
  if ((double)st->B * (double)st->D >= 4294967296.0 * 0.75) return RAD_EINVAL;
  if (((uintptr_t)st->values & 15) != 0) return RAD_EUNSUPPORTED;
  const bool replace = st->law != RAD_LAW_BERNOULLI;      // mask and weights come from a multiplicity matrix
  const bool fixed = st->law == RAD_LAW_FIXED;
  const int64_t k = replace ? draws_per_row_host(st->p, st->D) : 0;
  if (replace && st->variant == RAD_DIFFERENT_SAMPLE && counts_ld(st->D) > kMaxCountsRowBytes) return RAD_EUNSUPPORTED;
  if (fixed && st->variant == RAD_SAME_SAMPLE && st->D > kSameFixedMaxD) return RAD_EUNSUPPORTED;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t esz = st->dtype == RAD_BF16 ? 2 : 4;
  const PhiloxKeys ks = philox_expand_key(st->seed);
  const int64_t w32 = ceil_div(st->D, 32);
  // Bernoulli: 1 / p_eff; with replacement: D / k, the weight of a column drawn once
  const float scale = replace ? (float)st->D / (float)k : (float)kLaneRange / (float)T;
  const int64_t need = store_workspace_bytes(st->variant, st->B, st->D, st->law);
  if (need > 256 || st->variant == RAD_DIFFERENT_SAMPLE) {
    if (workspace == nullptr || workspace_bytes < need) return RAD_EWORKSPACE;
    if (((uintptr_t)workspace & 15) != 0) return RAD_EINVAL;
  }

  if (st->variant == RAD_DIFFERENT_SAMPLE) {
    StoreParams p;
    p.A = A; p.lda = lda; p.B = st->B; p.D = st->D;
    p.ncb = (int32_t)ceil_div(st->D, kTileCols);
    p.ntiles = (int32_t)(ceil_div(st->B, kTileRows) * p.ncb);
    p.T = make_keep_threshold(T); p.scale = scale;
    p.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE); p.c3 = st->step;
    p.values = st->values; p.capacity = st->values_capacity;
    p.keepbits = st->keepbits; p.offsets = st->offsets; p.nnz = st->nnz;
    p.relubits = st->relubits; p.w32 = (int32_t)w32;
    p.ticket = static_cast<uint32_t*>(workspace);
    p.status = reinterpret_cast<uint64_t*>(static_cast<char*>(workspace) + 256);
    p.dev_status = dev_status;
    p.vec_ok = (((uintptr_t)A & 15) == 0 && (lda * esz) % 16 == 0) ? 1 : 0;
    p.counts = nullptr; p.ldc = 0;
    p.wait_limit_ns = wait_limit_ns();
    if (fixed) {
      // exactly k columns per row: the index part comes from the key alone (Floyd's sampling, a warp per row),
      // then one CTA per tile places the values; no multiplicity matrix, no look-back
      rc = launch_fixed_index(st, true, dev_status, s);
      if (rc == RAD_OK) return launch_store_fill(p, ks, st->dtype, store_keep_fraction(st), s);
      if (rc != RAD_EUNSUPPORTED) return rc;      // rows too long for shared memory: the multiplicity matrix below
    }
    if (replace && !fixed) {
      // the same road for k draws with replacement: index part from the key alone, values placed with the
      // weight of one draw, the few entries drawn more than once written again with theirs (their list takes
      // the place of the multiplicity matrix in the workspace)
      uint32_t* extras = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + status_bytes(st->B, st->D));
      rc = launch_replace_index(st, extras, true, dev_status, s);
      if (rc == RAD_OK) {
        rc = launch_store_fill(p, ks, st->dtype, store_keep_fraction(st), s);
        if (rc != RAD_OK) return rc;
        return launch_replace_extras(A, lda, st, extras, s);
      }
      if (rc != RAD_EUNSUPPORTED) return rc;      // many draws or long rows: the multiplicity matrix below
    }
    RAD_CUDA_TRY(cudaMemsetAsync(workspace, 0, (size_t)status_bytes(st->B, st->D), s));
    if (replace) {
      // first the multiplicities of every row, then the generic kernel with the mask and the weights
      // taken from them
      ReplaceParams rp;
      rp.B = st->B; rp.D = st->D; rp.k = k;
      rp.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE, st->law); rp.c3 = st->step;
      rp.counts = reinterpret_cast<uint8_t*>(static_cast<char*>(workspace) + status_bytes(st->B, st->D));
      rp.ldc = counts_ld(st->D);
      rp.dev_status = dev_status;
      count_launch();
      if (fixed) {
        const int words = (int)ceil_div(st->D, 32);
        const int rows = (int)std::max<int64_t>(1, std::min<int64_t>(kFixedRows, kMaxCountsRowBytes / (4 * (int64_t)words)));
        const size_t smem = (size_t)rows * words * 4;
        if (smem > 48 * 1024)
          RAD_CUDA_TRY(cudaFuncSetAttribute(fixed_counts_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kMaxCountsRowBytes));
        fixed_counts_kernel<<<(unsigned)ceil_div(st->B, rows), 128, smem, s>>>(rp, ks, rows, words);
      } else {
        if (rp.ldc > 48 * 1024)
          RAD_CUDA_TRY(cudaFuncSetAttribute(replace_counts_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)kMaxCountsRowBytes));
        replace_counts_kernel<<<(unsigned)st->B, 128, (size_t)rp.ldc, s>>>(rp, ks);
      }
      RAD_CUDA_TRY(cudaGetLastError());
      p.counts = rp.counts; p.ldc = rp.ldc;
    }
    return launch_store_different(p, ks, st->dtype, T, s);
  }

  if (st->values_ld <= 0 || st->values_ld % 8 != 0 || st->values_capacity < st->B * st->values_ld)
    return RAD_EINVAL;
  SameParams p;
  p.A = A; p.lda = lda; p.B = st->B; p.D = st->D; p.T = make_keep_threshold(T); p.scale = scale;
  p.c2 = counter_word2(st->layer, RAD_SAME_SAMPLE); p.c3 = st->step;
  p.values = st->values; p.ld = st->values_ld; p.keepbits = st->keepbits; p.idx = st->offsets;
  p.nnz = st->nnz; p.dev_status = dev_status;
  const float* colscale = nullptr;
  count_launch(2);
  if (replace) {
    SameReplaceParams r;
    r.D = st->D; r.k = k;
    r.c2 = counter_word2(st->layer, RAD_SAME_SAMPLE, st->law); r.c3 = st->step;
    r.scale = scale;
    r.fixed = fixed ? 1 : 0;
    r.hist = reinterpret_cast<uint32_t*>(static_cast<char*>(workspace) + 256);
    r.colscale = reinterpret_cast<float*>(static_cast<char*>(workspace) + 256 + 4 * st->D);
    colscale = r.colscale;
    same_replace_mask_kernel<<<1, 1024, 0, s>>>(p, r, ks);
  } else {
    same_mask_kernel<<<1, 1024, 0, s>>>(p, ks);
  }
  // Dense masks (most 32-byte sectors of a row hold a kept column) and calls that also want the ReLU bits take
  // the row-staging kernel; sparse masks without ReLU bits keep the gather that skips the sectors it does not need.
  {
    const int64_t row_bytes = st->D * (int64_t)esz, idx_bytes = round_up(st->values_ld * 2, 16);
    const int64_t smem_budget = 200 * 1024;
    const int warps = (int)std::min<int64_t>(8, row_bytes > 0 ? (smem_budget - idx_bytes) / row_bytes : 0);
    const bool rows_ok = colscale == nullptr && st->D % 32 == 0 && st->D <= 65536 && warps >= 2 &&
                         ((uintptr_t)A & 15) == 0 && (lda * esz) % 16 == 0 && ((uintptr_t)st->values & 15) == 0;
    const double pe = store_keep_fraction(st);
    if (rows_ok && (st->relubits != nullptr || pe >= 0.15)) {
      const size_t smem = (size_t)(idx_bytes + warps * row_bytes);
      static int sms = 0;
      if (sms == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
          sms = 148;
      }
      const int grid_r = (int)std::min<int64_t>(ceil_div(st->B, warps), sms);
      if (st->dtype == RAD_BF16) {
        RAD_CUDA_TRY(cudaFuncSetAttribute(same_gather_rows_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_budget));
        same_gather_rows_kernel<bf16><<<grid_r, 256, smem, s>>>(p, st->relubits, w32, warps);
      } else {
        RAD_CUDA_TRY(cudaFuncSetAttribute(same_gather_rows_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_budget));
        same_gather_rows_kernel<float><<<grid_r, 256, smem, s>>>(p, st->relubits, w32, warps);
      }
      RAD_CUDA_TRY(cudaGetLastError());
      return RAD_OK;
    }
  }
  const int grid = (int)std::min<int64_t>(ceil_div(st->B, 8), 148 * 8);
  if (st->dtype == RAD_BF16)
    same_gather_kernel<bf16><<<grid, 256, 0, s>>>(p, colscale);
  else
    same_gather_kernel<float><<<grid, 256, 0, s>>>(p, colscale);
  if (st->relubits != nullptr) {
    const int64_t n = st->B * w32;
    const int g2 = (int)std::min<int64_t>(ceil_div(n, 256), 148 * 16);
    count_launch();
    if (st->dtype == RAD_BF16)
      relu_bits_kernel<bf16><<<g2, 256, 0, s>>>(static_cast<const bf16*>(A), lda, st->B, st->D, w32, st->relubits);
    else
      relu_bits_kernel<float><<<g2, 256, 0, s>>>(static_cast<const float*>(A), lda, st->B, st->D, w32, st->relubits);
  }
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}

// ---- the store without a caller-provided workspace ------------------------------------------------
// Scratch of the different-sample kernel for callers that cannot allocate: a claim counter (first
// 256 bytes) and one status word per tile.  The name below is only a handle in host code; the
// device address is looked up once per device.
static __device__ __align__(256) unsigned char g_static_store_scratch[256 + 8 * RAD_STATIC_STORE_MAX_TILES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_ptr[kMaxDevices] = {};

int static_scratch_address(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RAD_ECUDA;
  if (dev < 0 || dev >= kMaxDevices) return RAD_EUNSUPPORTED;
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_store_scratch) != cudaSuccess || ptr == nullptr) return RAD_ECUDA;
    g_static_scratch_ptr[dev] = ptr;
  }
  *out = g_static_scratch_ptr[dev];
  return RAD_OK;
}
}  // namespace

extern "C" int rad_linear_forward_store_static(const void* A, int64_t lda, const rad_store* st,
                                               int32_t* dev_status, void* stream) {
  if (A == nullptr || st == nullptr) return RAD_EINVAL;
  if (st->B <= 0 || st->D <= 0 || lda < st->D) return RAD_EINVAL;
  if (st->variant != RAD_DIFFERENT_SAMPLE || st->law != RAD_LAW_BERNOULLI) return RAD_EUNSUPPORTED;
  if (st->dtype != RAD_F32 && st->dtype != RAD_BF16) return RAD_EINVAL;
  if (st->values == nullptr || st->keepbits == nullptr || st->offsets == nullptr || st->nnz == nullptr)
    return RAD_EINVAL;
  const uint32_t T = keep_threshold_host(st->p);
  if (T == 0) return RAD_EINVAL;
  if ((double)st->B * (double)st->D >= 4294967296.0 * 0.75) return RAD_EINVAL;
  if (((uintptr_t)st->values & 15) != 0) return RAD_EUNSUPPORTED;
  const int64_t ntiles = ceil_div(st->B, kTileRows) * ceil_div(st->D, kTileCols);
  if (ntiles > RAD_STATIC_STORE_MAX_TILES) return RAD_ELIMIT;
  int rc = check_device();
  if (rc != RAD_OK) return rc;
  void* scratch = nullptr;
  rc = static_scratch_address(&scratch);
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t esz = st->dtype == RAD_BF16 ? 2 : 4;
  const PhiloxKeys ks = philox_expand_key(st->seed);
  StoreParams p;
  p.A = A; p.lda = lda; p.B = st->B; p.D = st->D;
  p.ncb = (int32_t)ceil_div(st->D, kTileCols);
  p.ntiles = (int32_t)ntiles;
  p.T = make_keep_threshold(T); p.scale = (float)kLaneRange / (float)T;
  p.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE); p.c3 = st->step;
  p.values = st->values; p.capacity = st->values_capacity;
  p.keepbits = st->keepbits; p.offsets = st->offsets; p.nnz = st->nnz;
  p.relubits = st->relubits; p.w32 = (int32_t)ceil_div(st->D, 32);
  p.ticket = static_cast<uint32_t*>(scratch);
  p.status = reinterpret_cast<uint64_t*>(static_cast<char*>(scratch) + 256);
  p.dev_status = dev_status;
  p.vec_ok = (((uintptr_t)A & 15) == 0 && (lda * esz) % 16 == 0) ? 1 : 0;
  p.counts = nullptr; p.ldc = 0;
  p.wait_limit_ns = wait_limit_ns();
  // the array keeps what the last call left: the counter and this call's status words start at zero
  RAD_CUDA_TRY(cudaMemsetAsync(scratch, 0, 256 + 8 * (size_t)ntiles, s));
  return launch_store_different(p, ks, st->dtype, T, s);
}
