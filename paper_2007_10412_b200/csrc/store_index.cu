// Index part of a different-sample store from the key alone (Sec. 3.2: the random P is independent of the
// data; Sec. 4.2: it is drawn per layer input).  The keep decision of entry (b, d) depends on (seed, layer,
// step, b, d) only, so keep bits, row offsets, tile offsets and the kept count can be produced without
// reading the layer input, before that input exists.  The forward GEMM of the layer that produces the input
// then drops the kept values into place from its epilogue (tc.cu), and a caller learns the exact size of a
// store before it allocates `values`.
//
//   store_index_kernel   one tile (64 x 128 entries) per warp and turn: draw and write the keep-bit words,
//                        in-tile row offsets from warp scans, exact kept count of the tile into offsets[tile]
//   offsets_scan_kernel  one CTA turns the counts into padded exclusive prefixes in place and writes nnz
//
// Layout and bits are those of the one-pass store kernels.
#include <algorithm>

#include "common.cuh"

namespace rad {
namespace {

struct IndexParams {
  int64_t B, D;
  int32_t ncb, ntiles;
  KeepThreshold T;
  uint32_t c2, c3;
  uint32_t* keepbits;
  uint32_t* offsets;
  int64_t* nnz;
  int64_t capacity;     // elements of `values` the caller holds; < 0: not checked
  int32_t* dev_status;
};

// One warp per tile and turn, no CTA-wide step: lane l draws words l, l + 32, ... of the tile (word t = row
// t / 4, columns 32 (t % 4) ..), so a warp's stores are contiguous and a warp scan per turn, carried over
// the eight turns, gives every row its offset in (row, column) order.
constexpr int kIndexWarps = 4;
__global__ void __launch_bounds__(32 * kIndexWarps) store_index_kernel(const IndexParams p, const PhiloxKeys ks) {
  const int lane = threadIdx.x & 31;
  const uint32_t warp0 = blockIdx.x * kIndexWarps + (threadIdx.x >> 5), nwarps = gridDim.x * kIndexWarps;
  const uint32_t nrows = (uint32_t)p.B, ncols = (uint32_t)p.D, ncb = (uint32_t)p.ncb;
  const int w = lane & 3;
  for (uint32_t tile = warp0; tile < (uint32_t)p.ntiles; tile += nwarps) {
    const uint32_t slab = tile / ncb, cb = tile - slab * ncb;
    const uint32_t col0 = cb * kTileCols + 32u * w;
    uint32_t* tw = p.keepbits + (int64_t)tile * kTileWords;
    uint32_t base = 0;
#pragma unroll 2
    for (int i = 0; i < kBitWords / 32; ++i) {
      const int r = i * 8 + (lane >> 2);
      const uint32_t row = slab * kTileRows + r;
      uint32_t m = 0;
      if (row < nrows && col0 < ncols) {
        m = philox_keep32(col0 >> 5, row, p.c2, p.c3, ks, p.T);
        const uint32_t nv = ncols - col0;
        if (nv < 32) m &= (1u << nv) - 1u;
      }
      tw[i * 32 + lane] = m;
      const uint32_t c = __popc(m);
      uint32_t incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (w == 0) reinterpret_cast<uint16_t*>(tw + kBitWords)[r] = (uint16_t)(base + incl - c);
      base += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) p.offsets[tile] = base;
  }
}

// offsets[t] holds the exact kept count of tile t on entry and the first element of tile t in `values` on
// exit (every tile padded to a multiple of kValueAlign); offsets[ntiles] = elements used.  One CTA, 16384
// tiles per round; a thread takes 16 consecutive tiles (four 16-byte loads and stores where `offsets` is
// 16-byte aligned), adds them up locally, and one warp scan plus one pass over the warp sums places them.
constexpr int kScanPer = 16;
__global__ void __launch_bounds__(1024) offsets_scan_kernel(const IndexParams p, int vec) {
  __shared__ uint64_t s_warp[32];                   // padded sum in the high half, exact sum in the low half
  __shared__ uint64_t s_carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  const int64_t ntiles = p.ntiles;
  for (int64_t r0 = 0; r0 < ntiles; r0 += 1024 * kScanPer) {
    const int64_t t0 = r0 + (int64_t)tid * kScanPer;
    const bool whole = vec != 0 && t0 + kScanPer <= ntiles;
    uint32_t c[kScanPer];
    if (whole) {
#pragma unroll
      for (int i = 0; i < kScanPer; i += 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(p.offsets + t0 + i);
        c[i] = q.x; c[i + 1] = q.y; c[i + 2] = q.z; c[i + 3] = q.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < kScanPer; ++i) c[i] = t0 + i < ntiles ? p.offsets[t0 + i] : 0u;
    }
    // a round holds at most 16384 * 8192 entries: 32 bits each for the padded and the exact sum
    uint64_t mine = 0;
#pragma unroll
    for (int i = 0; i < kScanPer; ++i)
      mine += ((uint64_t)((c[i] + kValueAlign - 1) / kValueAlign * kValueAlign) << 32) | c[i];
    uint64_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint64_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    const uint64_t carry = s_carry;
    uint64_t before = incl - mine, round_total = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const uint64_t t = s_warp[i];
      if (i < warp) before += t;
      round_total += t;
    }
    uint32_t at = (uint32_t)((carry >> 32) + (before >> 32));     // the padded total stays below 2^32
    uint32_t o[kScanPer];
#pragma unroll
    for (int i = 0; i < kScanPer; ++i) {
      o[i] = at;
      at += (c[i] + kValueAlign - 1) / kValueAlign * kValueAlign;
    }
    if (whole) {
#pragma unroll
      for (int i = 0; i < kScanPer; i += 4)
        *reinterpret_cast<uint4*>(p.offsets + t0 + i) = make_uint4(o[i], o[i + 1], o[i + 2], o[i + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < kScanPer; ++i)
        if (t0 + i < ntiles) p.offsets[t0 + i] = o[i];
    }
    __syncthreads();                                // everyone has read the carry and the warp sums
    if (tid == 0) s_carry = carry + round_total;
    __syncthreads();
  }
  if (tid == 0) {
    const uint64_t total = s_carry;
    p.offsets[ntiles] = (uint32_t)(total >> 32);
    p.nnz[0] = (int64_t)(total & 0xffffffffu);
    p.nnz[1] = (int64_t)(total >> 32);
    if (p.capacity >= 0 && (int64_t)(total >> 32) > p.capacity) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
  }
}

}  // namespace

// Exact kept counts per tile in offsets[0 .. ntiles) -> padded exclusive prefixes, offsets[ntiles] and nnz.
int launch_offsets_scan(uint32_t* offsets, int64_t ntiles, int64_t* nnz, int64_t capacity, int32_t* dev_status,
                        cudaStream_t s) {
  IndexParams p = {};
  p.ntiles = (int32_t)ntiles; p.offsets = offsets; p.nnz = nnz; p.capacity = capacity; p.dev_status = dev_status;
  count_launch();
  offsets_scan_kernel<<<1, 1024, 0, s>>>(p, ((uintptr_t)offsets & 15) == 0 ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// Index part (keep bits, row offsets, tile offsets, nnz) of a different-sample Bernoulli store.
int launch_store_index(const rad_store* st, bool check_capacity, int32_t* dev_status, cudaStream_t s) {
  const uint32_t T = keep_threshold_host(st->p);
  IndexParams p;
  p.B = st->B; p.D = st->D;
  p.ncb = (int32_t)ceil_div(st->D, kTileCols);
  p.ntiles = (int32_t)(ceil_div(st->B, kTileRows) * p.ncb);
  p.T = make_keep_threshold(T);
  p.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE); p.c3 = st->step;
  p.keepbits = st->keepbits; p.offsets = st->offsets; p.nnz = st->nnz;
  p.capacity = check_capacity ? st->values_capacity : -1;
  p.dev_status = dev_status;
  const PhiloxKeys ks = philox_expand_key(st->seed);
  const int grid = (int)std::min<int64_t>(ceil_div(p.ntiles, kIndexWarps), 148 * 12);
  if (st->law == RAD_LAW_FIXED) return launch_fixed_index(st, check_capacity, dev_status, s);
  count_launch();
  store_index_kernel<<<grid, 32 * kIndexWarps, 0, s>>>(p, ks);
  if (cudaGetLastError() != cudaSuccess) return RAD_ECUDA;
  return launch_offsets_scan(p.offsets, p.ntiles, p.nnz, p.capacity, dev_status, s);
}

}  // namespace rad

using namespace rad;

extern "C" int rad_store_index(const rad_store* st, int32_t* dev_status, void* stream) {
  if (st == nullptr || st->B <= 0 || st->D <= 0) return RAD_EINVAL;
  if (st->variant != RAD_DIFFERENT_SAMPLE || (st->law != RAD_LAW_BERNOULLI && st->law != RAD_LAW_FIXED)) return RAD_EUNSUPPORTED;
  if (st->keepbits == nullptr || st->offsets == nullptr || st->nnz == nullptr) return RAD_EINVAL;
  if (keep_threshold_host(st->p) == 0) return RAD_EINVAL;
  if ((double)st->B * (double)st->D >= 4294967296.0 * 0.75) return RAD_EINVAL;
  const int rc = check_device();
  if (rc != RAD_OK) return rc;
  return launch_store_index(st, st->values != nullptr, dev_status, static_cast<cudaStream_t>(stream));
}
