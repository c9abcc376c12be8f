// Index part of a different-sample store from the key alone (Sec. 3.2: the random P is independent of the
// data; Sec. 4.2: it is drawn per layer input).  The keep decision of entry (b, d) depends on (seed, layer,
// step, b, d) only, so keep bits, row offsets, tile offsets and the kept count can be produced without
// reading the layer input, before that input exists.  The forward GEMM of the layer that produces the input
// then drops the kept values into place from its epilogue (tc.cu), and a caller learns the exact size of a
// store before it allocates `values`.
//
//   store_index_kernel   one tile (64 x 128 entries) per CTA and turn, one keep-bit word per thread: draw, write
//                        the word, in-tile row offsets from a CTA scan, exact kept count of the tile into
//                        offsets[tile]
//   offsets_scan_kernel  one CTA turns the counts into padded exclusive prefixes in place and writes nnz
//
// Layout and bits are those of the one-pass store kernels.
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

__global__ void __launch_bounds__(256) store_index_kernel(const IndexParams p, const PhiloxKeys ks) {
  __shared__ uint32_t s_warp[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = tid >> 2, w = tid & 3;              // row of the tile, keep-bit word of the row
  for (int64_t tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
    const int64_t slab = tile / p.ncb;
    const int cb = (int)(tile - slab * p.ncb);
    const int64_t row = slab * kTileRows + r;
    const int64_t col0 = (int64_t)cb * kTileCols + 32 * w;
    uint32_t m = 0;
    if (row < p.B && col0 < p.D) {
      m = philox_keep32((uint32_t)(col0 >> 5), (uint32_t)row, p.c2, p.c3, ks, p.T);
      const int64_t nv = p.D - col0;
      if (nv < 32) m &= (1u << nv) - 1u;
    }
    p.keepbits[tile * kTileWords + tid] = m;
    // exclusive prefix over the tile's words in (row, word) order = thread order
    const uint32_t c = __popc(m);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t before = 0, total = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t t = s_warp[i];
      if (i < warp) before += t;
      total += t;
    }
    if (w == 0) reinterpret_cast<uint16_t*>(p.keepbits + tile * kTileWords + kBitWords)[r] = (uint16_t)(before + incl - c);
    if (tid == 0) p.offsets[tile] = total;
    __syncthreads();                                // s_warp is rewritten in the next turn
  }
}

// offsets[t] holds the exact kept count of tile t on entry and the first element of tile t in `values` on
// exit (every tile padded to a multiple of kValueAlign); offsets[ntiles] = elements used.
__global__ void __launch_bounds__(1024) offsets_scan_kernel(const IndexParams p) {
  __shared__ uint64_t s_pad[32], s_exact[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t per = (p.ntiles + 1023) / 1024;
  const int64_t t0 = min((int64_t)tid * per, (int64_t)p.ntiles), t1 = min(t0 + per, (int64_t)p.ntiles);
  uint64_t pad = 0, exact = 0;
  for (int64_t t = t0; t < t1; ++t) {
    const uint32_t c = p.offsets[t];
    exact += c;
    pad += (c + kValueAlign - 1) / kValueAlign * kValueAlign;
  }
  uint64_t ipad = pad, iex = exact;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint64_t a = __shfl_up_sync(0xffffffffu, ipad, o), b = __shfl_up_sync(0xffffffffu, iex, o);
    if (lane >= o) { ipad += a; iex += b; }
  }
  if (lane == 31) { s_pad[warp] = ipad; s_exact[warp] = iex; }
  __syncthreads();
  uint64_t base = ipad - pad, all_pad = 0, all_exact = 0;
  for (int i = 0; i < 32; ++i) {
    if (i < warp) base += s_pad[i];
    all_pad += s_pad[i];
    all_exact += s_exact[i];
  }
  for (int64_t t = t0; t < t1; ++t) {
    const uint32_t c = p.offsets[t];
    p.offsets[t] = (uint32_t)base;
    base += (c + kValueAlign - 1) / kValueAlign * kValueAlign;
  }
  if (tid == 0) {
    p.offsets[p.ntiles] = (uint32_t)all_pad;
    p.nnz[0] = (int64_t)all_exact;
    p.nnz[1] = (int64_t)all_pad;
    if (p.capacity >= 0 && (int64_t)all_pad > p.capacity) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
  }
}

}  // namespace

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
  const int grid = (int)std::min<int64_t>(p.ntiles, 148 * 8);
  count_launch(2);
  store_index_kernel<<<grid, 256, 0, s>>>(p, ks);
  offsets_scan_kernel<<<1, 1024, 0, s>>>(p);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad

using namespace rad;

extern "C" int rad_store_index(const rad_store* st, int32_t* dev_status, void* stream) {
  if (st == nullptr || st->B <= 0 || st->D <= 0) return RAD_EINVAL;
  if (st->variant != RAD_DIFFERENT_SAMPLE || st->law != RAD_LAW_BERNOULLI) return RAD_EUNSUPPORTED;
  if (st->keepbits == nullptr || st->offsets == nullptr || st->nnz == nullptr) return RAD_EINVAL;
  if (keep_threshold_host(st->p) == 0) return RAD_EINVAL;
  if ((double)st->B * (double)st->D >= 4294967296.0 * 0.75) return RAD_EINVAL;
  const int rc = check_device();
  if (rc != RAD_OK) return rc;
  return launch_store_index(st, st->values != nullptr, dev_status, static_cast<cudaStream_t>(stream));
}
