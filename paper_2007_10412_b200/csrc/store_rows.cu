// Fixed-count law without replacement (App. A, remark under the fraction sweep: sampling without replacement
// makes fraction 1.0 the exact gradient): every row keeps a uniformly random subset of exactly k = ceil(f D)
// columns, weight D / k, drawn by Floyd's subset sampling from the Philox stream of the row.  Because k is
// the same for every row, what is held has a static shape: B x k values and B x k 16-bit column numbers.
//
// A warp owns a row.  Floyd's step i (draw t_i in [0, D - k + i]; keep t_i unless it is already in, then keep
// D - k + i) needs the outcome of the steps before it, but only through membership tests, so 32 steps run
// side by side: the draws of a row are made up front, four per generator call; a group of 32 consecutive steps
// tests its draws against the row's bitmap (all earlier groups), finds equal draws inside the group with a
// match, settles the rare draw that hits the fall-back column of an earlier step of the same group by
// iterating to a fixed point, and then sets its 32 bits.  The result is bit for bit the sequential algorithm.
//
//   rows_fixed_kernel<T, kRowsOut>    kRowsOut: gathers the kept entries of the row in ascending column order
//                                     into the static-shape store;
//                                     else: writes the row's keep bits in the tile-major layout, the in-tile row
//                                     offsets (a CTA owns the 64 rows of a slab) and the tile counts: the index
//                                     part of a bitmask store, from the key alone
//   rows_to_tiles_kernel<T>           places the values of a static-shape store into the tile-major layout
//                                     whose index part the kernel above has written (weight gradient)
#include <algorithm>

#include "common.cuh"
#include "store.cuh"

namespace rad {
namespace {

struct RowsParams {
  const void* A;
  int64_t lda;
  int64_t B, D, k, ld;      // ld: columns of the static-shape store (>= k, multiple of 8)
  int32_t ncb;
  float scale;              // D / k
  uint32_t c2, c3;
  void* values;             // kRowsOut: B x ld
  uint16_t* cols;           // kRowsOut: B x ld
  uint32_t* keepbits;       // index mode: tile-major
  uint32_t* offsets;        // index mode: exact kept count per tile (turned into offsets by the scan kernel)
  int64_t* nnz;
  int32_t words;            // keep-bit words per row, ceil(D / 32)
  int32_t draws_stride;     // 32-bit words of shared memory per warp for the draws (k rounded up to 4)
  int32_t* dev_status;
};

// Floyd's subset of row `row` into `bm` (words of the row's bitmap in shared memory, zero on entry), by one
// warp.  `draws`: k words of the warp's own shared memory.
__device__ __forceinline__ void floyd_row(uint32_t* bm, uint32_t* draws, uint32_t row, uint32_t D, uint32_t k, uint32_t c2,
                                          uint32_t c3, const PhiloxKeys& ks, int lane) {
  const uint32_t first_j = D - k;                   // step i falls back on column first_j + i
  for (uint32_t c = lane; 4 * c < k; c += 32) {
    uint32_t w[4];
    philox4x32_10(c, row, c2, c3, ks, w);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const uint32_t i = 4 * c + jj;
      if (i < k) draws[i] = __umulhi(w[jj], first_j + i + 1u);
    }
  }
  __syncwarp();
  const uint32_t below = (1u << lane) - 1u;
#pragma unroll 1
  for (uint32_t i0 = 0; i0 < k; i0 += 32) {
    const uint32_t i = i0 + lane;
    const bool active = i < k;
    const uint32_t t = active ? draws[i] : 0u;
    const uint32_t bit = 1u << (t & 31);
    // in the set after the groups before this one?
    const bool in_before = active && (bm[t >> 5] & bit) != 0;
    __syncwarp();
    // Every draw that is not in yet goes in now.  Two steps of the group with the same draw are rare; one of
    // them finds the bit already set, and only then the group is matched to tell which step came first.
    const bool fresh = active && !in_before;
    const bool lost = fresh && (atomicOr(&bm[t >> 5], bit) & bit) != 0;
    bool coll = in_before;
    if (__any_sync(0xffffffffu, lost)) {
      const uint32_t same = __match_any_sync(0xffffffffu, fresh ? t : 0xffffffffu - (uint32_t)lane);
      coll = coll || (fresh && (same & below) != 0);
    }
    // a draw equal to the fall-back column of an earlier step of this group is a collision iff that step
    // collided (its bit is then set twice, which is harmless); settled by iterating to a fixed point
    const uint32_t m_lane = t - first_j - i0;       // wraps to a large number when t < first_j + i0
    const bool dep = active && !coll && m_lane < (uint32_t)lane;
    if (__any_sync(0xffffffffu, dep)) {
      for (int it = 0; it < 32; ++it) {
        const uint32_t cm = __ballot_sync(0xffffffffu, coll);
        const bool now = dep && ((cm >> (m_lane & 31)) & 1u) != 0;
        if (!__any_sync(0xffffffffu, now && !coll)) break;
        coll = coll || now;
      }
    }
    if (coll) {
      const uint32_t j = first_j + i;
      atomicOr(&bm[j >> 5], 1u << (j & 31));
    }
    __syncwarp();
  }
}

constexpr int kRowsWarps = 8;

template <typename T, bool kRowsOut>
__global__ void __launch_bounds__(32 * kRowsWarps) rows_fixed_kernel(const RowsParams p, const PhiloxKeys ks) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // per warp: bitmap (words), draws (draws_stride), column list (k 16-bit numbers, kRowsOut only)
  const int list_words = kRowsOut ? (int)((p.k + 1) / 2) : 0;
  const int per_warp = p.words + p.draws_stride + list_words;
  uint32_t* bm = s_dyn + warp * per_warp;
  uint32_t* draws = bm + p.words;
  uint16_t* list = reinterpret_cast<uint16_t*>(draws + p.draws_stride);
  uint8_t* s_cnt = reinterpret_cast<uint8_t*>(s_dyn + kRowsWarps * per_warp);   // index mode: [64 rows][ncb] kept per (row, block)
  const T* A = static_cast<const T*>(p.A);

  if (kRowsOut) {
    for (int64_t row = (int64_t)blockIdx.x * kRowsWarps + warp; row < p.B; row += (int64_t)gridDim.x * kRowsWarps) {
      for (int i = lane; i < p.words; i += 32) bm[i] = 0;
      __syncwarp();
      floyd_row(bm, draws, (uint32_t)row, (uint32_t)p.D, (uint32_t)p.k, p.c2, p.c3, ks, lane);
      // ascending list: a lane takes a run of consecutive words, so its kept columns are consecutive in the list
      const int per_lane = (p.words + 31) / 32;
      const int w0 = lane * per_lane, w1 = min(w0 + per_lane, p.words);
      uint32_t cnt = 0;
      for (int w = w0; w < w1; ++w) cnt += __popc(bm[w]);
      uint32_t incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      uint32_t pos = incl - cnt;
      for (int w = w0; w < w1; ++w) {
        uint32_t m = bm[w];
        while (m != 0) {
          const uint32_t b = __ffs(m) - 1;
          m &= m - 1;
          list[pos++] = (uint16_t)(w * 32 + b);
        }
      }
      __syncwarp();
      const T* rowp = A + row * p.lda;
      T* vrow = static_cast<T*>(p.values) + row * p.ld;
      uint16_t* crow = p.cols + row * p.ld;
      for (int64_t j = lane; j < p.ld; j += 32) {
        uint16_t col = 0;
        float v = 0.0f;
        if (j < p.k) {
          col = list[j];
          v = __fmul_rn(to_float(rowp[col]), p.scale);
        }
        vrow[j] = from_float<T>(v);
        crow[j] = col;
      }
      __syncwarp();
    }
    if (blockIdx.x == 0 && tid == 0) { p.nnz[0] = p.B * p.k; p.nnz[1] = p.B * p.ld; }
  } else {
    // one CTA per slab of 64 rows; warp w takes rows w, w + 8, ...
    for (int64_t slab = blockIdx.x; slab * kTileRows < p.B; slab += gridDim.x) {
      for (int r = warp; r < kTileRows; r += kRowsWarps) {
        const int64_t row = slab * kTileRows + r;
        for (int i = lane; i < p.words; i += 32) bm[i] = 0;
        __syncwarp();
        if (row < p.B) floyd_row(bm, draws, (uint32_t)row, (uint32_t)p.D, (uint32_t)p.k, p.c2, p.c3, ks, lane);
        // the row's words go to their tiles (word 4 r + w of tile slab * ncb + block), four words at a time
        for (int cb = lane; cb < p.ncb; cb += 32) {
          uint32_t q[4];
#pragma unroll
          for (int w = 0; w < 4; ++w) q[w] = 4 * cb + w < p.words ? bm[4 * cb + w] : 0u;
          *reinterpret_cast<uint4*>(p.keepbits + (slab * p.ncb + cb) * kTileWords + r * 4) = make_uint4(q[0], q[1], q[2], q[3]);
          s_cnt[r * p.ncb + cb] = (uint8_t)(__popc(q[0]) + __popc(q[1]) + __popc(q[2]) + __popc(q[3]));   // at most 128
        }
        __syncwarp();
      }
      __syncthreads();
      // in-tile row offsets: prefix down the 64 rows of each column block
      for (int cb = tid; cb < p.ncb; cb += 32 * kRowsWarps) {
        uint32_t* tw = p.keepbits + (slab * p.ncb + cb) * kTileWords;
        uint32_t run = 0;
        for (int r = 0; r < kTileRows; r += 2) {
          const uint32_t c0 = s_cnt[r * p.ncb + cb], c1 = s_cnt[(r + 1) * p.ncb + cb];
          tw[kBitWords + (r >> 1)] = run | ((run + c0) << 16);
          run += c0 + c1;
        }
        p.offsets[slab * p.ncb + cb] = run;
      }
      __syncthreads();
    }
  }
}

// Static-shape store -> values of the tile-major store with the same mask (whose keep bits, row offsets and tile
// offsets are in place).  A warp owns a row; its entries come in ascending column order, 32 at a time: entry j
// of column block cb goes to offsets[tile] + row offset + (j - first entry of the row in that block).
template <typename T>
__global__ void __launch_bounds__(256) rows_to_tiles_kernel(const T* values, const uint16_t* cols, int64_t B, int64_t k,
                                                            int64_t ld, int32_t ncb, const uint32_t* keepbits,
                                                            const uint32_t* offsets, T* out, int64_t capacity,
                                                            int32_t* dev_status) {
  const int lane = threadIdx.x & 31;
  for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < B; row += (int64_t)gridDim.x * 8) {
    const int64_t slab = row >> 6;
    const int r = (int)(row & 63);
    uint32_t prev_cb = 0xffffffffu;
    int64_t prev_start = 0;                         // first entry of the row in column block prev_cb
    for (int64_t j0 = 0; j0 < k; j0 += 32) {
      const int64_t j = j0 + lane;
      const bool active = j < k;
      const uint32_t col = active ? cols[row * ld + j] : 0u;
      const uint32_t cb = active ? col >> 7 : 0xfffffffeu;
      const uint32_t same = __match_any_sync(0xffffffffu, cb);
      const int leader = __ffs(same) - 1;
      int64_t start = j0 + leader;                  // first entry of this block inside the group ...
      if (cb == prev_cb) start = prev_start;        // ... unless the block began in an earlier group
      if (active) {
        const int64_t tile = slab * ncb + cb;
        const uint32_t rowoff = reinterpret_cast<const uint16_t*>(keepbits + tile * kTileWords + kBitWords)[r];
        const int64_t pos = (int64_t)offsets[tile] + rowoff + (j - start);
        if (pos < capacity) out[pos] = values[row * ld + j];
        else raise_status(dev_status, RAD_DEV_ECAPACITY);
      }
      // carry the block of the group's last active entry
      const int last = active ? lane : -1;
      const int last_lane = __reduce_max_sync(0xffffffffu, last);
      if (last_lane >= 0) {
        prev_cb = __shfl_sync(0xffffffffu, cb, last_lane);
        prev_start = __shfl_sync(0xffffffffu, start, last_lane);
      }
    }
  }
}

// zeros between the last value of a tile and its padded end
template <typename T>
__global__ void __launch_bounds__(256) tile_padding_kernel(const uint32_t* keepbits, const uint32_t* offsets, int64_t ntiles,
                                                           T* out, int64_t capacity) {
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < ntiles; t += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t* tw = keepbits + t * kTileWords;
    const uint4 q = *reinterpret_cast<const uint4*>(tw + 63 * 4);
    const uint32_t exact = reinterpret_cast<const uint16_t*>(tw + kBitWords)[63] + __popc(q.x) + __popc(q.y) + __popc(q.z) + __popc(q.w);
    const int64_t end = min((int64_t)offsets[t + 1], capacity);
    for (int64_t i = (int64_t)offsets[t] + exact; i < end; ++i) out[i] = from_float<T>(0.0f);
  }
}

constexpr int64_t kRowsSmemBudget = 200 * 1024;

// shared memory of rows_fixed_kernel, or -1 if a row does not fit
int64_t rows_smem(int64_t D, int64_t k, bool rows_out, int64_t ncb) {
  const int64_t words = ceil_div(D, 32), draws = round_up(k, 4), list = rows_out ? (k + 1) / 2 : 0;
  const int64_t bytes = kRowsWarps * (words + draws + list) * 4 + (rows_out ? 0 : round_up(kTileRows * ncb, 16));
  return bytes <= kRowsSmemBudget ? bytes : -1;
}

RowsParams rows_params(const rad_store* st, int64_t k) {
  RowsParams p = {};
  p.B = st->B; p.D = st->D; p.k = k;
  p.ncb = (int32_t)ceil_div(st->D, kTileCols);
  p.scale = (float)st->D / (float)k;
  p.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE, RAD_LAW_FIXED); p.c3 = st->step;
  p.words = (int32_t)ceil_div(st->D, 32);
  p.draws_stride = (int32_t)round_up(k, 4);
  return p;
}

template <bool kRowsOut>
int launch_rows_fixed(const RowsParams& p, int dtype, uint64_t seed, int64_t smem, int grid, cudaStream_t s) {
  const PhiloxKeys ks = philox_expand_key(seed);
  count_launch();
  if (dtype == RAD_BF16) {
    RAD_CUDA_TRY(cudaFuncSetAttribute(rows_fixed_kernel<bf16, kRowsOut>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowsSmemBudget));
    rows_fixed_kernel<bf16, kRowsOut><<<grid, 32 * kRowsWarps, (size_t)smem, s>>>(p, ks);
  } else {
    RAD_CUDA_TRY(cudaFuncSetAttribute(rows_fixed_kernel<float, kRowsOut>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowsSmemBudget));
    rows_fixed_kernel<float, kRowsOut><<<grid, 32 * kRowsWarps, (size_t)smem, s>>>(p, ks);
  }
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace

bool rows_store_ok(const rad_store* st) {
  const int64_t k = draws_per_row_host(st->p, st->D);
  return k > 0 && st->law == RAD_LAW_FIXED && st->D <= 65536 && st->values != nullptr && st->keepbits != nullptr &&
         st->nnz != nullptr && st->values_ld >= k && st->values_ld % 8 == 0 && st->values_capacity >= st->B * st->values_ld &&
         rows_smem(st->D, k, true, ceil_div(st->D, kTileCols)) >= 0;
}

// The static-shape store of a layer input: B x ld values and B x ld 16-bit column numbers (in st->keepbits).
int rows_forward_store(const void* A, int64_t lda, const rad_store* st, int32_t* dev_status, cudaStream_t s) {
  if (!rows_store_ok(st)) return st->D > 65536 ? RAD_EUNSUPPORTED : RAD_EINVAL;
  const int64_t k = draws_per_row_host(st->p, st->D);
  RowsParams p = rows_params(st, k);
  p.A = A; p.lda = lda; p.ld = st->values_ld;
  p.values = st->values; p.cols = reinterpret_cast<uint16_t*>(st->keepbits); p.nnz = st->nnz; p.dev_status = dev_status;
  const int grid = (int)std::min<int64_t>(ceil_div(st->B, kRowsWarps), 148 * 4);
  int rc = launch_rows_fixed<true>(p, st->dtype, st->seed, rows_smem(st->D, k, true, p.ncb), grid, s);
  if (rc != RAD_OK) return rc;
  if (st->relubits != nullptr) return launch_relu_bits(st->dtype, A, lda, st->B, st->D, st->relubits, s);
  return RAD_OK;
}

// Index part (keep bits, row offsets, tile offsets, nnz) of a tile-major store under the fixed-count law, from
// the key alone.  RAD_EUNSUPPORTED where a row's scratch does not fit shared memory.
int launch_fixed_index(const rad_store* st, bool check_capacity, int32_t* dev_status, cudaStream_t s) {
  const int64_t k = draws_per_row_host(st->p, st->D);
  if (k <= 0) return RAD_EINVAL;
  RowsParams p = rows_params(st, k);
  const int64_t smem = rows_smem(st->D, k, false, p.ncb);
  if (smem < 0 || ((uintptr_t)st->keepbits & 15) != 0) return RAD_EUNSUPPORTED;
  p.keepbits = st->keepbits; p.offsets = st->offsets; p.nnz = st->nnz; p.dev_status = dev_status;
  const int64_t slabs = ceil_div(st->B, kTileRows);
  int rc = launch_rows_fixed<false>(p, st->dtype, st->seed, smem, (int)std::min<int64_t>(slabs, 148 * 8), s);
  if (rc != RAD_OK) return rc;
  return launch_offsets_scan(st->offsets, slabs * p.ncb, st->nnz, check_capacity ? st->values_capacity : -1, dev_status, s);
}

// Values of the tile-major store `tiles` (index part in place) from the static-shape store `rows` of the same key.
int rows_to_tiles(const rad_store* rows, const rad_store* tiles, int32_t* dev_status, cudaStream_t s) {
  const int64_t k = draws_per_row_host(rows->p, rows->D);
  const int32_t ncb = (int32_t)ceil_div(rows->D, kTileCols);
  const int64_t ntiles = ceil_div(rows->B, kTileRows) * ncb;
  const int grid = (int)std::min<int64_t>(ceil_div(rows->B, 8), 148 * 8);
  const int grid_t = (int)std::min<int64_t>(ceil_div(ntiles, 256), 148 * 8);
  count_launch(2);
  if (rows->dtype == RAD_BF16) {
    rows_to_tiles_kernel<bf16><<<grid, 256, 0, s>>>(static_cast<const bf16*>(rows->values), reinterpret_cast<const uint16_t*>(rows->keepbits),
                                                    rows->B, k, rows->values_ld, ncb, tiles->keepbits, tiles->offsets,
                                                    static_cast<bf16*>(tiles->values), tiles->values_capacity, dev_status);
    tile_padding_kernel<bf16><<<grid_t, 256, 0, s>>>(tiles->keepbits, tiles->offsets, ntiles, static_cast<bf16*>(tiles->values),
                                                     tiles->values_capacity);
  } else {
    rows_to_tiles_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(rows->values), reinterpret_cast<const uint16_t*>(rows->keepbits),
                                                     rows->B, k, rows->values_ld, ncb, tiles->keepbits, tiles->offsets,
                                                     static_cast<float*>(tiles->values), tiles->values_capacity, dev_status);
    tile_padding_kernel<float><<<grid_t, 256, 0, s>>>(tiles->keepbits, tiles->offsets, ntiles, static_cast<float*>(tiles->values),
                                                      tiles->values_capacity);
  }
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

}  // namespace rad
