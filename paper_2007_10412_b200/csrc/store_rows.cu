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
//
// The with-replacement law (Sec. 3.2: k draws per row, an entry drawn c times weighs c d / k) takes the same
// road to a bitmask store without a B x D multiplicity matrix in HBM:
//   replace_index_kernel              a warp's k draws set bits in the bitmap of its row in shared memory; a
//                                     draw that finds its bit set is a repeat.  The row's keep bits go to the
//                                     tile-major layout as above, and the few columns drawn more than once go,
//                                     with their counts, to a short list per row
//   replace_extras_kernel<T>          after the values have been placed with the weight of a single draw: the
//                                     listed entries are written again with their own weight
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

// With-replacement law, index part.  One CTA per slab of 64 rows; warp w takes rows w, w + 8, ...  A draw sets
// its column's bit in the row's bitmap (shared memory, the row's keep-bit words); a draw that finds the bit set
// is a repeat and goes to the warp's short list of repeats.  A column drawn c times is on that list c - 1 times.
// extras: `extras_ld` words per row: word 0 = entries that follow, each (column | count << 16), count >= 2.
__global__ void __launch_bounds__(32 * kRowsWarps) replace_index_kernel(const RowsParams p, const PhiloxKeys ks, uint32_t* extras,
                                                                        int32_t extras_ld) {
  extern __shared__ __align__(16) uint32_t s_dyn[];
  __shared__ uint32_t s_nrep[kRowsWarps], s_nex[kRowsWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_warp = p.words + p.draws_stride;            // bitmap, then up to k repeats as 16-bit columns
  uint32_t* bm = s_dyn + warp * per_warp;
  uint16_t* rep = reinterpret_cast<uint16_t*>(bm + p.words);
  uint8_t* s_cnt = reinterpret_cast<uint8_t*>(s_dyn + kRowsWarps * per_warp);   // [64 rows][ncb] kept per (row, block)
  for (int64_t slab = blockIdx.x; slab * kTileRows < p.B; slab += gridDim.x) {
    for (int r = warp; r < kTileRows; r += kRowsWarps) {
      const int64_t row = slab * kTileRows + r;
      for (int i = lane; i < p.words; i += 32) bm[i] = 0;
      if (lane == 0) { s_nrep[warp] = 0; s_nex[warp] = 0; }
      __syncwarp();
      if (row < p.B) {
        for (uint32_t c = lane; 4 * (int64_t)c < p.k; c += 32) {
          uint32_t w[4];
          philox4x32_10(c, (uint32_t)row, p.c2, p.c3, ks, w);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (4 * (int64_t)c + j < p.k) {
              const uint32_t col = __umulhi(w[j], (uint32_t)p.D);
              const uint32_t bit = 1u << (col & 31);
              if (atomicOr(&bm[col >> 5], bit) & bit) rep[atomicAdd(&s_nrep[warp], 1u)] = (uint16_t)col;   // fewer than k
            }
          }
        }
        __syncwarp();
        // repeats of one column are counted together; the first of them on the list writes the entry
        const uint32_t n = s_nrep[warp];
        uint32_t* ex = extras + row * extras_ld;
        for (uint32_t j = lane; j < n; j += 32) {
          const uint32_t col = rep[j];
          uint32_t cnt = 0;
          bool first = true;
          for (uint32_t i = 0; i < n; ++i) {
            const bool same = rep[i] == col;
            cnt += same ? 1u : 0u;
            first = first && !(same && i < j);
          }
          if (first) {
            const uint32_t slot = atomicAdd(&s_nex[warp], 1u) + 1u;
            if ((int)slot < extras_ld) ex[slot] = col | ((cnt + 1u) << 16);
            else raise_status(p.dev_status, RAD_DEV_EINTERNAL);
          }
        }
        __syncwarp();
        if (lane == 0) ex[0] = min(s_nex[warp], (uint32_t)(extras_ld - 1));
      }
      __syncwarp();
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

// The entries drawn more than once, written again with their own weight fl32(c * (D / k)) (one product with the
// entry, as for every other value).  A warp per row; the entry's place follows from the index part.
template <typename T>
__global__ void __launch_bounds__(256) replace_extras_kernel(const T* A, int64_t lda, int64_t B, int32_t ncb, const uint32_t* extras,
                                                             int32_t extras_ld, const uint32_t* keepbits, const uint32_t* offsets,
                                                             T* values, int64_t capacity, float scale) {
  const int lane = threadIdx.x & 31;
  for (int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); row < B; row += (int64_t)gridDim.x * 8) {
    const uint32_t* ex = extras + row * extras_ld;
    const uint32_t n = ex[0];
    const int64_t slab = row >> 6;
    const int r = (int)(row & 63);
    for (uint32_t j = lane; j < n; j += 32) {
      const uint32_t e = ex[1 + j];
      const uint32_t col = e & 0xffffu, c = e >> 16;
      const int64_t tile = slab * ncb + (col >> 7);
      const uint32_t* tw = keepbits + tile * kTileWords;
      const uint4 q = *reinterpret_cast<const uint4*>(tw + r * 4);
      const uint32_t wq = (col & 127u) >> 5, bit = col & 31u;
      const uint32_t word = wq == 0 ? q.x : wq == 1 ? q.y : wq == 2 ? q.z : q.w;
      uint32_t rank = __popc(word & ((1u << bit) - 1u));
      if (wq > 0) rank += __popc(q.x);
      if (wq > 1) rank += __popc(q.y);
      if (wq > 2) rank += __popc(q.z);
      const uint32_t rowoff = reinterpret_cast<const uint16_t*>(tw + kBitWords)[r];
      if ((int64_t)offsets[tile + 1] <= capacity)       // a tile that does not fit is left out as a whole
        values[(int64_t)offsets[tile] + rowoff + rank] = from_float<T>(__fmul_rn(to_float(A[row * lda + col]), __fmul_rn((float)c, scale)));
    }
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

// Words per row of the list of entries drawn more than once (first word: their number).  k draws hit at most
// k / 2 columns twice or more; the list takes the place of the row of the multiplicity matrix, so it has to fit
// in D bytes.  0: the law's index cannot be made this way (too many draws for the list, or a row's histogram
// does not fit shared memory).
int64_t replace_extras_ld(int64_t D, int64_t k) {
  const int64_t words = ceil_div(D, 32), ncb = ceil_div(D, kTileCols);
  if (D > 65536 || k / 2 + 1 > D / 4) return 0;
  if (kRowsWarps * (words + round_up(k, 4)) * 4 + round_up(kTileRows * ncb, 16) > kRowsSmemBudget) return 0;
  return D / 4;
}

// Index part of a tile-major store under the with-replacement law, from the key alone, plus the list of entries
// drawn more than once (`extras`: B x replace_extras_ld words).  RAD_EUNSUPPORTED where that does not apply.
int launch_replace_index(const rad_store* st, uint32_t* extras, bool check_capacity, int32_t* dev_status, cudaStream_t s) {
  const int64_t k = draws_per_row_host(st->p, st->D);
  if (k <= 0) return RAD_EINVAL;
  const int64_t ld = replace_extras_ld(st->D, k);
  if (ld == 0 || ((uintptr_t)st->keepbits & 15) != 0) return RAD_EUNSUPPORTED;
  RowsParams p = rows_params(st, k);
  p.c2 = counter_word2(st->layer, RAD_DIFFERENT_SAMPLE, RAD_LAW_REPLACE);
  p.keepbits = st->keepbits; p.offsets = st->offsets; p.nnz = st->nnz; p.dev_status = dev_status;
  const int64_t slabs = ceil_div(st->B, kTileRows);
  const int64_t smem = kRowsWarps * ((int64_t)p.words + p.draws_stride) * 4 + round_up(kTileRows * p.ncb, 16);
  const PhiloxKeys ks = philox_expand_key(st->seed);
  count_launch();
  RAD_CUDA_TRY(cudaFuncSetAttribute(replace_index_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kRowsSmemBudget));
  replace_index_kernel<<<(int)std::min<int64_t>(slabs, 148 * 8), 32 * kRowsWarps, (size_t)smem, s>>>(p, ks, extras, (int32_t)ld);
  if (cudaGetLastError() != cudaSuccess) return RAD_ECUDA;
  return launch_offsets_scan(st->offsets, slabs * p.ncb, st->nnz, check_capacity ? st->values_capacity : -1, dev_status, s);
}

// The listed entries written again with their own weight (after the values have been placed with D / k).
int launch_replace_extras(const void* A, int64_t lda, const rad_store* st, const uint32_t* extras, cudaStream_t s) {
  const int64_t k = draws_per_row_host(st->p, st->D);
  const int64_t ld = replace_extras_ld(st->D, k);
  if (ld == 0) return RAD_EUNSUPPORTED;
  const int32_t ncb = (int32_t)ceil_div(st->D, kTileCols);
  const float scale = (float)st->D / (float)k;
  const int grid = (int)std::min<int64_t>(ceil_div(st->B, 8), 148 * 64);   // short dependent chains: many warps in flight
  count_launch();
  if (st->dtype == RAD_BF16)
    replace_extras_kernel<bf16><<<grid, 256, 0, s>>>(static_cast<const bf16*>(A), lda, st->B, ncb, extras, (int32_t)ld, st->keepbits,
                                                     st->offsets, static_cast<bf16*>(st->values), st->values_capacity, scale);
  else
    replace_extras_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(A), lda, st->B, ncb, extras, (int32_t)ld, st->keepbits,
                                                      st->offsets, static_cast<float*>(st->values), st->values_capacity, scale);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
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
