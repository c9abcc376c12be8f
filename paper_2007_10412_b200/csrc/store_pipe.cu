// Different-sample store as a persistent, software-pipelined kernel (Sec. 3.2 / 4.2 of the paper: the
// layer input is sampled, scaled by 1 / p_eff and only the kept entries are held).
//
// A CTA claims chunks of kChunk consecutive 64 x 128 tiles in ticket order and runs two phases per
// chunk, the first phase of the next chunk ahead of the second phase of the current one:
//   phase 1  needs no data: every compute thread draws the 32 keep decisions of one keep-bit word
//            per tile (two Philox calls), writes the word, and the warp totals go to shared memory;
//   look-back a service warp adds the chunk's padded and exact counts, publishes them, and finds where
//            the chunk starts in `values` from the chunks before it (decoupled look-back);
//   phase 2  the tile of A arrives in shared memory by TMA (a second service warp runs a ring of
//            loads ahead of the compute warps); a warp scan over the counts gives every word its
//            place in (row, column) order, and each thread walks the set bits of its word, scaling
//            the kept entries into a staging buffer;
//   output   a third service warp pads the tile to a multiple of eight entries and sends the staging
//            buffer to `values` with one bulk copy.
// The look-back of chunk c+1 therefore has the whole second phase of chunk c to finish in, and no
// compute thread ever loads from or stores to global memory except for the index words.
// The layout produced is the one of the generic kernel: the order of tiles in `values` is the tile index.
//
// Every wait is bounded (2 s on the global timer).  On expiry the CTA raises RAD_DEV_ETIMEOUT, all
// roles leave their loops, outstanding loads and bulk copies are waited for, and the kernel returns.
#include <cuda.h>

#include "common.cuh"
#include "store.cuh"

namespace rad {
namespace {

constexpr int kChunk = 4;                       // tiles per claimed chunk
constexpr int kComputeWarps = 8;                // 256 threads: one keep-bit word of a tile each
constexpr int kLoaderWarp = kComputeWarps, kLookbackWarp = kComputeWarps + 1;   // the output warp is the last one
constexpr int kPipeThreads = (kComputeWarps + 3) * 32;
constexpr int kSlots = 4;                       // chunk descriptors in flight
constexpr uint32_t kNoChunk = 0xffffffffu;
constexpr uint64_t kPipeWaitLimitNs = 2000000000ull;
constexpr int kTileElems = kTileRows * kTileCols;

template <typename T, int S>
struct PipeSmem {
  alignas(128) T raw[S][kTileElems];            // tiles of A as loaded
  alignas(128) T outv[2][kTileElems];           // kept values of a tile in (row, column) order
  uint64_t full[S], empty[S];                   // raw ring
  uint64_t staged[2], out_free[2];              // staging buffers
  uint64_t chunk_ready[kSlots], cnt_ready[kSlots], base_ready[kSlots];
  uint32_t chunk_id[kSlots];
  uint32_t warp_total[kSlots][kChunk][kComputeWarps];
  uint32_t tile_total[kSlots][kChunk];
  int64_t tile_base[kSlots][kChunk];            // first element in `values`; -1: do not write
  int abort_flag;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait; false when the CTA is giving up (this wait or another one ran out of time).
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (bar_try_wait(bar, parity)) return true;
  const uint64_t t0 = timer_ns();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (bar_try_wait(bar, parity)) return true;
    if (*abort_flag != 0) return false;
    if (timer_ns() - t0 > kPipeWaitLimitNs) {
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_load_tile(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_addr(ssrc)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ uint32_t warp_inclusive_scan(uint32_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t n = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += n;
  }
  return v;
}

__device__ __forceinline__ float raw_to_float(float v) { return v; }
__device__ __forceinline__ float raw_to_float(bf16 v) { return __bfloat162float(v); }

// Bits of (a > 0) for 32 consecutive entries in shared memory; zero of either sign gives 0.
__device__ __forceinline__ uint32_t positive32(const float* src) {
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float4 v = reinterpret_cast<const float4*>(src)[i];
    m |= (v.x > 0.0f ? 1u : 0u) << (4 * i) | (v.y > 0.0f ? 1u : 0u) << (4 * i + 1) |
         (v.z > 0.0f ? 1u : 0u) << (4 * i + 2) | (v.w > 0.0f ? 1u : 0u) << (4 * i + 3);
  }
  return m;
}
__device__ __forceinline__ uint32_t positive32(const bf16* src) {
  uint32_t m = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 q = reinterpret_cast<const uint4*>(src)[i];
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      // positive: sign clear and some other bit set (the add carries into the sign position)
      const uint32_t nz = ((w[j] & 0x7fff7fffu) + 0x7fff7fffu) & ~w[j] & 0x80008000u;
      m |= ((nz >> 15) & 1u) << (8 * i + 2 * j) | (nz >> 31) << (8 * i + 2 * j + 1);
    }
  }
  return m;
}

template <typename T, int S>
__global__ void __launch_bounds__(kPipeThreads) store_pipelined_kernel(const StoreParams p, const PhiloxKeys ks,
                                                                      const __grid_constant__ CUtensorMap tmA) {
  extern __shared__ unsigned char smem_raw[];
  PipeSmem<T, S>& sm = *reinterpret_cast<PipeSmem<T, S>*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile int* abort_flag = &sm.abort_flag;
  const uint32_t ntiles = (uint32_t)p.ntiles;
  const uint32_t nchunks = (ntiles + kChunk - 1) / kChunk;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { bar_init(&sm.full[s], 1); bar_init(&sm.empty[s], kComputeWarps); }
    for (int b = 0; b < 2; ++b) { bar_init(&sm.staged[b], kComputeWarps); bar_init(&sm.out_free[b], 1); }
    for (int q = 0; q < kSlots; ++q) {
      bar_init(&sm.chunk_ready[q], 1);
      bar_init(&sm.cnt_ready[q], kComputeWarps);
      bar_init(&sm.base_ready[q], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp < kComputeWarps) {
    // ---------------------------------------------------------------------------------------------
    // compute warps.  Thread (warp, lane) owns keep-bit word warp * 32 + lane of every tile: row
    // 8 * warp + lane / 4 of the tile, columns 32 * (lane % 4) .. + 31.
    // ---------------------------------------------------------------------------------------------
    const int r = warp * 8 + (lane >> 2), wq = lane & 3;
    uint32_t n = 0;                               // tiles this CTA has worked through (ring position)
    uint32_t m_cur[kChunk], m_nxt[kChunk];
    uint32_t chunk_cur = kNoChunk, chunk_nxt = kNoChunk;

    auto phase1 = [&](uint32_t seq, uint32_t (&m)[kChunk]) -> uint32_t {
      const int slot = seq % kSlots;
      if (!bar_wait(&sm.chunk_ready[slot], (seq / kSlots) & 1u, abort_flag)) return kNoChunk;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) return kNoChunk;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) {
        const uint32_t tile = chunk * kChunk + g;
        uint32_t mm = 0;
        if (tile < ntiles) {
          const uint32_t slab = tile / (uint32_t)p.ncb, cb = tile - slab * (uint32_t)p.ncb;
          const int64_t row = (int64_t)slab * kTileRows + r;
          const int64_t col0 = (int64_t)cb * kTileCols + wq * 32;
          const int64_t nv = p.D - col0;
          if (row < p.B && nv > 0) {
            const uint32_t g16 = (uint32_t)(col0 >> 4);
            const uint32_t lo = philox_keep16(g16, (uint32_t)row, p.c2, p.c3, ks, p.T);
            const uint32_t hi = philox_keep16(g16 + 1u, (uint32_t)row, p.c2, p.c3, ks, p.T);
            mm = lo | (hi << 16);
            if (nv < 32) mm &= (1u << (int)nv) - 1u;
          }
          p.keepbits[(int64_t)tile * kTileWords + warp * 32 + lane] = mm;
        }
        m[g] = mm;
        const uint32_t wt = __reduce_add_sync(0xffffffffu, __popc(mm));
        if (lane == 0) sm.warp_total[slot][g][warp] = wt;
      }
      __syncwarp();
      if (lane == 0) bar_arrive(&sm.cnt_ready[slot]);
      return chunk;
    };

    uint32_t seq = 0;
    chunk_nxt = phase1(seq, m_nxt);
    bool ok = true;
    while (ok && chunk_nxt != kNoChunk) {
      chunk_cur = chunk_nxt;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) m_cur[g] = m_nxt[g];
      const int slot = seq % kSlots;
      const uint32_t slot_parity = (seq / kSlots) & 1u;
      ++seq;
      chunk_nxt = phase1(seq, m_nxt);
      // phase 2 of chunk_cur; the other warps' totals of its first phase are needed now
      if (!bar_wait(&sm.cnt_ready[slot], slot_parity, abort_flag)) break;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) {
        const uint32_t tile = chunk_cur * kChunk + g;
        if (tile >= ntiles) break;
        const int s = n % S, b = n & 1;
        uint32_t mm = m_cur[g];
        const uint32_t cnt = __popc(mm);
        const uint32_t incl = warp_inclusive_scan(cnt, lane);
        const uint32_t wt = sm.warp_total[slot][g][lane & 7];
        const uint32_t wbase = __reduce_add_sync(0xffffffffu, lane < warp ? wt : 0u);
        uint32_t pos = wbase + incl - cnt;
        if (wq == 0)
          reinterpret_cast<uint16_t*>(p.keepbits + (int64_t)tile * kTileWords + kBitWords)[r] = (uint16_t)pos;
        if (!bar_wait(&sm.out_free[b], ((n >> 1) & 1u) ^ 1u, abort_flag) ||
            !bar_wait(&sm.full[s], (n / S) & 1u, abort_flag)) {
          ok = false;
          break;
        }
        const T* src = sm.raw[s] + r * kTileCols + wq * 32;
        T* dst = sm.outv[b] + pos;
        uint32_t rev = __brev(mm);                // leading zeros of rev = index of the lowest set bit
        while (rev != 0) {
          const int q = __clz(rev);
          rev &= ~(0x80000000u >> q);
          *dst++ = from_float<T>(raw_to_float(src[q]) * p.scale);
        }
        if (p.relubits != nullptr) {
          const uint32_t slab = tile / (uint32_t)p.ncb, cb = tile - slab * (uint32_t)p.ncb;
          const int64_t row = (int64_t)slab * kTileRows + r;
          const int word = (int)cb * 4 + wq;
          if (row < p.B && word < p.w32) {
            uint32_t rb = positive32(src);
            const int64_t nv = p.D - (int64_t)word * 32;
            if (nv < 32) rb &= (1u << (int)nv) - 1u;
            p.relubits[row * p.w32 + word] = rb;
          }
        }
        fence_async_smem();                       // the staging buffer leaves through the async proxy
        __syncwarp();
        if (lane == 0) {
          bar_arrive(&sm.staged[b]);
          bar_arrive(&sm.empty[s]);
        }
        ++n;
      }
    }
  } else if (warp == kLoaderWarp) {
    // ---------------------------------------------------------------------------------------------
    // loader: claims chunks one ahead of the loads it issues, so that the compute warps can run the
    // first phase of the next chunk before the second phase of the current one.
    // ---------------------------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t n = 0, seq_claim = 0;
      bool more = true;
      auto claim = [&]() -> uint32_t {
        const uint32_t t = atomicAdd(p.ticket, 1u);
        const uint32_t id = t < nchunks ? t : kNoChunk;
        const int slot = seq_claim % kSlots;
        sm.chunk_id[slot] = id;
        bar_arrive(&sm.chunk_ready[slot]);
        ++seq_claim;
        if (id == kNoChunk) more = false;
        return id;
      };
      uint32_t cur = claim();
      uint32_t nxt = more ? claim() : kNoChunk;
      bool ok = true;
      while (ok && cur != kNoChunk) {
        for (int g = 0; g < kChunk && ok; ++g) {
          const uint32_t tile = cur * kChunk + g;
          if (tile >= ntiles) break;
          const int s = n % S;
          if (!bar_wait(&sm.empty[s], ((n / S) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t slab = tile / (uint32_t)p.ncb, cb = tile - slab * (uint32_t)p.ncb;
          bar_arrive_expect_tx(&sm.full[s], (uint32_t)(kTileElems * sizeof(T)));
          tma_load_tile(sm.raw[s], &tmA, (int)(cb * kTileCols), (int)(slab * kTileRows), &sm.full[s]);
          ++n;
        }
        cur = nxt;
        nxt = (ok && more) ? claim() : kNoChunk;
      }
      if (*abort_flag != 0) {
        // loads already issued still write this CTA's shared memory: wait for the last one of each stage
        const uint32_t first = n > (uint32_t)S ? n - S : 0u;
        for (uint32_t i = first; i < n; ++i) {
          const uint64_t t0 = timer_ns();
          while (!bar_try_wait(&sm.full[i % S], (i / S) & 1u) && timer_ns() - t0 < kPipeWaitLimitNs) {}
        }
      }
    }
  } else if (warp == kLookbackWarp) {
    // ---------------------------------------------------------------------------------------------
    // look-back: one status word per chunk (flag, padded prefix in granules of 8, exact count)
    // ---------------------------------------------------------------------------------------------
    for (uint32_t seq = 0;; ++seq) {
      const int slot = seq % kSlots;
      const uint32_t par = (seq / kSlots) & 1u;
      if (!bar_wait(&sm.chunk_ready[slot], par, abort_flag)) break;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) break;
      if (!bar_wait(&sm.cnt_ready[slot], par, abort_flag)) break;
      // lane (8 g + w) reads warp w's total of tile g; a butterfly over eight lanes sums a tile
      static_assert(kChunk * kComputeWarps == 32, "one lane per (tile, warp)");
      uint32_t t = sm.warp_total[slot][lane >> 3][lane & 7];
      t += __shfl_xor_sync(0xffffffffu, t, 1);
      t += __shfl_xor_sync(0xffffffffu, t, 2);
      t += __shfl_xor_sync(0xffffffffu, t, 4);
      uint32_t tot[kChunk], gran[kChunk];
      uint32_t chunk_gran = 0, chunk_exact = 0;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) {
        tot[g] = __shfl_sync(0xffffffffu, t, 8 * g);
        gran[g] = (tot[g] + kValueAlign - 1) / kValueAlign;
        chunk_gran += gran[g];
        chunk_exact += tot[g];
      }
      if (lane == 0)
        store_status(p.status + chunk, ((chunk == 0 ? kFlagPrefix : kFlagAggregate) << kFlagShift) |
                                           pack_counts(chunk_gran, chunk_exact));
      uint64_t excl = 0;
      bool failed = false;
      if (chunk != 0) {
        int64_t idx = (int64_t)chunk - 1;
        bool done = false;
        while (!done) {
          const int64_t j = idx - lane;
          uint64_t w = kFlagPrefix << kFlagShift;          // before the first chunk: prefix 0
          if (j >= 0) {
            int spins = 0;
            w = load_status(p.status + j);
            while ((w >> kFlagShift) == 0 && spins < kSpinLimit) {
              __nanosleep(spins < 64 ? 32 : 256);
              w = load_status(p.status + j);
              ++spins;
            }
          }
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
      if (failed) {
        if (lane == 0) {
          store_status(p.status + chunk, kFlagPoison << kFlagShift);   // later chunks stop waiting too
          raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
        }
      } else if (lane == 0 && chunk != 0) {
        store_status(p.status + chunk, (kFlagPrefix << kFlagShift) | (excl + pack_counts(chunk_gran, chunk_exact)));
      }
      int64_t base = (int64_t)(excl >> 32) * kValueAlign;
      bool over = false;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) {
        const uint32_t tile = chunk * kChunk + g;
        if (tile < ntiles) {
          const int64_t padded = (int64_t)gran[g] * kValueAlign;
          const bool fits = base + padded <= p.capacity;
          over = over || !fits;
          if (lane == 0) {
            if (!failed) p.offsets[tile] = (uint32_t)base;
            sm.tile_total[slot][g] = tot[g];
            sm.tile_base[slot][g] = (failed || !fits) ? -1 : base;
          }
          base += padded;
        }
      }
      if (lane == 0 && !failed) {
        if (over) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
        if (chunk == nchunks - 1) {
          p.offsets[ntiles] = (uint32_t)base;
          p.nnz[0] = (int64_t)((excl & 0xffffffffu) + chunk_exact);
          p.nnz[1] = base;
        }
      }
      __syncwarp();
      if (lane == 0) bar_arrive(&sm.base_ready[slot]);
    }
  } else {
    // ---------------------------------------------------------------------------------------------
    // output: one bulk copy per tile from the staging buffer to `values`
    // ---------------------------------------------------------------------------------------------
    uint32_t n = 0;
    bool ok = true;
    for (uint32_t seq = 0; ok; ++seq) {
      const int slot = seq % kSlots;
      const uint32_t par = (seq / kSlots) & 1u;
      if (!bar_wait(&sm.chunk_ready[slot], par, abort_flag)) break;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) break;
      if (!bar_wait(&sm.base_ready[slot], par, abort_flag)) break;
      for (int g = 0; g < kChunk; ++g) {
        const uint32_t tile = chunk * kChunk + g;
        if (tile >= ntiles) break;
        const int b = n & 1;
        const uint32_t total = sm.tile_total[slot][g];
        const int64_t base = sm.tile_base[slot][g];
        const uint32_t padded = (total + kValueAlign - 1) / kValueAlign * kValueAlign;
        if (!bar_wait(&sm.staged[b], (n >> 1) & 1u, abort_flag)) { ok = false; break; }
        if (total + lane < padded) sm.outv[b][total + lane] = from_float<T>(0.0f);
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (base >= 0 && padded != 0) {
            bulk_store(static_cast<T*>(p.values) + base, sm.outv[b], padded * (uint32_t)sizeof(T));
            bulk_store_wait_read();
          }
          bar_arrive(&sm.out_free[b]);
        }
        ++n;
      }
    }
    if (lane == 0) bulk_store_wait_all();
  }
  __syncthreads();
  if (tid == 0 && sm.abort_flag != 0) raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <typename T, int S>
int launch_typed(const StoreParams& p, const PhiloxKeys& ks, const CUtensorMap& map, cudaStream_t s) {
  static int grid_cap[64] = {};                   // resident CTAs per device, found once
  int dev = 0;
  RAD_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return RAD_EUNSUPPORTED;
  const size_t smem = sizeof(PipeSmem<T, S>) + 128;
  auto kernel = store_pipelined_kernel<T, S>;
  if (grid_cap[dev] == 0) {
    RAD_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0, sms = 0;
    RAD_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPipeThreads, smem));
    RAD_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (per_sm <= 0 || sms <= 0) return RAD_ECUDA;
    grid_cap[dev] = per_sm * sms;
  }
  const int64_t nchunks = ceil_div(p.ntiles, kChunk);
  const int grid = (int)std::min<int64_t>(nchunks, grid_cap[dev]);
  count_launch();
  kernel<<<grid, kPipeThreads, smem, s>>>(p, ks, map);
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}

}  // namespace

int launch_store_pipelined(const StoreParams& p, const PhiloxKeys& ks, int dtype, cudaStream_t s) {
  const size_t esz = dtype == RAD_BF16 ? 2 : 4;
  if (((uintptr_t)p.A & 15) != 0 || ((size_t)p.lda * esz) % 16 != 0) return RAD_EUNSUPPORTED;
  EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(tensor_map_encoder());
  if (fn == nullptr) return RAD_EUNSUPPORTED;
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)p.D, (cuuint64_t)p.B};
  const cuuint64_t strides[1] = {(cuuint64_t)p.lda * esz};
  const cuuint32_t box[2] = {(cuuint32_t)kTileCols, (cuuint32_t)kTileRows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(&map, dtype == RAD_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        const_cast<void*>(p.A), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return RAD_EUNSUPPORTED;
  if (dtype == RAD_BF16) return launch_typed<bf16, 3>(p, ks, map, s);
  return launch_typed<float, 2>(p, ks, map, s);
}

}  // namespace rad
