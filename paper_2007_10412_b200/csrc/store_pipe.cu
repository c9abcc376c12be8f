// Different-sample store as a persistent, software-pipelined kernel (Sec. 3.2 / 4.2 of the paper: the
// layer input is sampled, scaled by 1 / p_eff and only the kept entries are held).
//
// A CTA claims chunks of kChunk consecutive 64 x 128 tiles in ticket order.  Its warps have four roles:
//   drawing    four warps that need no data: a thread draws the 64 keep decisions of two adjacent keep-bit
//              words of a row (six Philox calls), writes the words to `keepbits`, and the warp's kept count
//              per tile goes to shared memory.  They run kAhead + 1 chunks ahead of the loads, and their
//              multiplies fill the issue slots that the other warps leave while they wait for memory;
//   look-back  one warp adds the chunk's padded and exact counts, publishes them, and finds where the chunk
//              starts in `values` from the chunks before it (decoupled look-back over one status word per
//              chunk);
//   loader     one warp claims chunks and runs a ring of TMA loads of the tiles of A;
//   compaction eight warps, two tiles side by side, four warps each: a thread reads its two words back, a
//              warp scan over the counts gives every word its place in (row, column) order; each thread
//              walks the set bits of its two words and copies the kept entries into its warp's staging
//              buffer, which the warp then writes to `values` in 16-byte vectors, scaling on the way.  No
//              compaction warp waits for another one.
// The look-back of a chunk has about kAhead chunk periods to finish in.
// The layout produced is the one of the generic kernel: the order of tiles in `values` is the tile index.
//
// Every wait is bounded (a kernel argument, 2 s on the global timer unless the caller sets it).  On expiry the CTA raises RAD_DEV_ETIMEOUT, all
// roles leave their loops, outstanding loads are waited for, and the kernel returns.
#include <cuda.h>

#include <type_traits>

#include "common.cuh"
#include "store.cuh"

namespace rad {
namespace {

constexpr int kChunk = 8;                       // tiles per claimed chunk
constexpr int kComputeWarps = 8;
constexpr int kWarpsPerTile = 4;                // 128 threads per tile: two keep-bit words (64 columns of a row) each
constexpr int kTilesPerStep = kComputeWarps / kWarpsPerTile;   // tiles the compute warps work on side by side
constexpr int kDrawWarps = kWarpsPerTile;       // one per quarter of a tile
constexpr int kLoaderWarp = kComputeWarps + kDrawWarps;   // the look-back warp is the last one
constexpr int kPipeThreads = (kComputeWarps + kDrawWarps + 2) * 32;
constexpr int kAhead = 2;                       // chunks between the first and the second phase
constexpr int kSlots = 8;                       // chunk descriptors in flight
constexpr int kLookWindows = 8;                 // look-back: 32 status words per window
constexpr uint32_t kNoChunk = 0xffffffffu;
constexpr int kTileElems = kTileRows * kTileCols;
constexpr int kWarpElems = kTileElems / kWarpsPerTile;   // entries of a tile that one warp owns (16 rows)

template <typename T, int S>
struct PipeSmem {
  alignas(128) T raw[S][kTileElems];            // tiles of A as loaded
  alignas(16) T wbuf[kComputeWarps][kWarpElems + 8];   // kept values of a warp's sixteen rows, in order (from index 0 .. 7)
  uint64_t full[S], empty[S];                   // raw ring
  uint64_t chunk_ready[kSlots], cnt_ready[kSlots], base_ready[kSlots];
  uint32_t chunk_id[kSlots];
  uint32_t tile_slab[kSlots][kChunk], tile_cb[kSlots][kChunk];   // row slab and column block of each tile
  uint32_t warp_total[kSlots][kChunk][kWarpsPerTile];
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
// Bounded wait; false when the CTA is giving up (this wait or another one ran out of time).  The
// slow path is kept out of line: it is rarely taken and the kernel's code should stay small.
struct PipeWait {
  volatile int* abort_flag;   // the CTA's flag: set by the wait that runs out, seen by all the others
  uint64_t limit_ns;          // time limit of the launch (a kernel argument)
};
__device__ __noinline__ bool bar_wait_slow(uint64_t* bar, uint32_t parity, const PipeWait& wc, uint32_t sleep_ns) {
  const uint64_t t0 = timer_ns();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      if (bar_try_wait(bar, parity)) return true;
      if (sleep_ns != 0) __nanosleep(sleep_ns);   // a waiting warp leaves the issue slots to the others
    }
    if (*wc.abort_flag != 0) return false;
    if (timer_ns() - t0 > wc.limit_ns) {
      *wc.abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, const PipeWait& wc, uint32_t sleep_ns = 40) {
  if (bar_try_wait(bar, parity)) return true;
  return bar_wait_slow(bar, parity, wc, sleep_ns);
}
__device__ __forceinline__ void tma_load_tile(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_addr(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_addr(bar)) : "memory");
}
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

// One entry of the working type at a 32-bit shared-memory address.
__device__ __forceinline__ uint32_t lds_elem(uint32_t a, const bf16*) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds_elem(uint32_t a, const float*) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts_elem(uint32_t a, uint32_t v, const bf16*) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ void sts_elem(uint32_t a, uint32_t v, const float*) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t scale_pair(uint32_t v, float scale) {
  const __nv_bfloat162 h2 = __floats2bfloat162_rn(__fmul_rn(__uint_as_float(v << 16), scale),
                                                  __fmul_rn(__uint_as_float(v & 0xffff0000u), scale));
  return *reinterpret_cast<const uint32_t*>(&h2);
}

// Copies entries [first, end) of a warp's staging buffer to `out` (same indices), multiplied by `scale`
// and rounded once to the working type.  wb + 0 and out + 0 are 16-byte aligned and first < 16 bytes' worth
// of entries: whole 16-byte vectors go as such, the entries before the first and after the last whole
// vector one by one (lanes 0-7 and 8-15).
template <typename T>
__device__ __forceinline__ void copy_scaled(const T* wb, T* out, uint32_t first, uint32_t end, float scale, int lane) {
  constexpr uint32_t kVec = 16 / sizeof(T);
  const uint32_t v0 = first == 0 ? 0u : kVec, v1 = end & ~(kVec - 1);
  const uint32_t head_end = min(v0, end), tail = max(v1, head_end);
  {
    const uint32_t i = lane < 8 ? first + lane : tail + (lane - 8);
    const uint32_t lim = lane < 8 ? head_end : (lane < 16 ? end : 0u);
    if (i < lim) out[i] = from_float<T>(__fmul_rn(raw_to_float(wb[i]), scale));
  }
  for (uint32_t i = v0 + kVec * lane; i < v1; i += 32 * kVec) {
    uint4 q = *reinterpret_cast<const uint4*>(wb + i);
    if constexpr (sizeof(T) == 2) {
      q.x = scale_pair(q.x, scale); q.y = scale_pair(q.y, scale);
      q.z = scale_pair(q.z, scale); q.w = scale_pair(q.w, scale);
    } else {
      q.x = __float_as_uint(__fmul_rn(__uint_as_float(q.x), scale));
      q.y = __float_as_uint(__fmul_rn(__uint_as_float(q.y), scale));
      q.z = __float_as_uint(__fmul_rn(__uint_as_float(q.z), scale));
      q.w = __float_as_uint(__fmul_rn(__uint_as_float(q.w), scale));
    }
    *reinterpret_cast<uint4*>(out + i) = q;
  }
}

// kFill: the index part of the store (keep bits, row offsets, tile offsets, nnz) is in place already, made
// from the key alone under whatever law; only the loader and the compaction warps work, a tile's place in
// `values` and a warp's place in the tile are read instead of computed, and nothing waits for a look-back.
template <typename T, int S, bool kFill>
__global__ void __launch_bounds__(kPipeThreads, 2) store_pipelined_kernel(const StoreParams p, const PhiloxKeys ks,
                                                                      const __grid_constant__ CUtensorMap tmA) {
  // A stage of the ring must always serve the same half of the compute warps: a waiter tells the phases of
  // a barrier apart by one parity bit, which only works if it has itself waited for the phase before.
  static_assert(S % kTilesPerStep == 0, "stages and tiles worked on side by side");
  extern __shared__ unsigned char smem_raw[];
  PipeSmem<T, S>& sm = *reinterpret_cast<PipeSmem<T, S>*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  volatile int* abort_flag = &sm.abort_flag;
  const PipeWait wc = {abort_flag, p.wait_limit_ns};
  const uint32_t ntiles = (uint32_t)p.ntiles;
  const uint32_t nchunks = (ntiles + kChunk - 1) / kChunk;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { bar_init(&sm.full[s], 1); bar_init(&sm.empty[s], kWarpsPerTile); }
    for (int q = 0; q < kSlots; ++q) {
      bar_init(&sm.chunk_ready[q], 1);
      bar_init(&sm.cnt_ready[q], kDrawWarps);
      bar_init(&sm.base_ready[q], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp < kComputeWarps) {
    // ---------------------------------------------------------------------------------------------
    // compaction warps.  Warps 0-3 take the even tiles of a chunk, warps 4-7 the odd ones.  Within a tile
    // warp v owns rows 16 v .. 16 v + 15 and lane l row 16 v + l / 2, columns 64 (l % 2) .. + 63: keep-bit
    // words 4 row + 2 (l % 2) and the next one.  Lane order is (row, column) order.
    // ---------------------------------------------------------------------------------------------
    const int side = warp / kWarpsPerTile, v = warp % kWarpsPerTile, half = lane & 1;
    const int r = v * 16 + (lane >> 1);
    const uint32_t nrows = (uint32_t)p.B, ncols = (uint32_t)p.D;   // B * D < 2^32 (checked by the host)
    uint32_t n = 0;                               // tiles this CTA has worked through (ring position)
#pragma unroll 1
    for (uint32_t seq = 0;; ++seq) {
      const int slot = seq % kSlots;
      const uint32_t slot_parity = (seq / kSlots) & 1u;
      if (!bar_wait(&sm.chunk_ready[slot], slot_parity, wc)) break;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) break;
      // the keep-bit words and totals of the chunk, then its place in `values`
      if (!kFill && !bar_wait(&sm.cnt_ready[slot], slot_parity, wc)) break;
      const uint32_t valid = min((uint32_t)kChunk, ntiles - chunk * kChunk);   // tiles of this chunk
      // this thread's two words of its tile in a step of the chunk, as the drawing warps left them, are
      // asked for one step ahead (kFill: with the warp's first row offset and the tile's bounds in `values`)
      struct Ahead { uint2 m; uint32_t wbase, first, end; };
      auto keep_words = [&](uint32_t g) {
        Ahead a = {make_uint2(0u, 0u), 0u, 0u, 0u};
        if (g < valid) {
          const uint32_t tile = chunk * kChunk + g;
          const uint32_t* tw = p.keepbits + tile * (uint32_t)kTileWords;
          a.m = __ldcg(reinterpret_cast<const uint2*>(tw + (uint32_t)(r * 4 + half * 2)));
          if (kFill) {
            a.wbase = __ldcg(reinterpret_cast<const uint16_t*>(tw + kBitWords) + 16 * v);
            a.first = __ldcg(p.offsets + tile);
            a.end = __ldcg(p.offsets + tile + 1);
          }
        }
        return a;
      };
      Ahead mw = keep_words((uint32_t)side);
      if (!kFill && !bar_wait(&sm.base_ready[slot], slot_parity, wc)) break;
      bool ok = true;
      T* const wb = sm.wbuf[warp];
#pragma unroll 1
      for (int i = 0; i < kChunk / kTilesPerStep; ++i) {
        const int g = kTilesPerStep * i + side;
        if ((uint32_t)g >= valid) break;
        const uint32_t tile = chunk * kChunk + g;
        const uint32_t pos = n + g;               // the tile's place in the ring of loads
        const int s = pos % S;
        const uint32_t m0 = mw.m.x, m1 = mw.m.y;
        const Ahead here = mw;
        mw = keep_words((uint32_t)g + kTilesPerStep);
        const uint32_t cnt = __popc(m0) + __popc(m1);
        const uint32_t incl = warp_inclusive_scan(cnt, lane);
        const uint32_t wtotal = __shfl_sync(0xffffffffu, incl, 31);
        uint32_t wbase;
        int64_t base;
        if (kFill) {
          wbase = here.wbase;
          base = (int64_t)here.end <= p.capacity ? (int64_t)here.first : -1;
          if (base < 0 && v == 0 && lane == 0) raise_status(p.dev_status, RAD_DEV_ECAPACITY);
        } else {
          const uint32_t wt = sm.warp_total[slot][g][lane & 3];
          wbase = __reduce_add_sync(0xffffffffu, lane < v ? wt : 0u);
          if (half == 0)
            reinterpret_cast<uint16_t*>(p.keepbits + (int64_t)tile * kTileWords + kBitWords)[r] =
                (uint16_t)(wbase + incl - cnt);
          base = sm.tile_base[slot][g];
        }
        if (!bar_wait(&sm.full[s], (pos / S) & 1u, wc)) { ok = false; break; }
        const T* src = sm.raw[s] + r * kTileCols + half * 64;
        // Kept entries go to the warp's buffer as they are; scaling waits for the copy to `values`, where
        // every lane has work.  The buffer is filled from index `lead` on, so that an entry's index in it
        // and its index in `values` agree modulo a 16-byte vector.  One loop serves both words and takes two
        // entries a turn: it runs half as long as the fullest pair of words of the warp.  Clearing the
        // lowest set bit (x & (x - 1)) is the only step one turn waits for from the turn before; the
        // columns come off it by a population count.
        constexpr uint32_t kVec = 16 / sizeof(T), kElem = sizeof(T);
        const uint32_t lead = wbase & (kVec - 1);
        uint32_t sa = smem_addr(src);                       // column 0 of the word being walked
        uint32_t da = smem_addr(wb) + (lead + incl - cnt) * kElem;
        uint32_t x = m0, x_next = m1;
        if (x == 0) { x = x_next; x_next = 0; sa += 32 * kElem; }
        while (x != 0) {
          const uint32_t below0 = x - 1u;                   // ones below the lowest set bit
          const uint32_t c0 = __popc(~x & below0);          // its column
          const uint32_t x1 = x & below0;
          const uint32_t below1 = x1 - 1u;
          const uint32_t c1 = __popc(~x1 & below1);         // 32 if there is no second one
          const uint32_t v0 = lds_elem(sa + c0 * kElem, src);
          sts_elem(da, v0, src);
          if (x1 != 0) sts_elem(da + kElem, lds_elem(sa + c1 * kElem, src), src);
          da += x1 != 0 ? 2 * kElem : kElem;
          x = x1 & below1;
          if (x == 0) { x = x_next; x_next = 0; sa += 32 * kElem; }
        }
        if (p.relubits != nullptr) {
          const uint32_t row = sm.tile_slab[slot][g] * kTileRows + r;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint32_t word = sm.tile_cb[slot][g] * 4 + half * 2 + j;
            if (row < nrows && word < (uint32_t)p.w32) {
              uint32_t rb = positive32(src + 32 * j);
              const uint32_t nv = ncols - word * 32;
              if (nv < 32) rb &= (1u << nv) - 1u;
              p.relubits[(int64_t)row * p.w32 + word] = rb;
            }
          }
        }
        __syncwarp();
        if (lane == 0) bar_arrive(&sm.empty[s]);   // the tile of A is not read again
        if (base >= 0) {
          T* out = static_cast<T*>(p.values) + base + wbase - lead;   // a multiple of 16 bytes from `values`
          const uint32_t end = lead + wtotal;
          copy_scaled(wb, out, lead, end, p.scale, lane);
          if (v == kWarpsPerTile - 1) {
            // zeros up to the next multiple of kValueAlign after the tile's last value
            const uint32_t total = wbase + wtotal;
            const uint32_t padded = (total + kValueAlign - 1) / kValueAlign * kValueAlign;
            if (total + lane < padded) out[end + lane] = from_float<T>(0.0f);
          }
        }
        __syncwarp();                             // the staging buffer is rewritten for the next tile
      }
      if (!ok) break;
      n += valid;
    }
  } else if (warp < kComputeWarps + kDrawWarps) {
    // ---------------------------------------------------------------------------------------------
    // drawing warps: the keep decisions need no data, so they run ahead of the loads, as far as the
    // loader has claimed chunks.  Warp v draws rows 16 v .. 16 v + 15 of every tile of a chunk, a lane the
    // two words it would own as a compaction lane (six Philox calls), writes them to `keepbits`, and
    // leaves the warp's kept count per tile in shared memory.
    // ---------------------------------------------------------------------------------------------
    const int v = warp - kComputeWarps, half = lane & 1;
    const int r = v * 16 + (lane >> 1);
    const uint32_t nrows = (uint32_t)p.B, ncols = (uint32_t)p.D;
    // kFew: the threshold has trailing zero digits and needs fewer generator outputs per word.  The two
    // forms are two loops, so that the usual one stays free of tests and its calls overlap.
    auto draw = [&](auto few) {
    constexpr bool kFew = decltype(few)::value;
#pragma unroll 1
    for (uint32_t seq = 0;; ++seq) {
      const int slot = seq % kSlots;
      if (!bar_wait(&sm.chunk_ready[slot], (seq / kSlots) & 1u, wc)) break;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) break;
#pragma unroll 2
      for (int g = 0; g < kChunk; ++g) {
        const uint32_t tile = chunk * kChunk + g;
        uint32_t m0 = 0, m1 = 0;
        if (tile < ntiles) {
          const uint32_t row = sm.tile_slab[slot][g] * kTileRows + r;
          const uint32_t col0 = sm.tile_cb[slot][g] * kTileCols + half * 64;
          if (row < nrows && col0 < ncols) {
            const uint32_t g32 = col0 >> 5;
            if constexpr (kFew) {
              m0 = philox_keep32_few(g32, row, p.c2, p.c3, ks, p.T);
              m1 = philox_keep32_few(g32 + 1u, row, p.c2, p.c3, ks, p.T);
            } else {
              m0 = philox_keep32(g32, row, p.c2, p.c3, ks, p.T);
              m1 = philox_keep32(g32 + 1u, row, p.c2, p.c3, ks, p.T);
            }
            const uint32_t nv = ncols - col0;     // valid columns from col0 on
            if (nv < 64) {
              m0 &= nv >= 32 ? 0xffffffffu : (1u << nv) - 1u;
              m1 &= nv <= 32 ? 0u : (1u << (nv - 32)) - 1u;
            }
          }
          *reinterpret_cast<uint2*>(p.keepbits + (tile * (uint32_t)kTileWords + (uint32_t)(r * 4 + half * 2))) =
              make_uint2(m0, m1);
        }
        const uint32_t wt = __reduce_add_sync(0xffffffffu, __popc(m0) + __popc(m1));
        if (lane == 0) sm.warp_total[slot][g][v] = wt;
      }
      __threadfence_block();                      // the words are read back by the compaction warps
      __syncwarp();
      if (lane == 0) bar_arrive(&sm.cnt_ready[slot]);
    }
    };
    if (!kFill) {
      if (p.T.outputs == kOutputsPerGroup) draw(std::false_type{}); else draw(std::true_type{});
    }
  } else if (warp == kLoaderWarp) {
    // ---------------------------------------------------------------------------------------------
    // loader: claims chunks kAhead + 1 ahead of the loads it issues, so that the compute warps can run
    // the first phase of a chunk kAhead chunks before its second phase.
    // ---------------------------------------------------------------------------------------------
    if (lane == 0) {
      uint32_t n = 0, seq_claim = 0;
      bool more = true;
      auto claim = [&]() -> uint32_t {
        const uint32_t t = atomicAdd(p.ticket, 1u);
        const uint32_t id = t < nchunks ? t : kNoChunk;
        const int slot = seq_claim % kSlots;
        sm.chunk_id[slot] = id;
        if (id != kNoChunk) {
          uint32_t slab = id * kChunk / (uint32_t)p.ncb, cb = id * kChunk - slab * (uint32_t)p.ncb;
          for (int g = 0; g < kChunk; ++g) {
            sm.tile_slab[slot][g] = slab;
            sm.tile_cb[slot][g] = cb;
            if (++cb == (uint32_t)p.ncb) { cb = 0; ++slab; }
          }
        }
        bar_arrive(&sm.chunk_ready[slot]);
        ++seq_claim;
        if (id == kNoChunk) more = false;
        return id;
      };
      uint32_t q[kAhead + 1];                     // claimed, not yet loaded, oldest first
#pragma unroll
      for (int a = 0; a <= kAhead; ++a) q[a] = more ? claim() : kNoChunk;
      bool ok = true;
      while (ok && q[0] != kNoChunk) {
        for (int g = 0; g < kChunk && ok; ++g) {
          const uint32_t tile = q[0] * kChunk + g;
          if (tile >= ntiles) break;
          const int s = n % S;
          if (!bar_wait(&sm.empty[s], ((n / S) & 1u) ^ 1u, wc, 0)) { ok = false; break; }
          const uint32_t slab = tile / (uint32_t)p.ncb, cb = tile - slab * (uint32_t)p.ncb;
          bar_arrive_expect_tx(&sm.full[s], (uint32_t)(kTileElems * sizeof(T)));
          tma_load_tile(sm.raw[s], &tmA, (int)(cb * kTileCols), (int)(slab * kTileRows), &sm.full[s]);
          ++n;
        }
#pragma unroll
        for (int a = 0; a < kAhead; ++a) q[a] = q[a + 1];
        q[kAhead] = (ok && more) ? claim() : kNoChunk;
      }
      if (*abort_flag != 0) {
        // loads already issued still write this CTA's shared memory: wait for the last one of each stage
        const uint32_t first = n > (uint32_t)S ? n - S : 0u;
        for (uint32_t i = first; i < n; ++i) {
          const uint64_t t0 = timer_ns();
          while (!bar_try_wait(&sm.full[i % S], (i / S) & 1u) && timer_ns() - t0 < p.wait_limit_ns) {}
        }
      }
    }
  } else {
    // ---------------------------------------------------------------------------------------------
    // look-back: one status word per chunk (flag, padded prefix in granules of 8, exact count)
    // ---------------------------------------------------------------------------------------------
    // A chunk's counts are published as soon as its first phase is done; its look-back starts one
    // chunk later, when the chunks before it (other CTAs work at the same pace) have published theirs.
    struct Counts { uint32_t tot[kChunk], chunk_gran, chunk_exact; };
    auto publish = [&](uint32_t seq, Counts& c) -> uint32_t {
      const int slot = seq % kSlots;
      const uint32_t par = (seq / kSlots) & 1u;
      if (!bar_wait(&sm.chunk_ready[slot], par, wc, 400)) return kNoChunk;
      const uint32_t chunk = sm.chunk_id[slot];
      if (chunk == kNoChunk) return kNoChunk;
      if (!bar_wait(&sm.cnt_ready[slot], par, wc, 400)) return kNoChunk;
      // lane (4 g + v) reads warp v's total of tile g; a butterfly over four lanes sums a tile
      static_assert(kChunk * kWarpsPerTile == 32, "one (tile, warp) entry per lane");
      uint32_t t = sm.warp_total[slot][lane >> 2][lane & 3];
      t += __shfl_xor_sync(0xffffffffu, t, 1);
      t += __shfl_xor_sync(0xffffffffu, t, 2);
      c.chunk_gran = 0;
      c.chunk_exact = 0;
#pragma unroll
      for (int g = 0; g < kChunk; ++g) {
        c.tot[g] = __shfl_sync(0xffffffffu, t, 4 * g);
        c.chunk_gran += (c.tot[g] + kValueAlign - 1) / kValueAlign;
        c.chunk_exact += c.tot[g];
      }
      if (lane == 0)
        store_status(p.status + chunk, ((chunk == 0 ? kFlagPrefix : kFlagAggregate) << kFlagShift) |
                                           pack_counts(c.chunk_gran, c.chunk_exact));
      return chunk;
    };
    Counts cur, nxt;
    uint32_t chunk = kFill ? kNoChunk : publish(0, cur);
    for (uint32_t seq = 0; chunk != kNoChunk; ++seq) {
      const int slot = seq % kSlots;
      const uint32_t chunk_nxt = publish(seq + 1, nxt);
      if (*abort_flag != 0) break;
      const uint32_t chunk_gran = cur.chunk_gran, chunk_exact = cur.chunk_exact;
      // Look-back.  The CTAs of the grid work through their chunks at the same pace, so the nearest
      // chunk whose prefix is known is typically a few hundred chunks back: every lane fetches
      // kLookWindows status words at once (all loads in flight together); the windows of 32 are
      // examined nearest first, every lane adds up what it holds, and one warp sum ends the walk.
      uint64_t mine = 0;
      bool failed = false;
      if (chunk != 0) {
        int64_t idx = (int64_t)chunk - 1;
        bool done = false;
        while (!done && !failed) {
          uint64_t w[kLookWindows];
#pragma unroll
          for (int k = 0; k < kLookWindows; ++k) {
            const int64_t j = idx - 32 * k - lane;
            w[k] = j >= 0 ? load_status(p.status + j) : (kFlagPrefix << kFlagShift);   // before chunk 0: prefix 0
          }
#pragma unroll
          for (int k = 0; k < kLookWindows; ++k) {
            if (done || failed) break;
            const int64_t j = idx - 32 * k - lane;
            if ((w[k] >> kFlagShift) == 0) w[k] = wait_status(p.status + j, p.wait_limit_ns);
            const uint64_t flag = w[k] >> kFlagShift;
            if (__any_sync(0xffffffffu, flag == 0 || flag == kFlagPoison)) { failed = true; break; }
            const uint32_t pm = __ballot_sync(0xffffffffu, flag == kFlagPrefix);
            if (pm != 0) {
              if (lane <= __ffs(pm) - 1) mine += w[k] & kValueMask;
              done = true;
            } else {
              mine += w[k] & kValueMask;
            }
          }
          idx -= 32 * kLookWindows;
        }
      }
      const uint64_t excl = warp_sum_u64(mine);
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
          const int64_t padded = (int64_t)((cur.tot[g] + kValueAlign - 1) / kValueAlign) * kValueAlign;
          const bool fits = base + padded <= p.capacity;
          over = over || !fits;
          if (lane == 0) {
            if (!failed) p.offsets[tile] = (uint32_t)base;
            sm.tile_total[slot][g] = cur.tot[g];
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
      chunk = chunk_nxt;
      cur = nxt;
    }
  }
  __syncthreads();
  if (tid == 0 && sm.abort_flag != 0) raise_status(p.dev_status, RAD_DEV_ETIMEOUT);
}

// The kernel's bounded barrier wait on a barrier nobody arrives at, in one CTA that has no loads in flight:
// the wait runs out, the abort flag goes up, and the status word reports the timeout on the way out.
__global__ void wait_probe_pipe_kernel(uint64_t limit_ns, int32_t* dev_status) {
  __shared__ uint64_t bar;
  __shared__ int flag;
  if (threadIdx.x == 0) {
    bar_init(&bar, 1);
    flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const PipeWait wc = {&flag, limit_ns};
  bool ok = true;
  if (threadIdx.x == 0) ok = bar_wait(&bar, 0u, wc, 100);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || flag != 0)) raise_status(dev_status, RAD_DEV_ETIMEOUT);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <typename T, int S, bool kFill>
int launch_typed(const StoreParams& p, const PhiloxKeys& ks, const CUtensorMap& map, cudaStream_t s) {
  static int grid_cap[64] = {};                   // resident CTAs per device, found once
  int dev = 0;
  RAD_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return RAD_EUNSUPPORTED;
  const size_t smem = sizeof(PipeSmem<T, S>) + 128;
  auto kernel = store_pipelined_kernel<T, S, kFill>;
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

int launch_wait_probe_pipe(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s) {
  count_launch();
  wait_probe_pipe_kernel<<<1, 64, 0, s>>>(limit_ns, dev_status);
  return cudaGetLastError() == cudaSuccess ? RAD_OK : RAD_ECUDA;
}

// fill: values (and ReLU bits) only, into an index part that is already in place; p.ticket must be zero.
int launch_store_pipelined(const StoreParams& p, const PhiloxKeys& ks, int dtype, cudaStream_t s, bool fill) {
  const size_t esz = dtype == RAD_BF16 ? 2 : 4;
  if (((uintptr_t)p.A & 15) != 0 || ((size_t)p.lda * esz) % 16 != 0) return RAD_EUNSUPPORTED;
  if (((uintptr_t)p.keepbits & 7) != 0) return RAD_EUNSUPPORTED;   // keep-bit words leave in pairs
  if (((uintptr_t)p.values & 15) != 0) return RAD_EUNSUPPORTED;    // kept values leave in 16-byte vectors
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
  if (fill) return dtype == RAD_BF16 ? launch_typed<bf16, 4, true>(p, ks, map, s) : launch_typed<float, 4, true>(p, ks, map, s);
  if (dtype == RAD_BF16) return launch_typed<bf16, 4, false>(p, ks, map, s);
  return launch_typed<float, 4, false>(p, ks, map, s);
}

}  // namespace rad
