// Shared by the two different-sample store kernels: launch parameters and the look-back status word.
#pragma once

#include "common.cuh"

namespace rad {

// ---- look-back status word ---------------------------------------------------------------------
// bits 63..62 flag, 61..32 padded prefix in granules of 8 elements, 31..0 exact kept count.
constexpr uint64_t kFlagShift = 62;
constexpr uint64_t kFlagAggregate = 1, kFlagPrefix = 2, kFlagPoison = 3;
constexpr uint64_t kValueMask = (1ull << kFlagShift) - 1;

// Bounded wait for a status word to get its flag: polls with a back-off of 32 ns, then 256 ns, and gives up
// (returns the word with flag 0) once `limit_ns` has passed.
__device__ __forceinline__ uint64_t load_status(const uint64_t* p);
__device__ __forceinline__ uint64_t wait_status(const uint64_t* p, uint64_t limit_ns) {
  uint64_t w = load_status(p);
  if ((w >> kFlagShift) != 0) return w;
  uint64_t t0;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (int spins = 0;; ++spins) {
    __nanosleep(spins < 64 ? 32 : 256);
    w = load_status(p);
    if ((w >> kFlagShift) != 0) return w;
    if ((spins & 15) == 15) {
      uint64_t t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      if (t - t0 > limit_ns) return w;
    }
  }
}

__device__ __forceinline__ uint64_t pack_counts(uint32_t granules, uint32_t exact) {
  return ((uint64_t)granules << 32) | exact;
}
__device__ __forceinline__ uint64_t load_status(const uint64_t* p) {
  uint64_t v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void store_status(uint64_t* p, uint64_t v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint64_t warp_sum_u64(uint64_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

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

struct StoreParams {
  const void* A;
  int64_t lda;
  int64_t B, D;
  int32_t ncb;        // column blocks
  int32_t ntiles;
  KeepThreshold T;    // keep threshold
  float scale;
  uint32_t c2, c3;    // counter words 2 and 3
  void* values;
  int64_t capacity;
  uint32_t* keepbits;
  uint32_t* offsets;
  int64_t* nnz;
  uint32_t* relubits;
  int32_t w32;        // relu-bit words per row
  uint64_t* status;   // ntiles look-back words (zeroed before launch)
  uint32_t* ticket;   // zeroed before launch
  int32_t* dev_status;
  uint64_t wait_limit_ns;   // every device-side wait of the launch gives up after this long
  int32_t vec_ok;     // rows are 16-byte aligned: 8-element vector loads allowed
  // with-replacement law: multiplicities, one byte per entry, rows of ldc bytes (ldc a multiple of 16);
  // nullptr: Bernoulli keeps drawn in the kernel
  const uint8_t* counts;
  int64_t ldc;
};

// store_pipe.cu: the persistent TMA-fed kernel.  RAD_EUNSUPPORTED (nothing enqueued) when the input does not
// meet the alignment rules of a tensor map; the caller then takes the generic kernel.
int launch_store_pipelined(const StoreParams& p, const PhiloxKeys& ks, int dtype, cudaStream_t s, bool fill = false);

}  // namespace rad
