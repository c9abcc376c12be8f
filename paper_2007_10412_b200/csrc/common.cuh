// Shared device/host helpers of the RAD library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/rad.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "this library is written for sm_100a only"
#endif

namespace rad {

typedef __nv_bfloat16 bf16;

constexpr int kTileRows = RAD_TILE_ROWS;
constexpr int kTileCols = RAD_TILE_COLS;
constexpr int kBitWords = kTileRows * kTileCols / 32;    // 256 keep-bit words per tile
constexpr int kTileWords = RAD_TILE_WORDS;               // plus 64 16-bit row offsets
constexpr int kValueAlign = RAD_VALUE_ALIGN;

// ---------------------------------------------------------------------------------------------
// Philox-4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0,k1); per round the counter
// becomes (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)); the key advances by the
// Weyl constants between rounds.  The ten round keys depend on the seed only, so the host
// expands them once and kernels take them by value.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

struct PhiloxKeys {
  uint32_t k0[10];
  uint32_t k1[10];
};

inline PhiloxKeys philox_expand_key(uint64_t seed) {
  PhiloxKeys ks;
  uint32_t a = (uint32_t)(seed & 0xffffffffu), b = (uint32_t)(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    ks.k0[r] = a;
    ks.k1[r] = b;
    a += kPhiloxW0;
    b += kPhiloxW1;
  }
  return ks;
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& ks, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)kPhiloxM0 * c0;
    const uint64_t p1 = (uint64_t)kPhiloxM1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ ks.k0[r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ ks.k1[r];
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// An entry is kept iff its 12-bit number u is below T (1..4096).  The numbers of 32 consecutive columns are
// laid across the twelve words w_0 .. w_11 of three generator outputs, one bit plane per word: bit c of w_i
// is the complement of bit 11 - i of the number of column c.  Comparing from the least significant digit of
// T upwards, "u < T so far" becomes (w_i | x) where the digit of T is 1 and (w_i & x) where it is 0, so the
// 32 decisions of a keep-bit word are twelve three-input logic operations, no compares.
constexpr int kLaneBits = 12;
constexpr uint32_t kLaneRange = 1u << kLaneBits;
constexpr int kOutputsPerGroup = kLaneBits / 4;   // generator outputs behind one keep-bit word

struct KeepThreshold {
  uint32_t digit[kLaneBits];   // digit[i]: all ones if bit 11 - i of T is set (T = 4096: all set)
  uint32_t start;              // decisions before any digit: none kept, or all kept for T = 4096
  int32_t outputs;             // generator outputs that can change a decision: the planes below the lowest set
                               // bit of T leave "none kept" as it is, so outputs made of such planes only are
                               // not drawn (T = 2048: one output instead of three; T = 4096: none)
};
inline KeepThreshold make_keep_threshold(uint32_t T) {
  KeepThreshold k;
  for (int i = 0; i < kLaneBits; ++i)
    k.digit[i] = (T >= kLaneRange || ((T >> (kLaneBits - 1 - i)) & 1u)) ? 0xffffffffu : 0u;
  k.start = T >= kLaneRange ? 0xffffffffu : 0u;
  k.outputs = 0;
  if (T > 0 && T < kLaneRange) {
    int lowest = 0;                                // lowest set bit of T = plane kLaneBits - 1 - lowest
    while (((T >> lowest) & 1u) == 0) ++lowest;
    k.outputs = (kLaneBits - 1 - lowest) / 4 + 1;
  }
  return k;
}

// The AND / OR steps on the four words of output j of a group (planes 4 j .. 4 j + 3), given the
// decisions x of the planes below them; the outputs are folded in from the last one to the first.
__device__ __forceinline__ uint32_t keep_fold(uint32_t x, const uint32_t (&w)[4], int j, const KeepThreshold& k) {
#pragma unroll
  for (int i = 3; i >= 0; --i) x = (w[i] & x) | ((w[i] | x) & k.digit[4 * j + i]);
  return x;
}

// Keep bits of columns 32 * group32 .. + 31 of one row: bit c = column c of the group.
__device__ __forceinline__ uint32_t philox_keep32(uint32_t group32, uint32_t row, uint32_t c2, uint32_t c3,
                                                  const PhiloxKeys& ks, const KeepThreshold& k) {
  uint32_t x = k.start;
#pragma unroll
  for (int j = kOutputsPerGroup - 1; j >= 0; --j) {
    uint32_t w[4];
    philox4x32_10((uint32_t)kOutputsPerGroup * group32 + (uint32_t)j, row, c2, c3, ks, w);
    x = keep_fold(x, w, j, k);
  }
  return x;
}
// The same word from the first k.outputs generator outputs only (see KeepThreshold): for thresholds with
// trailing zero digits.  A caller that draws several words at once tests k.outputs once and takes this
// form for all of them, so that the calls of the usual form stay in one piece and overlap.
__device__ __forceinline__ uint32_t philox_keep32_few(uint32_t group32, uint32_t row, uint32_t c2, uint32_t c3,
                                                      const PhiloxKeys& ks, const KeepThreshold& k) {
  uint32_t x = k.start;
#pragma unroll
  for (int j = kOutputsPerGroup - 1; j >= 0; --j) {
    if (j < k.outputs) {
      uint32_t w[4];
      philox4x32_10((uint32_t)kOutputsPerGroup * group32 + (uint32_t)j, row, c2, c3, ks, w);
      x = keep_fold(x, w, j, k);
    }
  }
  return x;
}

// The same word made by four adjacent lanes (4 q .. 4 q + 3, which pass the same group and row): lane j of
// the four makes output j (the fourth lane repeats the last one), the words cross over by shuffles.  Every
// lane of the warp has to call it; all four lanes get the word.
__device__ __forceinline__ uint32_t philox_keep32_quad(uint32_t group32, uint32_t row, uint32_t c2, uint32_t c3,
                                                       const PhiloxKeys& ks, const KeepThreshold& k, int lane) {
  const int j = min(lane & 3, kOutputsPerGroup - 1);
  uint32_t mine[4];
  philox4x32_10((uint32_t)kOutputsPerGroup * group32 + (uint32_t)j, row, c2, c3, ks, mine);
  uint32_t x = k.start;
#pragma unroll
  for (int o = kOutputsPerGroup - 1; o >= 0; --o) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) w[i] = __shfl_sync(0xffffffffu, mine[i], (lane & ~3) + o);
    x = keep_fold(x, w, o, k);
  }
  return x;
}

// Host-side twins of the threshold arithmetic (double rint, one float32 division).
uint32_t keep_threshold_host(float p);
inline uint32_t counter_word2(uint32_t layer, int variant, int law = RAD_LAW_BERNOULLI) {
  const uint32_t stream = (variant == RAD_SAME_SAMPLE ? 1u : 0u) + 2u * (uint32_t)law;   // 0..5
  return (layer & 0xffffffu) | (stream << 24);
}
int64_t draws_per_row_host(float fraction, int64_t D);   // k of the with-replacement law; 0: bad fraction
double store_keep_fraction(const rad_store* st);        // expected share of kept entries under the store's law

// ---------------------------------------------------------------------------------------------
// element access
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ void raise_status(int32_t* dev_status, int32_t code) {
  if (dev_status != nullptr) atomicCAS(dev_status, 0, code);
}

__device__ __forceinline__ float gelu_f(float z) {
  return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f));
}
__device__ __forceinline__ float gelu_grad_f(float z) {
  return 0.5f * (1.0f + erff(z * 0.70710678118654752440f)) +
         z * 0.39894228040143267794f * __expf(-0.5f * z * z);
}

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }
// Bytes of the index part (keep bits + row offsets, 256-byte rounded) of a tile-major store of B x D entries:
// what a RAD_REDRAWN_SAMPLE store keeps in a workspace instead of holding it.
inline int64_t redrawn_index_bytes(int64_t B, int64_t D) {
  return round_up(ceil_div(B, kTileRows) * ceil_div(D, kTileCols) * kTileWords * 4, 256);
}

#define RAD_CUDA_TRY(expr)                          \
  do {                                              \
    cudaError_t e__ = (expr);                       \
    if (e__ != cudaSuccess) return RAD_ECUDA;       \
  } while (0)

// internal launchers shared across translation units --------------------------------------------
uint64_t wait_limit_ns();       // time after which a device-side wait gives up (api.cu; rad_set_wait_limit_ns)
int launch_wait_probe_pair(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s);      // tc.cu
int launch_wait_probe_pipe(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s);      // store_pipe.cu
int launch_wait_probe_lookback(uint64_t limit_ns, int32_t* dev_status, cudaStream_t s);  // store.cu
int check_device();   // RAD_OK on an sm_100 device
void count_launch(int n = 1);   // host-side tally of kernels this library has launched
void* tensor_map_encoder();     // cuTensorMapEncodeTiled, or nullptr (tc.cu)

// random-projection variant (project.cu)
int64_t project_ld(int64_t k);
bool project_store_ok(const rad_store* st);
int64_t project_store_workspace(int dtype, int64_t D, int64_t ld);
int64_t project_weight_grad_workspace(const rad_store* st, int64_t H);
int project_forward_store(const void* A, int64_t lda, const rad_store* st, void* workspace, int64_t workspace_bytes,
                          int32_t* dev_status, void* stream);
int project_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW, int64_t ldw,
                        void* workspace, int64_t workspace_bytes, int32_t* dev_status, void* stream);
int launch_relu_bits(int dtype, const void* A, int64_t lda, int64_t B, int64_t D, uint32_t* relubits, cudaStream_t s);

// f32/bf16 CUDA-core kernels (small or unaligned problems)
int simt_forward(int dtype, int act, int64_t B, int64_t D, int64_t H, const void* A, int64_t lda,
                 const void* W, int64_t ldw, const float* bias, void* out_act, int64_t ld_act,
                 float* out_z, int64_t ld_z, void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
                 cudaStream_t s);
int simt_input_grad(int dtype, int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz,
                    const void* W, int64_t ldw, const uint32_t* relubits_prev, const void* z_prev,
                    int64_t ld_zprev, void* dZ_prev, int64_t ldp, cudaStream_t s);
// The operands of an input gradient dZ_prev = (dZ W^T) * act'(.) that go with a dW of the same layer.
struct SimtInputGrad {
  const void* W; int64_t ldw;
  const uint32_t* relubits_prev; const void* z_prev; int64_t ld_zprev;
  void* dZ_prev; int64_t ldp;
};
// db: also the column sums of dZ, where the kernel can.  ig: also the input gradient, in the same launch, where
// the kernel can (*ig_done says whether it did).
int simt_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW,
                     int64_t ldw, int32_t* dev_status, cudaStream_t s,
                     float* db = nullptr, bool* db_written = nullptr,
                     const SimtInputGrad* ig = nullptr, bool* ig_done = nullptr);
int column_sums(int dtype, int64_t B, int64_t H, const void* dZ, int64_t ldz, float* db,
                void* workspace, int64_t workspace_bytes, cudaStream_t s);
int64_t column_sums_workspace(int64_t B, int64_t H);

// 3x3 convolution layers (conv.cu)
int conv_forward_pool(int dtype, int64_t B, int H, int W, int Cin, int Cout, const void* X, const void* Wt,
                      const float* bias, void* P, uint32_t* relubits, cudaStream_t st);
int conv_dz(int dtype, int64_t B, int H, int W, int Cout, const void* dP, const uint32_t* relubits, void* dZ,
            cudaStream_t st);
int conv_input_grad(int dtype, int64_t B, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, void* dX,
                    cudaStream_t st);
int64_t conv_weight_grad_workspace(int64_t B, int Cin, int Cout);
int conv_weight_grad(const rad_store* store, int H, int W, int Cin, int Cout, const void* dZ, float* dW, void* workspace,
                     int64_t workspace_bytes, cudaStream_t st);

// 3x3 convolutions on the tensor cores (conv_tc.cu)
bool conv_tc_ok(int dtype, int H, int W, int Cin, int Cout, const void* X, const void* Wt);
int conv_tc_forward_pool(int64_t B, int H, int W, int Cin, int Cout, const void* X, const void* Wt, const float* bias, void* P,
                         uint32_t* relubits, int32_t* dev_status, cudaStream_t st);
int64_t conv_tc_weight_grad_workspace(int64_t B, int H, int W, int Cin, int Cout);
int conv_tc_weight_grad(const rad_store* store, int H, int W, int Cin, int Cout, const void* dZ, float* dW, void* workspace,
                        int64_t workspace_bytes, int32_t* dev_status, cudaStream_t st);
bool conv_tc_dx_ok(int dtype, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, const void* dX);
int conv_tc_input_grad(int64_t B, int H, int W, int Cin, int Cout, const void* dZ, const void* Wt, void* dX, int32_t* dev_status,
                       cudaStream_t st);

// tcgen05 kernels (bf16, aligned)
bool tc_shape_ok(int64_t B, int64_t D, int64_t H, const void* p0, int64_t ld0, const void* p1,
                 int64_t ld1);
int tc_forward(int act, int64_t B, int64_t D, int64_t H, const void* A, int64_t lda, const void* W,
               int64_t ldw, const float* bias, void* out_act, int64_t ld_act, float* out_z,
               int64_t ld_z, void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
               int32_t* dev_status, cudaStream_t s, const rad_store* next = nullptr);
// store_index.cu: keep bits, row offsets, tile offsets and nnz of a different-sample Bernoulli store from the
// key alone (no layer input is read)
int launch_store_index(const rad_store* st, bool check_capacity, int32_t* dev_status, cudaStream_t s);
int launch_offsets_scan(uint32_t* offsets, int64_t ntiles, int64_t* nnz, int64_t capacity, int32_t* dev_status, cudaStream_t s);
// store_rows.cu: fixed-count law (exactly k columns per row): static-shape store, key-only index, re-tiling
bool rows_store_ok(const rad_store* st);
int rows_forward_store(const void* A, int64_t lda, const rad_store* st, int32_t* dev_status, cudaStream_t s);
int launch_fixed_index(const rad_store* st, bool check_capacity, int32_t* dev_status, cudaStream_t s);
int rows_to_tiles(const rad_store* rows, const rad_store* tiles, int32_t* dev_status, cudaStream_t s);
int64_t replace_extras_ld(int64_t D, int64_t k);
int launch_replace_index(const rad_store* st, uint32_t* extras, bool check_capacity, int32_t* dev_status, cudaStream_t s);
int launch_replace_extras(const void* A, int64_t lda, const rad_store* st, const uint32_t* extras, cudaStream_t s);
int tc_input_grad(int64_t B, int64_t D, int64_t H, const void* dZ, int64_t ldz, const void* W,
                  int64_t ldw, const uint32_t* relubits_prev, const void* z_prev, int64_t ld_zprev,
                  void* dZ_prev, int64_t ldp, int32_t* dev_status, cudaStream_t s);
int tc_weight_grad(const rad_store* st, const void* dZ, int64_t ldz, int64_t H, float* dW,
                   int64_t ldw, void* workspace, int64_t workspace_bytes, int32_t* dev_status,
                   cudaStream_t s);
int64_t tc_weight_grad_workspace(const rad_store* st, int64_t H);
int sm_pairs();   // SM pairs the dW plans count on (see rad_sm_pairs)

}  // namespace rad
