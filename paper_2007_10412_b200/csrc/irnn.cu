// ReLU recurrent net (IRNN) with a fresh activation sample at every time step (paper, Sec. 4.3:
// "we sample different activations at each time-step"; App. A: per step the hidden state entering
// the cell is kept at the sampling fraction, the scalar input whole, ReLU derivatives at 1 bit).
//
// The recurrence of one minibatch row never looks at another row, so one CTA owns one row for all
// T steps and no CTA ever waits for another.  Four warps carry the hidden units (one per thread,
// the unit's column of W_hh in registers, the state broadcast from shared memory); a fifth warp
// draws the step's Philox mask, compacts the kept entries of h_{t-1} and writes keep bits and
// offsets.  Backward through time mirrors it: the fifth warp prefetches a step's kept entries into
// shared memory while the others form dz_t, dh_{t-1} = dz_t W_hh^T and the row's share of dW_hh;
// per-row partial gradients are summed over rows in row order by a last kernel.
#include <algorithm>
#include <cmath>

#include "common.cuh"

namespace rad {
namespace {

constexpr int kHdMax = 128;          // hidden units per CTA row (one thread each)
constexpr int kRnnThreads = 160;     // backward: 4 unit warps + 1 helper warp
constexpr int kRnnFwdThreads = 192;  // forward: 4 unit warps, the store warp, the warp that draws the masks

struct RnnParams {
  int64_t B, T;
  int32_t Hd, w32, ngroups;
  int32_t same;                      // same-sample: the mask does not depend on the row
  KeepThreshold keepT;               // keep threshold
  float scale;
  uint32_t c2, step0;
  const float* x;                    // B x T
  const float* W_ih; const float* b_ih; const float* W_hh; const float* b_hh;
  float* h_last;                     // B x Hd
  float* values; int64_t cap_row;    // B x cap_row
  uint32_t* offsets;                 // T x B: start of step t's values inside the row's region
  uint32_t* keepbits;                // T x B x w32
  uint32_t* relubits;                // T x B x w32: (h_t > 0)
  int64_t* nnz_rows;                 // B: kept entries of the row over all steps
  // backward
  const float* dh_last;              // B x Hd
  float* part_whh;                   // B x Hd x Hd
  float* part_vec;                   // B x 2 x Hd: dW_ih, db
  int32_t* dev_status;
};

__global__ void __launch_bounds__(kRnnFwdThreads) irnn_forward_kernel(const RnnParams p, const PhiloxKeys ks) {
  extern __shared__ float sm[];
  float* s_x = sm;                                   // T inputs of this row
  __shared__ __align__(16) float s_h[2][kHdMax];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t b = blockIdx.x;
  const int Hd = p.Hd;
  for (int64_t t = tid; t < p.T; t += kRnnFwdThreads) s_x[t] = p.x[b * p.T + t];
  if (tid < kHdMax) { s_h[0][tid] = 0.0f; s_h[1][tid] = 0.0f; }
  // unit j keeps column j of W_hh in registers (zero beyond Hd)
  float wcol[kHdMax];
  float bias = 0.0f, wih = 0.0f;
  const int j = tid;
  if (warp < 4) {
#pragma unroll
    for (int k = 0; k < kHdMax; ++k) wcol[k] = (k < Hd && j < Hd) ? p.W_hh[(int64_t)k * Hd + j] : 0.0f;
    if (j < Hd) { bias = p.b_ih[j] + p.b_hh[j]; wih = p.W_ih[j]; }
  }
  // The keep decisions need no data: the sixth warp draws the words of step t + 2 while step t runs (one
  // keep-bit word decides 32 units; four lanes make it together, one generator output each).
  __shared__ uint32_t s_mask[4][8];
  const uint32_t mask_row = p.same ? 0u : (uint32_t)b;
  auto draw = [&](int64_t t) {
    const uint32_t m = philox_keep32_quad((uint32_t)(lane >> 2), mask_row, p.c2, p.step0 + (uint32_t)t, ks, p.keepT, lane);
    if ((lane & 3) == 0) s_mask[t & 3][lane >> 2] = m;
  };
  if (warp == 5) {
    draw(1);
    if (p.T >= 2) draw(2);
  }
  __syncthreads();
  uint32_t off = 0;                                  // store warp: values of this row so far
  for (int64_t t = 1; t <= p.T; ++t) {
    const float* hc = s_h[(t - 1) & 1];
    if (warp == 5) {
      if (t + 2 <= p.T) draw(t + 2);
    } else if (warp == 4) {
      // store of h_{t-1}: keep bits of the step, kept entries scaled and appended to the row's values
      // four lanes share a keep-bit word and place eight of its units each
      const int wi = lane >> 2, q = lane & 3;
      uint32_t m = s_mask[t & 3][wi];
      const bool word_ok = wi * 32 < Hd;
      m = word_ok ? m & (0xffffffffu >> (32 - min(32, Hd - wi * 32))) : 0u;
      // the word's count enters the scan once (first lane of the four); every lane then places a quarter of it
      const uint32_t c = q == 0 ? __popc(m) : 0u;
      uint32_t incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
      const uint32_t word_pos = __shfl_sync(0xffffffffu, off + incl - c, lane & ~3);
      if ((int64_t)off + total <= p.cap_row) {
        // units 8 q .. 8 q + 7 of the word: loaded whether kept or not (two 16-byte loads instead of up to
        // eight dependent ones), stored where kept
        const uint32_t sub = (m >> (8 * q)) & 0xffu;
        if (sub != 0) {
          const float4 lo = *reinterpret_cast<const float4*>(hc + wi * 32 + 8 * q);
          const float4 hi = *reinterpret_cast<const float4*>(hc + wi * 32 + 8 * q + 4);
          const float v[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
          float* out = p.values + b * p.cap_row + word_pos + __popc(m & ((1u << (8 * q)) - 1u));
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if ((sub >> i) & 1u) *out++ = v[i] * p.scale;
        }
      } else if (lane == 0) {
        raise_status(p.dev_status, RAD_DEV_ECAPACITY);
      }
      const int64_t sb = (t - 1) * p.B + b;
      if (q == 0 && wi < p.w32) p.keepbits[sb * p.w32 + wi] = m;
      if (lane == 0) p.offsets[sb] = off;
      off += total;
    } else {
      // z_j = x_t W_ih[j] + b_ih[j] + b_hh[j] + sum_k h_{t-1}[k] W_hh[k][j]
      // four partial sums keep the FMA pipe busy; they are combined in a fixed order
      float z0 = fmaf(s_x[t - 1], wih, bias), z1 = 0.0f, z2 = 0.0f, z3 = 0.0f;
#pragma unroll
      for (int k = 0; k < kHdMax; k += 4) {
        const float4 h4 = *reinterpret_cast<const float4*>(hc + k);
        z0 = fmaf(h4.x, wcol[k], z0); z1 = fmaf(h4.y, wcol[k + 1], z1);
        z2 = fmaf(h4.z, wcol[k + 2], z2); z3 = fmaf(h4.w, wcol[k + 3], z3);
      }
      const float z = (z0 + z1) + (z2 + z3);
      const float hn = (j < Hd) ? fmaxf(z, 0.0f) : 0.0f;
      s_h[t & 1][j] = hn;
      const uint32_t bits = __ballot_sync(0xffffffffu, hn > 0.0f);
      if (lane == 0 && warp < p.w32) p.relubits[((t - 1) * p.B + b) * p.w32 + warp] = bits;
    }
    __syncthreads();
  }
  if (warp < 4 && j < Hd) p.h_last[b * Hd + j] = s_h[p.T & 1][j];
  if (warp == 4 && lane == 0) p.nnz_rows[b] = off;
}

constexpr int kRing = 8;             // steps of kept entries in flight in the backward kernel

__global__ void __launch_bounds__(kRnnThreads) irnn_backward_kernel(const RnnParams p) {
  extern __shared__ float sm[];
  const int Hd = p.Hd;
  const int S = Hd + 1;                               // odd stride: conflict-free rows and columns
  const int64_t Tp = (p.T + 3) & ~(int64_t)3;
  float* s_x = sm;                                    // T
  float* s_dw = s_x + Tp;                             // Hd x S: this row's share of dW_hh
  uint32_t* s_keep = reinterpret_cast<uint32_t*>(s_dw + ((Hd * S + 3) & ~3));   // T x w32 keep bits of the row
  uint32_t* s_rl = s_keep + p.T * p.w32;              // T x w32 ReLU bits
  uint32_t* s_off = s_rl + p.T * p.w32;               // T value offsets
  __shared__ __align__(16) float s_dz[2][kHdMax];
  __shared__ __align__(16) uint32_t s_kidx[kRing][kHdMax];
  __shared__ __align__(16) float s_kval[kRing][kHdMax];
  __shared__ uint32_t s_kcnt[kRing];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t b = blockIdx.x;
  for (int64_t t = tid; t < p.T; t += kRnnThreads) {
    s_x[t] = p.x[b * p.T + t];
    s_off[t] = p.offsets[t * p.B + b];
  }
  for (int64_t i = tid; i < p.T * p.w32; i += kRnnThreads) {
    const int64_t at = ((i / p.w32) * p.B + b) * p.w32 + (i % p.w32);
    s_keep[i] = p.keepbits[at];
    s_rl[i] = p.relubits[at];
  }
  for (int i = tid; i < Hd * S; i += kRnnThreads) s_dw[i] = 0.0f;
  if (tid < kHdMax) { s_dz[0][tid] = 0.0f; s_dz[1][tid] = 0.0f; }
  const int k = tid;                                  // unit k: row k of W_hh in registers
  float wrow[kHdMax];
  float dh = 0.0f, dwih = 0.0f, dbs = 0.0f, dwih_c = 0.0f, dbs_c = 0.0f;
  if (warp < 4) {
#pragma unroll
    for (int jj = 0; jj < kHdMax; ++jj) wrow[jj] = (k < Hd && jj < Hd) ? p.W_hh[(int64_t)k * Hd + jj] : 0.0f;
    if (k < Hd) dh = p.dh_last[b * Hd + k];
  }
  __syncthreads();
  // helper warp: list of the kept units of step t and an asynchronous copy of their values into
  // ring slot t % kRing; one commit group per call, so groups can be counted
  auto prefetch = [&](int64_t t) {
    if (t >= 1) {
      const int slot = (int)(t % kRing);
      uint32_t m = 0;
      if (lane < p.ngroups) m = (s_keep[(t - 1) * p.w32 + (lane >> 2)] >> (8 * (lane & 3))) & 0xffu;
      const uint32_t c = __popc(m);
      uint32_t incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
      const uint32_t off = s_off[t - 1];
      uint32_t pos = incl - c;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if ((m >> i) & 1u) s_kidx[slot][pos++] = (uint32_t)(lane * 8 + i);
      const bool fits = (int64_t)off + total <= p.cap_row;
      for (uint32_t i = lane; i < total; i += 32) {
        if (fits) {
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(&s_kval[slot][i])),
                       "l"(p.values + b * p.cap_row + off + i) : "memory");
        } else {
          s_kval[slot][i] = 0.0f;
        }
      }
      if (lane == 0) s_kcnt[slot] = total;
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if (warp == 4) {
    for (int d = 0; d < kRing - 1; ++d) prefetch(p.T - d);
    asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 2) : "memory");      // step T has landed
  }
  // dz_t = dh_t * relu'(h_t) and the exact gradients of the input weights and biases, by the thread of unit k;
  // the two buffers of dz alternate, so a step needs one barrier: the dz of step t - 1 is written at the end of
  // step t while the other threads may still read the dz of step t
  auto make_dz = [&](int64_t t) {
    const uint32_t rbits = warp < p.w32 ? s_rl[(t - 1) * p.w32 + warp] : 0u;
    const float dz = ((rbits >> lane) & 1u) ? dh : 0.0f;
    s_dz[t & 1][k] = dz;
    // compensated sums: T terms of one sign would otherwise drift past the float32 tolerance
    const float yi = fmaf(s_x[t - 1], dz, -dwih_c), ti = dwih + yi;
    dwih_c = (ti - dwih) - yi; dwih = ti;
    const float yb = dz - dbs_c, tb = dbs + yb;
    dbs_c = (tb - dbs) - yb; dbs = tb;
  };
  if (warp < 4) make_dz(p.T);
  __syncthreads();
  for (int64_t t = p.T; t >= 1; --t) {
    const int slot = (int)(t % kRing);
    if (warp < 4) {
      const float* dzv = s_dz[t & 1];
      // dh_{t-1}[k] = sum_j dz[j] W_hh[k][j]
      float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
#pragma unroll
      for (int jj = 0; jj < kHdMax; jj += 4) {
        const float4 d4 = *reinterpret_cast<const float4*>(dzv + jj);
        a0 = fmaf(d4.x, wrow[jj], a0); a1 = fmaf(d4.y, wrow[jj + 1], a1);
        a2 = fmaf(d4.z, wrow[jj + 2], a2); a3 = fmaf(d4.w, wrow[jj + 3], a3);
      }
      dh = (a0 + a1) + (a2 + a3);
      // dW_hh[kept unit d, j] += h_hat_{t-1}[d] * dz[j]: thread j owns column j of every row
      if (k < Hd) {
        const float dzj = dzv[k];
        const uint32_t cnt = s_kcnt[slot];
        uint32_t n = 0;
        // four kept units at a time: their rows of dW_hh are different, so the four updates do not wait
        // for one another
        for (; n + 4 <= cnt; n += 4) {
          const uint4 id = *reinterpret_cast<const uint4*>(&s_kidx[slot][n]);
          const float4 hv = *reinterpret_cast<const float4*>(&s_kval[slot][n]);
          float* c0 = s_dw + id.x * S + k; float* c1 = s_dw + id.y * S + k;
          float* c2 = s_dw + id.z * S + k; float* c3 = s_dw + id.w * S + k;
          const float x0 = *c0, x1 = *c1, x2 = *c2, x3 = *c3;
          *c0 = fmaf(hv.x, dzj, x0); *c1 = fmaf(hv.y, dzj, x1);
          *c2 = fmaf(hv.z, dzj, x2); *c3 = fmaf(hv.w, dzj, x3);
        }
        for (; n < cnt; ++n) {
          float* cell = s_dw + s_kidx[slot][n] * S + k;
          *cell = fmaf(s_kval[slot][n], dzj, *cell);
        }
      }
      if (t > 1) make_dz(t - 1);
    } else {
      // beside the unit warps: the list of a later step (its ring slot was read a step ago)
      prefetch(t - (kRing - 1));
      asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 2) : "memory");    // step t - 1 has landed
    }
    __syncthreads();
  }
  for (int i = tid; i < Hd * Hd; i += kRnnThreads) p.part_whh[b * Hd * Hd + i] = s_dw[(i / Hd) * S + (i % Hd)];
  if (warp < 4 && k < Hd) {
    p.part_vec[(b * 2 + 0) * Hd + k] = dwih;
    p.part_vec[(b * 2 + 1) * Hd + k] = dbs;
  }
}

// out[i] = sum over rows of part[b][i], in row order
__global__ void __launch_bounds__(256) sum_rows_kernel(const float* part, int64_t B, int64_t n, int64_t stride,
                                                       int64_t offset, float* out) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float s = 0.0f;
  for (int64_t b = 0; b < B; ++b) s += part[b * stride + offset + i];
  out[i] = s;
}

__global__ void sum_nnz_kernel(const int64_t* rows, int64_t B, int64_t* out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    int64_t s = 0;
    for (int64_t b = 0; b < B; ++b) s += rows[b];
    out[0] = s;
  }
}

struct RnnPlan {
  int64_t cap_row, values, offsets, keepbits, relubits, nnz_rows, h_last, dh_last, logits, dlogits, part_whh,
      part_vec, out_values, out_keepbits, out_offsets, out_nnz, scratch, scratch_bytes, total;
  rad_store_sizes out_sizes;
};

int make_rnn_plan(const rad_irnn_desc* d, RnnPlan* pl) {
  if (d == nullptr || d->B <= 0 || d->T <= 0 || d->Hd <= 0 || d->Hd > kHdMax || d->C <= 0) return RAD_EINVAL;
  if (d->variant != RAD_DIFFERENT_SAMPLE && d->variant != RAD_SAME_SAMPLE) return RAD_EINVAL;
  const uint32_t Tk = keep_threshold_host(d->p);
  if (Tk == 0) return RAD_EINVAL;
  const double pe = Tk / (double)kLaneRange, n = (double)d->T * d->Hd;
  int64_t cap = (int64_t)(n * pe + 8.0 * std::sqrt(n * pe * (1.0 - pe)) + 16.0);
  cap = std::min<int64_t>(round_up(cap, 4), round_up((int64_t)n, 4));
  pl->cap_row = cap;
  const int64_t w32 = ceil_div(d->Hd, 32);
  int64_t off = 0;
  auto take = [&](int64_t bytes) { const int64_t at = off; off += round_up(bytes, 256); return at; };
  pl->values = take(d->B * cap * 4);
  pl->offsets = take(d->T * d->B * 4);
  pl->keepbits = take(d->T * d->B * w32 * 4);
  pl->relubits = take(d->T * d->B * w32 * 4);
  pl->nnz_rows = take(d->B * 8);
  pl->h_last = take(d->B * d->Hd * 4);
  pl->dh_last = take(d->B * d->Hd * 4);
  pl->logits = take(d->B * d->C * 4);
  pl->dlogits = take(d->B * d->C * 4);
  pl->part_whh = take(d->B * d->Hd * d->Hd * 4);
  pl->part_vec = take(d->B * 2 * d->Hd * 4);
  int rc = rad_store_size_query(d->variant, RAD_F32, d->B, d->Hd, d->p, &pl->out_sizes);
  if (rc != RAD_OK) return rc;
  const rad_store_sizes& sz = pl->out_sizes;
  pl->out_values = take((d->variant == RAD_SAME_SAMPLE ? sz.values_worst : sz.values_typical) * 4);
  pl->out_keepbits = take(sz.keepbits_words * 4);
  pl->out_offsets = take(sz.offsets_words * 4);
  pl->out_nnz = take(16);
  pl->scratch_bytes = round_up(std::max<int64_t>(std::max<int64_t>(sz.workspace_bytes, column_sums_workspace(d->B, d->C)), d->B * 4), 256);
  pl->scratch = take(pl->scratch_bytes);
  pl->total = off;
  return RAD_OK;
}

}  // namespace
}  // namespace rad

using namespace rad;

extern "C" int rad_irnn_workspace(const rad_irnn_desc* d, int64_t* bytes, rad_step_stats* stats) {
  if (bytes == nullptr) return RAD_EINVAL;
  RnnPlan pl;
  int rc = make_rnn_plan(d, &pl);
  if (rc != RAD_OK) return rc;
  *bytes = pl.total;
  if (stats != nullptr) {
    const int64_t w32 = ceil_div(d->Hd, 32);
    rad_step_stats s = {};
    s.value_bytes = d->B * pl.cap_row * 4 + (d->variant == RAD_SAME_SAMPLE ? pl.out_sizes.values_worst : pl.out_sizes.values_typical) * 4;
    s.index_bytes = d->T * d->B * (w32 + 1) * 4 + (pl.out_sizes.keepbits_words + pl.out_sizes.offsets_words) * 4;
    s.relu_bytes = d->T * d->B * w32 * 4;
    s.unsampled_bytes = d->B * d->C * 4 + d->B * d->T * 4;          // softmax input and the scalar inputs
    s.full_backprop_bytes = d->B * (d->T * (1 + d->Hd) + d->Hd + d->C) * 4;
    *stats = s;
  }
  return RAD_OK;
}

extern "C" int rad_irnn_step(const rad_irnn_desc* d, const float* x, const int32_t* labels, const float* W_ih,
                             const float* b_ih, const float* W_hh, const float* b_hh, const float* W_out,
                             const float* b_out, float* dW_ih, float* db, float* dW_hh, float* dW_out,
                             float* db_out, float* loss, int64_t* nnz_out, void* workspace, int64_t workspace_bytes,
                             int32_t* dev_status, void* stream) {
  RnnPlan pl;
  int rc = make_rnn_plan(d, &pl);
  if (rc != RAD_OK) return rc;
  if (x == nullptr || labels == nullptr || W_ih == nullptr || b_ih == nullptr || W_hh == nullptr || b_hh == nullptr ||
      W_out == nullptr || dW_ih == nullptr || db == nullptr || dW_hh == nullptr || dW_out == nullptr ||
      db_out == nullptr || loss == nullptr)
    return RAD_EINVAL;
  if (workspace == nullptr || workspace_bytes < pl.total) return RAD_EWORKSPACE;
  if (((uintptr_t)workspace & 255) != 0) return RAD_EINVAL;
  rc = check_device();
  if (rc != RAD_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  const uint32_t Tk = keep_threshold_host(d->p);
  RnnParams p = {};
  p.B = d->B; p.T = d->T; p.Hd = (int32_t)d->Hd; p.w32 = (int32_t)ceil_div(d->Hd, 32); p.ngroups = (int32_t)ceil_div(d->Hd, 8);
  p.same = d->variant == RAD_SAME_SAMPLE ? 1 : 0;
  p.keepT = make_keep_threshold(Tk); p.scale = (float)kLaneRange / (float)Tk;
  p.c2 = counter_word2(0, d->variant); p.step0 = d->step0;
  p.x = x; p.W_ih = W_ih; p.b_ih = b_ih; p.W_hh = W_hh; p.b_hh = b_hh;
  p.h_last = reinterpret_cast<float*>(ws + pl.h_last);
  p.values = reinterpret_cast<float*>(ws + pl.values); p.cap_row = pl.cap_row;
  p.offsets = reinterpret_cast<uint32_t*>(ws + pl.offsets);
  p.keepbits = reinterpret_cast<uint32_t*>(ws + pl.keepbits);
  p.relubits = reinterpret_cast<uint32_t*>(ws + pl.relubits);
  p.nnz_rows = reinterpret_cast<int64_t*>(ws + pl.nnz_rows);
  p.dh_last = reinterpret_cast<float*>(ws + pl.dh_last);
  p.part_whh = reinterpret_cast<float*>(ws + pl.part_whh);
  p.part_vec = reinterpret_cast<float*>(ws + pl.part_vec);
  p.dev_status = dev_status;
  const PhiloxKeys ks = philox_expand_key(d->seed);
  const size_t smem_f = (size_t)d->T * 4;
  const int64_t w32s = ceil_div(d->Hd, 32);
  const size_t smem_b = (size_t)((d->T + 3) & ~(int64_t)3) * 4 + (size_t)((d->Hd * (d->Hd + 1) + 3) & ~3) * 4 +
                        (size_t)d->T * (2 * w32s + 1) * 4;
  if (smem_f > 200 * 1024 || smem_b > 200 * 1024) return RAD_ELIMIT;
  RAD_CUDA_TRY(cudaFuncSetAttribute(irnn_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)std::max<size_t>(smem_f, 1024)));
  RAD_CUDA_TRY(cudaFuncSetAttribute(irnn_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_b));
  count_launch();
  irnn_forward_kernel<<<(unsigned)d->B, kRnnFwdThreads, smem_f, s>>>(p, ks);
  RAD_CUDA_TRY(cudaGetLastError());

  // output layer on the last hidden state: sampled like any other layer input (layer index 1)
  rad_store st = {};
  st.variant = d->variant; st.dtype = RAD_F32; st.B = d->B; st.D = d->Hd; st.p = d->p;
  st.layer = 1; st.step = d->step0; st.seed = d->seed;
  st.values = ws + pl.out_values;
  st.values_ld = d->variant == RAD_SAME_SAMPLE ? pl.out_sizes.values_ld_worst : 0;
  st.values_capacity = d->variant == RAD_SAME_SAMPLE ? pl.out_sizes.values_worst : pl.out_sizes.values_typical;
  st.keepbits = reinterpret_cast<uint32_t*>(ws + pl.out_keepbits);
  st.offsets = reinterpret_cast<uint32_t*>(ws + pl.out_offsets);
  st.nnz = reinterpret_cast<int64_t*>(ws + pl.out_nnz);
  st.relubits = nullptr;
  rc = rad_linear_forward_store(p.h_last, d->Hd, &st, ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
  if (rc != RAD_OK) return rc;
  float* logits = reinterpret_cast<float*>(ws + pl.logits);
  float* dlogits = reinterpret_cast<float*>(ws + pl.dlogits);
  rc = rad_linear_forward(RAD_F32, RAD_ACT_NONE, d->B, d->Hd, d->C, p.h_last, d->Hd, W_out, d->C, b_out, nullptr, 0,
                          logits, d->C, nullptr, 0, nullptr, dev_status, stream);
  if (rc != RAD_OK) return rc;
  rc = rad_softmax_xent(RAD_F32, d->B, d->C, logits, d->C, labels, loss, dlogits, d->C, ws + pl.scratch,
                        pl.scratch_bytes, stream);
  if (rc != RAD_OK) return rc;
  rc = rad_linear_weight_grad(&st, dlogits, d->C, d->C, dW_out, d->C, nullptr, 0, dev_status, stream);
  if (rc != RAD_OK) return rc;
  rc = rad_linear_input_grad(RAD_F32, d->B, d->Hd, d->C, dlogits, d->C, W_out, d->C, nullptr, nullptr, 0,
                             ws + pl.dh_last, d->Hd, db_out, ws + pl.scratch, pl.scratch_bytes, dev_status, stream);
  if (rc != RAD_OK) return rc;

  count_launch(5);
  irnn_backward_kernel<<<(unsigned)d->B, kRnnThreads, smem_b, s>>>(p);
  const int64_t hh = d->Hd * d->Hd;
  sum_rows_kernel<<<(unsigned)ceil_div(hh, 256), 256, 0, s>>>(p.part_whh, d->B, hh, hh, 0, dW_hh);
  sum_rows_kernel<<<(unsigned)ceil_div(d->Hd, 256), 256, 0, s>>>(p.part_vec, d->B, d->Hd, 2 * d->Hd, 0, dW_ih);
  sum_rows_kernel<<<(unsigned)ceil_div(d->Hd, 256), 256, 0, s>>>(p.part_vec, d->B, d->Hd, 2 * d->Hd, d->Hd, db);
  if (nnz_out != nullptr) {
    sum_nnz_kernel<<<1, 32, 0, s>>>(p.nnz_rows, d->B, nnz_out);
    RAD_CUDA_TRY(cudaMemcpyAsync(nnz_out + 1, st.nnz, 8, cudaMemcpyDeviceToDevice, s));
  }
  RAD_CUDA_TRY(cudaGetLastError());
  return RAD_OK;
}
