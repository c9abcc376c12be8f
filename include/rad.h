/*
 * rad.h - C ABI of the RAD activation-sampling library for NVIDIA B200 (sm_100a).
 *
 * The library implements the neural-network instance of Randomized Automatic
 * Differentiation (Oktay et al., ICLR 2021, Sec. 4.2): for every linear layer
 * Z = A W + b the forward pass keeps only a random subsample of the layer input
 * A (B x D), rescaled so that it is an unbiased stand-in for A, and the backward
 * pass forms the weight gradient from that subsample, dW_hat = A_hat^T dZ, while
 * dX = dZ W^T, the bias gradient and the ReLU derivative stay exact.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA global-memory addresses owned by the caller; the
 *     library allocates nothing the caller must free and keeps no pointer after
 *     the call returns.  "host" pointers are ordinary process memory.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*); no call
 *     synchronises the device.  Outputs are valid once the stream reaches the end
 *     of the enqueued work.
 *   - Return value: RAD_OK or a negative host-detected error; nothing is enqueued
 *     when an error is returned unless stated otherwise.
 *   - `dev_status` (device int32, may be NULL) receives conditions only the device
 *     can see (RAD_DEV_*).  It is sticky: the first non-zero code wins and the
 *     library never clears it.  A kernel that raises one finishes without
 *     touching memory outside the caller's buffers.
 *   - Matrices are row-major with a leading dimension in elements.
 *   - bf16 paths need D and H to be multiples of 8 and all bf16 pointers and
 *     leading dimensions to be 16-byte aligned (TMA); otherwise
 *     RAD_EUNSUPPORTED.  f32 paths have no alignment rule beyond 4 bytes.
 */
#ifndef RAD_H_
#define RAD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RAD_OK            0
#define RAD_EINVAL       (-1)  /* bad argument (null pointer, size, p outside (0,1], enum)   */
#define RAD_EUNSUPPORTED (-2)  /* not an sm_100 device, or an alignment rule is not met      */
#define RAD_ECUDA        (-3)  /* a CUDA runtime or driver call failed                       */
#define RAD_EWORKSPACE   (-4)  /* workspace_bytes is smaller than the matching *_workspace   */
#define RAD_ELIMIT       (-5)  /* the problem is larger than a fixed built-in buffer          */

#define RAD_DEV_OK        0
#define RAD_DEV_ECAPACITY 1    /* the compact store did not fit values_capacity / values_ld  */
#define RAD_DEV_ETIMEOUT  2    /* a bounded device-side wait expired                         */
#define RAD_DEV_EINTERNAL 3    /* an index left its buffer; the access was skipped (a bug)   */

typedef enum { RAD_F32 = 0, RAD_BF16 = 1 } rad_dtype;
typedef enum { RAD_DIFFERENT_SAMPLE = 0, RAD_SAME_SAMPLE = 1, RAD_PROJECT = 2, RAD_ROWS_SAMPLE = 3,
               RAD_REDRAWN_SAMPLE = 4 } rad_variant;
typedef enum { RAD_ACT_NONE = 0, RAD_ACT_RELU = 1, RAD_ACT_GELU = 2 } rad_act;

/* Geometry of the compact store (fixed; part of the data layout). */
#define RAD_TILE_ROWS   64     /* minibatch rows per tile                                    */
#define RAD_TILE_COLS   128    /* layer-input columns per tile                               */
#define RAD_VALUE_ALIGN 8      /* every tile's values start at a multiple of 8 elements      */
#define RAD_TILE_WORDS  288    /* 32-bit words of index data per tile: 256 keep-bit words    */
                               /* followed by 64 16-bit row offsets                          */

/*
 * The mask (Sec. 3.2: a random P with E[P] = I; Sec. 4.3: "same sample" /
 * "different sample").  Entry (b, d) is kept iff its 12-bit number u is below
 * T = clamp(rint(p * 4096), 1, 4096):
 *   key     = (seed & 0xffffffff, seed >> 32)
 *   words   = w_0 .. w_11: the four words of the Philox-4x32-10 outputs for
 *             counters (3 * (d / 32) + j, row, layer | stream << 24, step),
 *             j = 0, 1, 2, first output first; row = b and stream = 0 for
 *             different-sample, row = 0 and stream = 1 for same-sample
 *   u       = sum over i of (1 - bit (d % 32) of w_i) << (11 - i): the numbers of
 *             32 columns lie across the twelve words, one bit plane per word, so
 *             a keep-bit word follows from twelve AND / OR steps along the binary
 *             digits of T.
 * p_eff = T / 4096 is the probability actually sampled (within 0.1 % of p for
 * p >= 0.01) and kept values are multiplied by fl32(4096 / T) = 1 / p_eff, so
 * E[A_hat] = A exactly.
 */
/*
 * Second sampling law, the paper's own (Sec. 3.2, the example after Eq. 5: k of
 * the d coordinates drawn with replacement, P = (d / k) sum_s e_s e_s^T; App. A: a
 * fraction of the activations).  Per row (different-sample) or once per
 * layer and step (same-sample), k = ceil(fraction * D) columns are drawn; a column
 * drawn c > 0 times is kept and its entry is multiplied by fl32(c * fl32(D / k)).
 *   draw j  = 32-bit word j % 4 of the Philox-4x32-10 output for
 *             counter (j / 4, row, layer | stream << 24, step), stream = 2
 *             (different-sample, row = b) or 3 (same-sample, row = 0)
 *   column  = floor(word * D / 2^32)
 *   k       = ceil(fraction * D * (1 - 2^-22)) in double, clamped to [1, D]: the
 *             fraction is a float32, so 0.1 * 300 gives 30 and not 31.
 * The compact store has the same layout as with the Bernoulli law (a kept entry
 * carries its weight in its value), so the weight-gradient calls take it as is.
 *
 * Third law (App. A, remark under the fraction sweep: sampling without
 * replacement makes a fraction of 1.0 the exact gradient): a uniformly random
 * subset of exactly k columns, each kept with weight fl32(D / k), drawn by
 * Floyd's subset sampling: step i = 0 .. k-1 takes t = floor(word_i * (D - k + i
 * + 1) / 2^32) and adds t to the subset unless it is already in, in which case
 * it adds D - k + i; word_i as for the with-replacement law with streams 4
 * (different-sample) and 5 (same-sample).
 */
typedef enum { RAD_LAW_BERNOULLI = 0, RAD_LAW_REPLACE = 1, RAD_LAW_FIXED = 2 } rad_law;
int64_t rad_draws_per_row(float fraction, int64_t D);   /* k; 0 if the fraction is outside (0, 1] */
float   rad_replace_scale(float fraction, int64_t D);   /* fl32(D / k)                            */

uint32_t rad_keep_threshold(float p);   /* T; 0 if p is outside (0, 1]                        */
float    rad_effective_p(float p);      /* T / 4096                                           */
float    rad_scale(float p);            /* fl32(4096 / T)                                     */

/*
 * One layer's compact store: plain data, all buffers device memory of the caller.
 *
 * different-sample layout.  Rows are cut into slabs of RAD_TILE_ROWS, columns
 * into blocks of RAD_TILE_COLS; tile t = slab * ceil(D / 128) + block.
 *   keepbits : RAD_TILE_WORDS words per tile.  Word (r * 4 + w), r < 64, w < 4, of
 *              tile t holds the keep bits of row slab*64 + r, columns
 *              block*128 + 32*w .. +31, LSB first; bits of rows >= B or columns
 *              >= D are 0.  Words 256..287 hold 64 unsigned 16-bit numbers
 *              (little endian, row r in half-word r): how many kept entries of
 *              the tile lie in rows before r, i.e. where row r starts inside
 *              the tile's values.
 *   values   : the kept entries of tile t, A[b,d] * scale rounded once to `dtype`,
 *              in (row, column) order, start at element offsets[t]; the tile is
 *              padded with zeros to a multiple of RAD_VALUE_ALIGN elements.
 *   offsets  : ntiles + 1 words; offsets[ntiles] = elements used in `values`.
 *   nnz      : nnz[0] = number of kept entries, nnz[1] = offsets[ntiles].
 * same-sample layout.
 *   keepbits : ceil(D / 32) words, bit d%32 of word d/32.
 *   offsets  : kept columns in ascending order (k' entries, room for D).
 *   values   : B x values_ld row-major; values[b, j] = A[b, offsets[j]] * scale
 *              for j < k', zero for k' <= j < values_ld.
 *   nnz      : nnz[0] = k', nnz[1] = B * k'.
 * relubits (optional, either variant): B x ceil(D / 32) words row-major,
 *   bit = (A[b,d] > 0): the 1-bit ReLU derivative of the layer that produced A
 *   (Sec. 4.2).  Zero of either sign gives 0.  NULL skips it.
 */
typedef struct rad_store {
  int32_t   variant;          /* rad_variant */
  int32_t   dtype;            /* rad_dtype of A and of `values` */
  int64_t   B, D;
  float     p;                /* requested keep probability, 0 < p <= 1 */
  uint32_t  layer, step;
  uint64_t  seed;
  void*     values;
  int64_t   values_capacity;  /* elements available in `values` */
  int64_t   values_ld;        /* same-sample: leading dimension (multiple of 8); else ignored */
  uint32_t* keepbits;
  uint32_t* offsets;
  int64_t*  nnz;              /* 2 device int64 */
  uint32_t* relubits;         /* or NULL */
  int32_t   law;              /* rad_law; 0 (Bernoulli keeps) unless set.  For the other two laws */
                              /* p is the fraction: k = ceil(p * D) draws or kept columns          */
} rad_store;

typedef struct rad_store_sizes {
  int64_t values_worst;       /* elements that always suffice (p_eff = 1 plus padding)        */
  int64_t values_typical;     /* mean + 8 sigma of the kept count plus padding                */
  int64_t values_ld_worst;    /* same-sample leading dimension that always suffices           */
  int64_t values_ld_typical;  /* same-sample: mean + 8 sigma of k', rounded up to 64          */
  int64_t keepbits_words, offsets_words, relubits_words;
  int64_t workspace_bytes;    /* scratch rad_linear_forward_store needs                        */
} rad_store_sizes;

/*
 * Static-shape variant, variant = RAD_ROWS_SAMPLE with law = RAD_LAW_FIXED (App. A, remark under the fraction
 * sweep: sampling without replacement): a different sample per minibatch row as with RAD_DIFFERENT_SAMPLE, but
 * every row keeps exactly k = ceil(p * D) columns, so the store has the same shape whatever the key:
 *   values   : B x values_ld row-major (values_ld a multiple of 8, at least k; the size query gives k rounded
 *              up to 8); values[b, j] = A[b, c] * fl32(D / k) for the j-th smallest kept column c of row b,
 *              zero for k <= j < values_ld.
 *   keepbits : read as uint16: B x values_ld column numbers, cols[b, j] = c (0 for j >= k); D <= 65536.
 *   offsets  : unused, may be NULL.   nnz[0] = B * k, nnz[1] = B * values_ld.
 * The kept set of a row is the one the fixed-count law of RAD_DIFFERENT_SAMPLE keeps for the same key.
 * rad_linear_weight_grad takes such a store: it rebuilds the index part of the tile-major layout from the key
 * alone, moves the values into it (both in its workspace) and runs the same contraction.
 */

/*
 * Redrawn-mask variant, variant = RAD_REDRAWN_SAMPLE (Sec. 3.2: the random matrix is independent of the data, so
 * what is held for the backward pass need not include it): the same key, mask, `values`, `offsets` and nnz as
 * RAD_DIFFERENT_SAMPLE under the same law (Bernoulli keeps or the fixed-count law), but the keep bits and row
 * offsets are not held between the passes.  `keepbits` is unused and may be NULL.  rad_linear_forward_store and
 * rad_linear_forward_fill build the index part of the tile-major layout in their workspace; rad_linear_weight_grad
 * draws it again from the key into its workspace (one pass that reads no activation) and runs the same
 * contraction, so dW_hat is the one of RAD_DIFFERENT_SAMPLE bit for bit.  Per layer 4 bytes per tile (`offsets`)
 * are held instead of 1156; the workspaces grow by the index of one layer (rad_store_size_query,
 * rad_weight_grad_workspace).
 */

/*
 * Random-projection variant, variant = RAD_PROJECT (Sec. 3.2 after Eq. 5; App. A "Random
 * Projections for RAD"): P = R R^T with R a D x k matrix of independent Rademacher signs scaled by
 * 1 / sqrt(k), k = ceil(p * D) as for the with-replacement law.  The store is the dense block
 * S = A R' (R' the unscaled signs), rounded to `dtype`:
 *   values   : B x values_ld row-major, values[b, j] = sum_d A[b, d] R'[d, j] for j < k, zero for
 *              k <= j < values_ld (values_ld a multiple of 8, at least k; the size query gives k
 *              rounded up to 64);  nnz[0] = k, nnz[1] = B * k;  keepbits, offsets and law unused.
 *   R'[d, j] : -1 if bit j % 32 of word (j % 128) / 32 of the Philox-4x32-10 output for counter
 *              (j / 128, d, layer | 6 << 24, step) is set, else +1.  R' is not stored: both passes
 *              draw it again into their workspace.
 * rad_linear_weight_grad forms dW_hat = R' G with G = (S^T dZ) * fl32(1 / k) rounded to `dtype`: two
 * dense contractions on the same GEMM kernels as the exact paths.
 * rad_rademacher writes R' (D x ld, row-major, type `dtype`, columns k .. ld-1 zero) to `out`.
 */
int rad_rademacher(int32_t dtype, int64_t D, float fraction, int64_t ld, uint64_t seed, uint32_t layer,
                   uint32_t step, void* out /* device */, void* stream);

/* Buffer sizes for a store of the given shape (host only, nothing is launched). */
int rad_store_size_query(int32_t variant, int32_t dtype, int64_t B, int64_t D, float p,
                         rad_store_sizes* out /* host */);

/* The same for a given sampling law (rad_law): capacities follow the number of distinct columns
 * k draws hit, and the workspace holds the multiplicities (B x D bytes for different-sample). */
int rad_store_size_query_law(int32_t variant, int32_t dtype, int32_t law, int64_t B, int64_t D, float p,
                             rad_store_sizes* out /* host */);

/*
 * Forward-pass store of one layer input (Sec. 3.2, last paragraph: the layer
 * input is sparsified, never the Jacobian; Sec. 4.2 sampling of dh/dW).  Reads A (device, B x D, leading dimension lda,
 * type st->dtype), draws the mask, and fills st->keepbits / values / offsets /
 * nnz (and relubits).  `st` is a host struct read during the call.  `workspace`
 * is device scratch of at least rad_store_sizes.workspace_bytes, 256-byte
 * aligned, contents irrelevant on entry.  If the kept entries do not fit the
 * capacity, RAD_DEV_ECAPACITY is raised, the overflowing values are dropped and
 * nnz still reports the exact counts.
 */
int rad_linear_forward_store(const void* A /* device */, int64_t lda, const rad_store* st /* host */,
                             void* workspace /* device */, int64_t workspace_bytes,
                             int32_t* dev_status /* device or NULL */, void* stream);

/*
 * Which kernel the different-sample store runs (Sec. 3.2 / 4.2: same operation,
 * same layout, bit-identical output).  The persistent TMA-fed kernel is made for
 * many tiles and sparse masks, the generic one-CTA-per-tile kernel for small or
 * dense problems and for inputs a tensor map cannot describe (A or lda not
 * 16-byte aligned).  RAD_STORE_KERNEL_AUTO picks by size and keep probability;
 * the other two values force a kernel where it can run (tests use them to put
 * both kernels through the same cases).  Host only, process-wide, not
 * synchronised with calls in flight on other threads.  Returns the previous
 * setting, or RAD_EINVAL.
 */
#define RAD_STORE_KERNEL_AUTO      0
#define RAD_STORE_KERNEL_GENERIC   1
#define RAD_STORE_KERNEL_PIPELINED 2
int rad_set_store_kernel(int32_t which);

/*
 * rad_linear_forward_store without a workspace argument (the paper has no
 * counterpart: this entry point exists for the sake of callers, not of the
 * method).  It is meant for programs that must not allocate device memory
 * while they run: a trainer that hands every byte of the GPU to its own pool
 * at start-up and treats a later cudaMalloc as a bug, or a step loop in which
 * an allocation would stall the device.  Such a caller still owns A and every
 * buffer of `st`, but has nowhere to take the kernel's scratch from, so the
 * scratch (one claim counter and one 8-byte word per tile) lives in a
 * fixed array inside the library: 256 + 8 * RAD_STATIC_STORE_MAX_TILES bytes
 * (about 1 MiB), held by every GPU that has loaded the library until the
 * process exits.  The call itself allocates nothing and frees nothing.
 *
 *   - different-sample stores with Bernoulli keeps only (the same-sample path
 *     of rad_linear_forward_store needs no scratch; pass it a NULL workspace;
 *     the with-replacement law needs a B x D byte matrix, far beyond a fixed
 *     array); RAD_EUNSUPPORTED otherwise.
 *   - ceil(B / 64) * ceil(D / 128) must not exceed RAD_STATIC_STORE_MAX_TILES,
 *     else RAD_ELIMIT and nothing is enqueued.
 *   - The first call on a device looks up the array's device address (with
 *     that device current) and remembers it; make that first call outside any
 *     stream capture.
 *   - All calls on one device share the array.  Each call clears the part it
 *     uses before its kernel runs, in stream order, so back-to-back calls on
 *     one stream are fine; two calls whose kernels may overlap on the GPU
 *     (different streams, no dependency) race on it and give wrong offsets.
 * Outputs are bit for bit those of rad_linear_forward_store.
 */
#define RAD_STATIC_STORE_MAX_TILES 131072
int rad_linear_forward_store_static(const void* A /* device */, int64_t lda, const rad_store* st /* host */,
                                    int32_t* dev_status /* device or NULL */, void* stream);

/* Scratch rad_linear_weight_grad needs for this store and H (host only). */
int rad_weight_grad_workspace(const rad_store* st /* host */, int64_t H, int64_t* bytes /* host */);

/*
 * Backward-pass weight gradient from the store alone (Sec. 4.2, the sampled
 * Jacobian S_P[dh/dW] in the chain): dW[d, h] = sum_b A_hat[b, d] dZ[b, h].
 * dZ is device, B x H, type st->dtype; dW is device float32, D x H, overwritten
 * (for same-sample the rows of columns that were not kept are set to zero,
 * Sec. 4.3).  Accumulation is in float32 in a fixed order: results are
 * bit-reproducible run to run.
 */
int rad_linear_weight_grad(const rad_store* st /* host */, const void* dZ /* device */, int64_t ldz,
                           int64_t H, float* dW /* device */, int64_t ldw,
                           void* workspace /* device */, int64_t workspace_bytes,
                           int32_t* dev_status, void* stream);

/*
 * Exact forward of one layer (Sec. 3: sampling changes only what the backward pass
 * reads, the forward pass computes the unsampled network): Z = A W + bias, out = act(Z).
 *   A device B x D (dtype), W device D x H (dtype), bias device float32[H] or NULL.
 *   out_act  device B x H (dtype) or NULL: act(Z) rounded to dtype.
 *   out_z    device B x H float32 or NULL: Z before the activation (the softmax input).
 *   out_zlow device B x H (dtype) or NULL: Z rounded to dtype (kept by GELU nets).
 *   relubits device B x ceil(H/32) words or NULL: (act(Z) > 0) packed as in rad_store.
 */
int rad_linear_forward(int32_t dtype, int32_t act, int64_t B, int64_t D, int64_t H,
                       const void* A, int64_t lda, const void* W, int64_t ldw, const float* bias,
                       void* out_act, int64_t ld_act, float* out_z, int64_t ld_z,
                       void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
                       int32_t* dev_status, void* stream);

/*
 * Index part of a different-sample store from the key alone (Sec. 3.2: P is drawn independently of the
 * data).  The keep decision of entry (b, d) depends on (seed, layer, step, b, d) only, so keepbits (keep
 * words and in-tile row offsets), offsets and nnz of `st` can be written before the layer input exists: no
 * input is read.  A caller can size `values` exactly from nnz[1] (read it back after the stream has
 * reached this point), and rad_linear_forward_fill can then place the kept values from the epilogue of the
 * GEMM that produces the input.  Bernoulli keeps and the fixed-count law (RAD_EUNSUPPORTED otherwise); st->values may be NULL
 * (no capacity check) and st->relubits is not touched.  Bits and layout are those of
 * rad_linear_forward_store.
 */
int rad_store_index(const rad_store* st /* host */, int32_t* dev_status /* device or NULL */, void* stream);

/*
 * rad_linear_forward of a hidden layer fused with the store of its output as the next layer's input
 * (Sec. 3: the forward pass is the original graph; Sec. 4.2: what is kept of it is a sample of each layer
 * input): out_act = act(A W + bias) as rad_linear_forward writes it, and `next` (B x H, same dtype) filled
 * exactly as rad_linear_forward_store(out_act, next) would fill it, without reading out_act back: the
 * epilogue that holds a row of activations drops the kept ones into next->values at the places the index
 * part of `next` gives.  index_ready != 0: the caller has already run rad_store_index on `next` with the
 * same key; 0: this call runs it first.  next->relubits is ignored (the bits of out_act go to `relubits`).
 * Different-sample stores under the Bernoulli or the fixed-count law are filled this way; shapes the fused
 * kernel does not take (f32, unaligned or tiny layers, same-sample, the with-replacement law) run the
 * two separate calls instead; `workspace` (device, rad_store_sizes.workspace_bytes of `next`) is used only
 * then.
 */
int rad_linear_forward_fill(int32_t dtype, int32_t act, int64_t B, int64_t D, int64_t H,
                            const void* A, int64_t lda, const void* W, int64_t ldw, const float* bias,
                            void* out_act, int64_t ld_act, void* out_zlow, int64_t ld_zlow, uint32_t* relubits,
                            const rad_store* next /* host */, int32_t index_ready,
                            void* workspace, int64_t workspace_bytes, int32_t* dev_status, void* stream);

/*
 * Loss Jacobian (exact, Sec. 4.2: not a memory bottleneck, never sampled):
 * loss = mean_b CE(softmax(logits_b), label_b), dZ = (softmax - onehot) / B.
 *   logits device float32 B x C; labels device int32[B]; loss device float32[1];
 *   dZ device B x C (dtype).  `workspace`: device, at least 4 * B bytes.
 */
int rad_softmax_xent(int32_t dtype, int64_t B, int64_t C, const float* logits, int64_t ldl,
                     const int32_t* labels, float* loss, void* dZ, int64_t ldz,
                     void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Exact input gradient and bias gradient (Sec. 4.2: W is batch-independent, the
 * activation derivative is stored exactly):
 *   dA = dZ W^T; dZ_prev = dA * act'(.) ; db[h] = sum_b dZ[b, h].
 *   dZ device B x H (dtype); W device D x H (dtype).
 *   relubits_prev device B x ceil(D/32) words (ReLU nets) or NULL.
 *   z_prev device B x D (dtype), pre-activation of the producing layer (GELU nets) or NULL.
 *   dZ_prev device B x D (dtype) or NULL (first layer: no input gradient wanted).
 *   db device float32[H] or NULL.  `workspace`: device scratch for the column
 *   sums, at least rad_input_grad_workspace bytes.
 */
int rad_input_grad_workspace(int64_t B, int64_t H, int64_t* bytes /* host */);
int rad_linear_input_grad(int32_t dtype, int64_t B, int64_t D, int64_t H,
                          const void* dZ, int64_t ldz, const void* W, int64_t ldw,
                          const uint32_t* relubits_prev, const void* z_prev, int64_t ld_zprev,
                          void* dZ_prev, int64_t ldp, float* db,
                          void* workspace, int64_t workspace_bytes,
                          int32_t* dev_status, void* stream);

/* One training step of a fully connected net with softmax cross-entropy. */
typedef struct rad_mlp_desc {
  int32_t  L;                 /* linear layers */
  int32_t  act;               /* rad_act between layers (none after the last) */
  int32_t  dtype;             /* rad_dtype of X, W, activations, dZ */
  int32_t  variant;           /* rad_variant */
  const int64_t* dims;        /* host, L + 1 entries: fan-in of layer 1 .. fan-out of layer L */
  int64_t  B;
  float    p;
  uint32_t step;
  uint64_t seed;
  int32_t  law;               /* rad_law of every layer's store; 0 = Bernoulli keeps */
} rad_mlp_desc;

typedef struct rad_step_stats {   /* bytes held between forward and backward (App. A accounting) */
  int64_t value_bytes;            /* rad_mlp_workspace: capacity reserved for kept values (mean  */
                                  /* + 8 sigma); rad_mlp_held_bytes: what a step really kept     */
  int64_t index_bytes;            /* keep bitmasks / kept-column lists and tile offsets          */
  int64_t relu_bytes;             /* 1-bit ReLU derivatives                                      */
  int64_t preact_bytes;           /* pre-activations kept whole (GELU nets only)                 */
  int64_t unsampled_bytes;        /* the softmax input, stored whole                             */
  int64_t full_backprop_bytes;    /* what exact backprop would hold: every layer input + logits  */
} rad_step_stats;

int rad_mlp_workspace(const rad_mlp_desc* net /* host */, int64_t* bytes /* host */,
                      rad_step_stats* stats /* host or NULL */);

/*
 * The same accounting from the counts of a step that has run (App. A, "memory saved": what is held between
 * the passes): `nnz` (host, 2 * L entries) is rad_mlp_step's nnz_out copied back by the caller; value_bytes
 * then counts the kept values themselves (different-sample: with the padding of every tile to a multiple
 * of 8 elements; same-sample: B * k' per layer) instead of the reservation.  Host only; the mask depends on
 * the key alone, so rad_store_index gives the same counts before any step has run.
 */
int rad_mlp_held_bytes(const rad_mlp_desc* net /* host */, const int64_t* nnz /* host */,
                       rad_step_stats* stats /* host */);

/*
 * Forward, loss and RAD backward of the whole net on one stream (Sec. 4.2 for
 * arbitrary depth): every layer input, the network input included, is stored
 * through the mask of (seed, layer l, step); the softmax input is kept whole;
 * dW_l comes from store l, everything else is exact.
 *   X device B x dims[0] (dtype, dense); labels device int32[B];
 *   W[l] device dims[l] x dims[l+1] (dtype, dense); b[l] device float32 or NULL entries;
 *   dW[l] device float32 dims[l] x dims[l+1]; db[l] device float32; loss device float32[1].
 *   W, b, dW, db are host arrays of L device pointers.
 *   nnz_out device int64[2*L] or NULL: the nnz pair of every layer's store.
 */
int rad_mlp_step(const rad_mlp_desc* net /* host */, const void* X, const int32_t* labels,
                 const void* const* W, const float* const* b,
                 float* const* dW, float* const* db, float* loss, int64_t* nnz_out,
                 void* workspace, int64_t workspace_bytes,
                 int32_t* dev_status, void* stream);

/*
 * One training step of a ReLU recurrent net fed one scalar per time step (the paper's IRNN,
 * App. A "Architectures Used"): h_t = relu(x_t W_ih + b_ih + h_{t-1} W_hh + b_hh), h_0 = 0,
 * logits = h_T W_out + b_out, softmax cross-entropy.  RAD as in Sec. 4.3 / App. A: the hidden
 * state entering step t is stored through the mask of (seed, layer 0, step0 + t), a fresh sample
 * every step; the state entering the output layer through (seed, layer 1, step0); the scalar
 * inputs and the softmax input are kept whole; ReLU derivatives take one bit.  dW_hh and dW_out
 * come from the stores, everything else is exact.  float32 only, Hd <= 128.
 *   x device B x T; labels device int32[B]; W_ih, b_ih, b_hh device float32[Hd];
 *   W_hh device Hd x Hd (row = input unit, column = output unit); W_out device Hd x C; b_out [C].
 *   dW_ih, db (gradient of b_ih and of b_hh) device [Hd]; dW_hh device Hd x Hd; dW_out Hd x C;
 *   db_out [C]; loss device float32[1].
 *   nnz_out device int64[2] or NULL: kept hidden entries over all steps, kept entries of h_T.
 * If a row keeps more entries than its reserved share (mean + 8 sigma), RAD_DEV_ECAPACITY is raised.
 */
typedef struct rad_irnn_desc {
  int64_t  B, T, Hd, C;
  int32_t  variant;           /* rad_variant */
  float    p;
  uint64_t seed;
  uint32_t step0;             /* added to the time index in the Philox counter */
} rad_irnn_desc;

int rad_irnn_workspace(const rad_irnn_desc* net /* host */, int64_t* bytes /* host */,
                       rad_step_stats* stats /* host or NULL */);
int rad_irnn_step(const rad_irnn_desc* net /* host */, const float* x, const int32_t* labels,
                  const float* W_ih, const float* b_ih, const float* W_hh, const float* b_hh,
                  const float* W_out, const float* b_out,
                  float* dW_ih, float* db, float* dW_hh, float* dW_out, float* db_out, float* loss,
                  int64_t* nnz_out, void* workspace, int64_t workspace_bytes,
                  int32_t* dev_status, void* stream);

/*
 * One training step of a small convolutional net (paper, Fig. "Convnet activation sampling",
 * Sec. 4.2): n_conv blocks of [3x3 convolution, zero padding 1, stride 1, + bias, ReLU, 2x2
 * average pooling], then n_fc linear layers (ReLU between them, none after the last) and softmax
 * cross-entropy.  NHWC.  The input of every convolution and of every linear layer is stored
 * through the mask of (seed, layer, step), layers numbered conv blocks first: one keep decision per
 * input entry, shared by every filter tap that reads it.  ReLU derivatives take one bit per conv
 * output, average pooling and biases need nothing.  Filter and weight gradients come from the
 * stores, everything else is exact.
 *   X device B x H x W x Cin (dtype); labels device int32[B];
 *   conv_W[l] device 3 x 3 x Cin_l x Cout_l (dtype), Cout_l multiple of 8; conv_b[l] device float32 or NULL;
 *   fc_W[l] device fc_in_l x fc_dims[l] (dtype) with fc_in_0 = (H / 2^n_conv)(W / 2^n_conv) Cout_last, the
 *   pooled map flattened in (y, x, c) order; fc_b[l] device float32 or NULL;
 *   dconv_W[l], dfc_W[l] device float32, same shapes; dconv_b[l], dfc_b[l] device float32; loss float32[1].
 *   The pointer tables are host arrays.  nnz_out device int64[2 * (n_conv + n_fc)] or NULL.
 */
typedef struct rad_cnn_desc {
  int64_t  B, H, W, Cin;
  int32_t  n_conv, n_fc;
  const int64_t* conv_channels;   /* host, n_conv entries */
  const int64_t* fc_dims;         /* host, n_fc entries: outputs of the linear layers */
  int32_t  dtype, variant;
  float    p;
  uint32_t step;
  uint64_t seed;
} rad_cnn_desc;

/*
 * Which kernels the 3x3 convolutions of rad_cnn_step run (same operation either way; Fig. "Convnet activation
 * sampling").  The tensor-core kernels compute the forward convolution and the filter gradient as implicit
 * GEMMs (bf16; Cin 16, 32 or 64; Cout a multiple of 8 up to 64); the CUDA-core kernels take every shape.
 * RAD_CONV_KERNEL_AUTO uses the tensor cores wherever the shape allows, RAD_CONV_KERNEL_SIMT never does;
 * RAD_CONV_KERNEL_TENSOR is the same as AUTO (shapes the tensor-core kernels cannot take still run on CUDA
 * cores).  Host only, process-wide.  Returns the previous setting, or RAD_EINVAL.
 */
#define RAD_CONV_KERNEL_AUTO   0
#define RAD_CONV_KERNEL_SIMT   1
#define RAD_CONV_KERNEL_TENSOR 2
int rad_set_conv_kernel(int32_t which);

int rad_cnn_workspace(const rad_cnn_desc* net /* host */, int64_t* bytes /* host */,
                      rad_step_stats* stats /* host or NULL */);
int rad_cnn_step(const rad_cnn_desc* net /* host */, const void* X, const int32_t* labels,
                 const void* const* conv_W, const float* const* conv_b,
                 const void* const* fc_W, const float* const* fc_b,
                 float* const* dconv_W, float* const* dconv_b, float* const* dfc_W, float* const* dfc_b,
                 float* loss, int64_t* nnz_out, void* workspace, int64_t workspace_bytes,
                 int32_t* dev_status, void* stream);

/*
 * Device-side waits (the paper has no counterpart: this is failure handling).  Every kernel that waits for
 * another party (an mbarrier a copy or a tensor-core commit completes, a look-back status word another CTA
 * publishes) gives up after a time limit, raises RAD_DEV_ETIMEOUT in dev_status, lets its CTAs leave in
 * order (copies in flight are waited for, tensor memory is released) and returns: the context stays usable.
 * The limit is an argument of every launch; rad_set_wait_limit_ns changes the value the library passes
 * (default 2 s; 0 only reads it) and returns the previous one.  Host only, process-wide.
 *
 * rad_wait_probe makes one of those waits run out on purpose, without faulting, trapping or hanging
 * anything: a kernel of one CTA (or one cluster of two) that holds no tensor memory and has no copy in
 * flight waits, through the same helper the real kernels use, for something that is never signalled, for
 * `limit_ns` (at most 1 s), then raises RAD_DEV_ETIMEOUT and returns.
 */
#define RAD_WAIT_PAIR_BARRIER 0   /* mbarrier wait of the SM-pair GEMM kernels (cluster of two CTAs)     */
#define RAD_WAIT_PIPE_BARRIER 1   /* mbarrier wait of the persistent store kernel                        */
#define RAD_WAIT_LOOKBACK     2   /* look-back wait of the store kernels on a status word                */
uint64_t rad_set_wait_limit_ns(uint64_t limit_ns);
int rad_wait_probe(int32_t which, uint64_t limit_ns, int32_t* dev_status /* device */, void* stream);

/* Kernels this library has launched since it was loaded (host-side tally; memsets not counted). */
int64_t rad_launch_count(void);

/* Clusters of two CTAs (SM pairs) the tensor-core kernels keep resident on the current device: the width the
 * K splits of a weight gradient are planned for.  74 on a B200 whose 148 SMs all pair up, fewer on a part with an
 * odd SM count in some GPC; 74 where there is no device to ask. */
int32_t rad_sm_pairs(void);

const char* rad_strerror(int code);
const char* rad_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RAD_H_ */
