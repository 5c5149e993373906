/*
 * compact.h -- C ABI of the CompAct compressed linear layer for NVIDIA B200 (sm_100a).
 *
 * The layer follows "CompAct: Compressed Activations for Memory-Efficient LLM
 * Training": the forward computes o = x W and keeps only z = x P for the
 * backward (Algorithm 1); the backward computes the compressed weight gradient
 * G_hat = z^T dL/do and the input gradient dL/dx = dL/do W^T (Algorithm 2); the
 * update runs Adam on G_hat with r x m moments and applies
 * W <- W - eta * alpha * P N (Algorithm 3).  P (n x r, entries N(0, 1/r),
 * Section 3.3) is never stored: every kernel regenerates the entries it needs
 * from (seed, layer_id, epoch) with Philox4x32-10 and Box-Muller.
 *
 * Conventions that hold for every entry point
 *   - Matrices are row-major with an explicit leading dimension in ELEMENTS.
 *     W is n x m as in the paper's Section 3.1 (not [out, in]).
 *   - All tensor pointers are DEVICE pointers owned by the caller.  The library
 *     allocates no tensor memory and dereferences no pointer after a call returns
 *     (it remembers encoded TMA descriptors by pointer, shape and pitch: values only).
 *   - Element type of X, W, Y, dY, dX, Z is the layer's dtype; Gc, M, V are
 *     always fp32.
 *   - `stream` is a cudaStream_t passed as void*.  Compute calls are asynchronous
 *     on it and never synchronise the host.
 *   - Base pointers must be 16-byte aligned and every leading dimension times
 *     the element size a multiple of 16 bytes.
 *   - Every function returns a compact_status_t; nothing throws or aborts.
 *     Argument checks happen on the host before any launch.
 *   - A layer handle must not be used from two threads at once.  Calls on one layer
 *     may go to different streams; workspaces and outputs of calls that can overlap
 *     on the GPU must then be distinct.
 *   - Only compute capability 10.x devices are supported; there is no fallback.
 */
#ifndef COMPACT_H_
#define COMPACT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct compact_layer compact_layer_t; /* opaque, host side */

typedef enum {
  COMPACT_OK = 0,
  COMPACT_ERR_INVALID_ARG = 1,
  COMPACT_ERR_SHAPE = 2,
  COMPACT_ERR_ALIGNMENT = 3,
  COMPACT_ERR_DTYPE = 4,
  COMPACT_ERR_EPOCH_MISMATCH = 5,
  COMPACT_ERR_WORKSPACE = 6,
  COMPACT_ERR_UNSUPPORTED_ARCH = 7,
  COMPACT_ERR_CUDA = 8,
  COMPACT_ERR_DEVICE_TIMEOUT = 9,
  COMPACT_ERR_SCRATCH_LIMIT = 10,
  COMPACT_ERR_TOO_MANY_LAYERS = 11
} compact_status_t;

typedef enum { COMPACT_F32 = 0, COMPACT_BF16 = 1 } compact_dtype_t;

/* Inputs of Algorithms 1 and 3: rank r, seed s, Adam decay rates, scale alpha,
 * learning rate eta, projection update gap T (refresh_T == 0: never refresh). */
typedef struct {
  int32_t n, m, r;
  int32_t dtype;      /* compact_dtype_t */
  uint64_t seed;
  uint32_t layer_id;
  uint32_t refresh_T;
  float lr, beta1, beta2, eps, alpha;
  int32_t sparse_s;   /* 0: Gaussian projection (Section 3.3).  s > 0: the sparse Johnson-Lindenstrauss
                       * projection of the ablation study, s terms of +-1/sqrt(s) per row of P, at
                       * Philox-hashed columns; terms that hit the same column add.  At most 64. */
} compact_layer_config_t;

typedef struct {
  uint64_t seed;
  uint32_t layer_id;
  uint32_t epoch;     /* number of refreshes so far: the "s <- s + 1" of Algorithm 3 line 12 */
  uint64_t step;      /* t of Algorithm 3: number of completed updates */
} compact_layer_state_t;

/* Creates a layer (host bookkeeping only; touches no device).  Fails with
 * SHAPE unless 1 <= r <= n, m >= 1, n and m multiples of 8 (bf16) or 4 (f32). */
compact_status_t compact_layer_create(const compact_layer_config_t* cfg, compact_layer_t** out);
compact_status_t compact_layer_destroy(compact_layer_t* layer);

/* Row pitch of Z in elements: r rounded up to a multiple of 16.  Columns
 * r..ldz-1 of Z are written as exact zeros by the forward. */
int64_t compact_z_ld(const compact_layer_t* layer);

/* Bytes of device scratch that compact_linear_bwd / compact_adam_update need
 * for `tokens` rows (split-K partials of Gc; the normalised step N), and never
 * less than compact_fwd_workspace_bytes: one buffer of this size serves all
 * three calls of a layer (not at the same time). */
size_t compact_workspace_bytes(const compact_layer_t* layer, int64_t tokens);

/* Bytes of device scratch with which compact_linear_fwd runs fastest: room for
 * the layer's projection of one epoch in bf16, n rows of ldz rounded up to a
 * multiple of 64 (0 for fp32 layers, which do not use it). */
size_t compact_fwd_workspace_bytes(const compact_layer_t* layer);

/* Bytes kept for the backward by one forward: tokens * ldz * sizeof(element)
 * (Table 1: b l n -> b l r). */
size_t compact_saved_bytes(const compact_layer_t* layer, int64_t tokens);

/* Algorithm 1.  Y[tokens x m] = X W and Z[tokens x ldz] = X P, both rounded once
 * from fp32 accumulators.  Row t of Z belongs to row t of X.  *epoch_used
 * (host pointer, may be NULL) receives the epoch P was generated with.
 * Z may be NULL: then nothing is kept for the backward, which must be
 * compact_linear_bwd_recompute (for layers under activation checkpointing).
 * workspace (device, 16-byte aligned; may be NULL): scratch that the call may
 * overwrite and that holds nothing afterwards.  P is a function of (seed,
 * layer, epoch) and is stored nowhere between calls (Section 3.3); a bf16
 * layer given at least compact_fwd_workspace_bytes(layer) of scratch writes
 * the current P out once at the start of the call and computes Z as further
 * columns of the product that computes Y; without the scratch the kernel
 * regenerates each tile of P where it is consumed, once per block of 512
 * tokens.  Both ways give the same Y and Z bit for bit; the first is faster
 * whenever the batch is longer than a few hundred tokens. */
compact_status_t compact_linear_fwd(compact_layer_t* layer, int64_t tokens,
                                    const void* X, int64_t ldx,
                                    const void* W, int64_t ldw,
                                    void* Y, int64_t ldy,
                                    void* Z, int64_t ldz,
                                    uint32_t* epoch_used,
                                    void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 2.  Gc[r x m] (fp32) = Z^T dY summed over all tokens, and
 * dX[tokens x n] = dY W^T.  dX may be NULL (skip it).  accumulate != 0 adds to
 * Gc instead of overwriting it (micro-batches of one step).  The reduction
 * order over tokens is fixed, so results are bitwise reproducible. */
compact_status_t compact_linear_bwd(compact_layer_t* layer, int64_t tokens,
                                    const void* dY, int64_t lddy,
                                    const void* Z, int64_t ldz,
                                    const void* W, int64_t ldw,
                                    void* dX, int64_t lddx,
                                    float* Gc, int64_t ldg, int accumulate,
                                    void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 2 without a stored z: recomputes Z = X P (the projection of epoch
 * epoch_of_fwd, which must be the layer's current epoch) into the workspace and
 * then does what compact_linear_bwd does.  This is the combination with
 * activation checkpointing that the paper's Limitations section proposes
 * ("recomputing the activation compression during the backward pass"): the
 * checkpointed segment recomputes X anyway, so z need not be kept at all.
 * Results are bitwise those of compact_linear_fwd + compact_linear_bwd.
 * workspace: at least compact_recompute_workspace_bytes(layer, tokens). */
size_t compact_recompute_workspace_bytes(const compact_layer_t* layer, int64_t tokens);
compact_status_t compact_linear_bwd_recompute(compact_layer_t* layer, int64_t tokens,
                                              const void* X, int64_t ldx, uint32_t epoch_of_fwd,
                                              const void* dY, int64_t lddy,
                                              const void* W, int64_t ldw,
                                              void* dX, int64_t lddx,
                                              float* Gc, int64_t ldg, int accumulate,
                                              void* workspace, size_t workspace_bytes, void* stream);

/* Layers that share their input (q, k, v of an attention block; gate and up of an
 * MLP): each has its own W and its own projection -- the paper's appendix on saved
 * tensors lists x P_q, x P_k, x P_v (and x P_gate, x P_up) as separate compressed
 * activations of the one input.  compact_group_fwd is Algorithm 1 for every layer of
 * the group in one launch (X is read once); compact_group_bwd is Algorithm 2 for
 * every layer with the input gradients summed, dX = sum_g dY_g W_g^T, accumulated in
 * one place instead of G tensors added afterwards.  Y and Z are bitwise those of the
 * single-layer calls; Gc may differ in summation order over tokens (still fixed, so
 * reproducible); dX is the sum rounded once.
 * Arrays have `count` entries, one per layer, in the same order.  All layers must
 * have the same n and dtype.  bf16 layers with one seed and count <= 3 run fused;
 * other groups run layer by layer with the same results up to the rounding of dX.
 * workspace of compact_group_bwd: at least compact_group_workspace_bytes(layers,
 * count, tokens).  workspace of compact_group_fwd: optional, as for
 * compact_linear_fwd; compact_group_fwd_workspace_bytes(layers, count) (the sum
 * over the layers, never more than compact_group_workspace_bytes) selects the
 * faster way. */
size_t compact_group_workspace_bytes(compact_layer_t* const* layers, int count, int64_t tokens);
size_t compact_group_fwd_workspace_bytes(compact_layer_t* const* layers, int count);
compact_status_t compact_group_fwd(compact_layer_t* const* layers, int count, int64_t tokens,
                                   const void* X, int64_t ldx,
                                   const void* const* W, const int64_t* ldw,
                                   void* const* Y, const int64_t* ldy,
                                   void* const* Z, const int64_t* ldz,
                                   uint32_t* epochs_used,
                                   void* workspace, size_t workspace_bytes, void* stream);
compact_status_t compact_group_bwd(compact_layer_t* const* layers, int count, int64_t tokens,
                                   const void* const* dY, const int64_t* lddy,
                                   const void* const* Z, const int64_t* ldz,
                                   const void* const* W, const int64_t* ldw,
                                   void* dX, int64_t lddx,
                                   float* const* Gc, const int64_t* ldg, int accumulate,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* Algorithm 3 lines 1-10.  In place on W, M, V (M, V: r x m fp32, pitch ldg);
 * stored moments are the uncorrected running averages and the bias correction
 * uses the 1-based count of this update.  epoch_of_Gc must equal the layer's
 * current epoch (the one the forward reported).  lr = NaN uses the config's.
 * Increments the layer's step.  bf16 layers on the tensor-core path form the
 * increment -eta * alpha * (P N) in fp32, round it to bf16 and add it to W with
 * one more rounding (the add is done by the TMA unit at the L2, so W makes one
 * trip instead of two); fp32 layers and the SIMT path round W once.
 * workspace: at least r * m * 4 bytes (rounded up to 256).  With
 * compact_workspace_bytes(layer, 0) bytes a bf16 layer has room for P written
 * out next to N, and the product P N runs on pairs of SMs like the forward's;
 * with less, the kernel regenerates P tile by tile.  Same W, M, V bit for bit. */
compact_status_t compact_adam_update(compact_layer_t* layer,
                                     void* W, int64_t ldw,
                                     const float* Gc, int64_t ldg,
                                     float* M, float* V,
                                     uint32_t epoch_of_Gc, float lr,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* Allocation-free variant of compact_adam_update (the paper has no counterpart: this is
 * a deployment convenience, not part of the method).
 *
 * Who needs it: a caller that is not allowed to obtain device memory at the moment it
 * wants to step the optimizer -- a serving or training process whose framework has
 * already claimed all of HBM for its own pool, a plugin running inside another runtime's
 * callback where cudaMalloc would serialise the whole device, or code whose memory budget
 * was fixed at start-up.  Such a caller cannot provide the workspace compact_adam_update
 * asks for.  Here the scratch (the normalised step N of Algorithm 3 line 5) lives in an
 * array that is part of the library image: COMPACT_NOALLOC_SCRATCH_BYTES of device memory
 * on every GPU that loads the library, held until the process exits.
 *
 * Same arguments, results and step/epoch bookkeeping as compact_adam_update, without the
 * workspace pair.  The call itself performs no cudaMalloc/cudaFree and calls nothing
 * that allocates.  Layers with r * m * 4 bytes > COMPACT_NOALLOC_SCRATCH_BYTES are
 * rejected with COMPACT_ERR_SCRATCH_LIMIT before anything is launched.
 *
 * The array comes into existence when the CUDA runtime loads this library's device code on
 * a GPU, which (with lazy loading) is the first library call that launches a kernel or asks
 * for a symbol's address there -- possibly this one.  A process that hands all of HBM to its
 * own pool must therefore make one library call on each device (any launch, or a first call
 * of this function) BEFORE it gives the memory away, or that first call fails with
 * COMPACT_ERR_CUDA.  That first call also looks up the array's device address (a runtime
 * query); make it outside any stream capture.  Later calls allocate nothing and query nothing.
 * All calls on a device share the one array, and it keeps whatever the previous call left in
 * it (each call overwrites the r x m entries it reads, so nothing needs clearing).  Two calls
 * whose kernels can overlap on the GPU -- different streams, different layers -- race on it:
 * keep them ordered on one stream or synchronise between them. */
#define COMPACT_NOALLOC_SCRATCH_BYTES (32u << 20)
compact_status_t compact_adam_update_noalloc(compact_layer_t* layer,
                                             void* W, int64_t ldw,
                                             const float* Gc, int64_t ldg,
                                             float* M, float* V,
                                             uint32_t epoch_of_Gc, float lr, void* stream);

/* Algorithm 3 lines 11-13 and Section 3.3: changing the projection only
 * replaces the seed.  If force != 0, or refresh_T > 0 and the step count is a
 * positive multiple of refresh_T not yet refreshed at, epoch <- epoch + 1.
 * Host only: launches nothing and moves no memory.  *new_epoch may be NULL. */
compact_status_t compact_refresh_projection(compact_layer_t* layer, int force, uint32_t* new_epoch);

/* Checkpoint / resume: P is never stored, so (W, M, V) plus this state is a
 * complete checkpoint of a layer. */
compact_status_t compact_layer_get_state(const compact_layer_t* layer, compact_layer_state_t* out);
compact_status_t compact_layer_set_state(compact_layer_t* layer, const compact_layer_state_t* in);

/* Reads and clears the layer's device status word (synchronises the device).
 * Returns DEVICE_TIMEOUT if a kernel gave up on a bounded wait since the last
 * call, OK otherwise. */
compact_status_t compact_layer_status(compact_layer_t* layer);

/* Test hook for the bounded waits (the paper has no counterpart): launches one small
 * CTA that waits, with a limit of a few thousand polls, on a barrier nothing arrives
 * at.  The wait gives up, sets the layer's status word and the kernel returns, exactly
 * as every wait inside the GEMM kernels would; compact_layer_status then reports
 * COMPACT_ERR_DEVICE_TIMEOUT once, and the context stays usable. */
compact_status_t compact_debug_wait_that_runs_out(compact_layer_t* layer, void* stream);

/* Test hooks that make the in-kernel generator observable.
 * compact_debug_philox_u32: out_dev[n x 4*ceil(r/8)] receives the raw Philox
 * words behind P (one call of four words per eight columns) (Algorithm 1 lines 1-2), from the generic ten-round function.
 * compact_debug_philox_layer_u32: the same words from the form the GEMM kernels'
 * generators call (first round partly precomputed on the host per layer).
 * compact_debug_projection: P_dev[n x r] (layer dtype, pitch r) receives P at
 * `epoch`, produced by the same device function the GEMM kernels call. */
compact_status_t compact_debug_philox_u32(uint64_t seed, uint32_t layer_id, uint32_t epoch,
                                          int32_t n, int32_t r, uint32_t* out_dev, void* stream);
compact_status_t compact_debug_philox_layer_u32(uint64_t seed, uint32_t layer_id, uint32_t epoch,
                                                int32_t n, int32_t r, uint32_t* out_dev, void* stream);
/* compact_debug_sparse_terms: for a layer with sparse_s > 0, out_dev[n x sparse_s] receives
 * the hashed terms of every row of P at `epoch`: column in the low 31 bits, sign in bit 31. */
compact_status_t compact_debug_sparse_terms(const compact_layer_t* layer, uint32_t epoch,
                                            uint32_t* out_dev, void* stream);
compact_status_t compact_debug_projection(const compact_layer_t* layer, uint32_t epoch,
                                          void* P_dev, void* stream);

/* Selects the kernel family: 0 = automatic (tensor-core kernels for bf16 where
 * the shape allows -- every product on pairs of SMs, with P written out into the
 * workspace where the call has one; without, a cluster of two CTAs shares every
 * tile of P it generates --, SIMT otherwise), 1 = force the SIMT kernels,
 * 2 = tensor-core kernels that work one SM at a time: every CTA computes its
 * own tiles and generates its own tiles of P (1 and 2 are used by the tests as
 * on-device cross-checks).  Returns the previous value. */
int compact_set_kernel_family(int family);

/* Number of kernels this library has launched since it was loaded. */
uint64_t compact_kernel_launch_count(void);

const char* compact_status_string(compact_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* COMPACT_H_ */
