/*
 * cfi — condensed constant-fan-in sparse linear layer, forward pass, for NVIDIA B200 (sm_100a).
 *
 * The layer is the one of "Dynamic Sparse Training with Structured Sparsity" (SRigL), Sec. 4.4 and
 * appendix "Condensed matrix multiplication": every non-ablated output neuron keeps exactly k incoming
 * weights, stored as two n_active x k arrays (values, column indices), and
 *
 *     y[b, o] = act( bias[o] + sum_{j<k} values[r, j] * x[b, indices[r, j]] )   if o = active_rows[r]
 *     y[b, o] = act( bias[o] )                                                  if o is ablated
 *
 * (Algorithm 1 is the bias = 0, act = identity case; an ablated neuron has all incoming weights pruned,
 * Sec. 3.1 step 4, so only its bias is left.)
 *
 * Conventions
 *   - Plain C ABI.  No call throws; every call returns a cfi_status_t (cfi_status_string() names it).
 *   - "host" / "device" in a parameter comment says where the pointer must live.
 *   - The caller owns every array it passes, before and after the call.  The library owns a layer's
 *     device memory from cfi_create until cfi_destroy.
 *   - All matrices are row-major and dense in memory (no padding between rows).
 *   - A layer is read-only after creation: cfi_forward may run concurrently on several streams.
 *   - The library has no CPU implementation of the forward: without a CUDA device every device call
 *     returns CFI_ERR_CUDA.
 */
#ifndef CFI_H_
#define CFI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cfi_layer cfi_layer_t;  /* opaque */
typedef struct cfi_stack cfi_stack_t;  /* opaque */
typedef struct CUstream_st* cfi_stream_t; /* same type as cudaStream_t; NULL = the default stream */

typedef enum {
    CFI_OK = 0,
    CFI_ERR_NULL = 1,                /* a required pointer was NULL                                  */
    CFI_ERR_SHAPE = 2,               /* a size is negative or inconsistent (k > in, n_active > out..) */
    CFI_ERR_NOT_CONSTANT_FAN_IN = 3, /* cfi_pack: two non-empty rows keep different numbers of weights */
    CFI_ERR_INDEX_RANGE = 4,         /* a column index or row number is out of range or repeated      */
    CFI_ERR_BUFFER_TOO_SMALL = 5,    /* batch larger than what a stack or staging buffer was sized for */
    CFI_ERR_DTYPE = 6,               /* unknown dtype / activation / variant, or layers do not chain   */
    CFI_ERR_ALLOC = 7,               /* host or device allocation failed                               */
    CFI_ERR_CUDA = 8,                /* a CUDA runtime call or kernel launch failed                    */
    CFI_ERR_DEVICE_FLAG = 9,         /* a kernel recorded an error in the layer's device status word   */
    CFI_ERR_ALIGNMENT = 10           /* x or y is not aligned to 16 bytes                              */
} cfi_status_t;

/* Storage type of values, x and y.  Products are exact in fp32 and accumulation is always fp32. */
typedef enum { CFI_F32 = 0, CFI_BF16 = 1 } cfi_dtype_t;

/* CFI_ACT_GELU_ERF is the exact GELU v * Phi(v) = 0.5 v (1 + erf(v / sqrt 2)), applied to every output,
 * ablated ones included.  The paper does not write the activation; its ViT MLP blocks use GELU. */
typedef enum { CFI_ACT_NONE = 0, CFI_ACT_GELU_ERF = 1 } cfi_act_t;

/* Kernel choice for cfi_forward_variant (tests and benchmarks; cfi_forward uses CFI_VARIANT_AUTO). */
typedef enum {
    CFI_VARIANT_AUTO = 0,
    CFI_VARIANT_SIMPLE = 1,   /* one thread per output element, no staging: a cross-check, not fast      */
    CFI_VARIANT_SPLITK = 2,   /* small batch: lanes split a row's k terms, x staged in shared memory     */
    CFI_VARIANT_BATCH = 3,    /* large batch: lanes own batch columns, x tile transposed in shared memory */
    CFI_VARIANT_SLAB = 5,     /* a few tens of batch rows (tiles of 16) on a very sparse layer: the columns of x are
                                 divided over a thread-block cluster that shares a group of output rows           */
    CFI_VARIANT_DENSE_TC = 4  /* batch above a handful of rows: dense copy of the weight on the tensor cores (tcgen05):
                                 bf16 layers directly, fp32 layers as three TF32 products of operands split into two
                                 TF32-exact parts each (K may be split over a thread-block cluster); needs row pitches
                                 of x, y and the weight that are multiples of 16 bytes and no repeated column in a
                                 row, otherwise CFI_ERR_SHAPE */
} cfi_variant_t;

/* Device layouts a layer may hold (cfi_create_layouts).  The condensed form exists to save memory (Sec. 4.4: n x k
 * values and indices instead of the n x d weight), so a caller chooses what to pay for. */
typedef enum {
    CFI_LAYOUT_SMALL_BATCH = 1, /* values + indices, n_active x k padded to 16-byte vectors: CFI_VARIANT_SPLITK / SIMPLE   */
    CFI_LAYOUT_GATHER = 2,      /* the same entries grouped by column slab for CFI_VARIANT_BATCH / SLAB: about as large     */
    CFI_LAYOUT_DENSE = 4,       /* dense out x in copy in the layer's dtype for CFI_VARIANT_DENSE_TC: 1 / density as large  */
    CFI_LAYOUT_ALL = 7
} cfi_layout_t;

const char* cfi_status_string(cfi_status_t s);

/*
 * cfi_pack — dense masked weight -> condensed arrays.  Host only, no CUDA involved.
 * (Appendix "Condensed matrix multiplication": values and column indices as two n x k arrays, Eq. 2:
 *  k distinct columns per row; Sec. 4.4: ablated neurons and zero weights are removed.)
 *
 *   w_dense      host, float  [out_features, in_features]
 *   mask         host, uint8  [out_features, in_features], non-zero = kept; or NULL, in which case an
 *                entry is kept iff w_dense != 0 (so -0.0 counts as pruned).  With a mask, a kept entry
 *                whose value is 0.0 still counts as one of the row's k.
 *   k, n_active  host, written on every successful call
 *   values       host, float  [n_active, k]   } all three NULL: size query only
 *   indices      host, int32  [n_active, k]   } all three non-NULL: filled; the caller sized them from
 *   active_rows  host, int32  [n_active]      } an earlier size query
 *
 * A row that keeps nothing is ablated.  Every other row must keep the same number k >= 1 of entries,
 * otherwise CFI_ERR_NOT_CONSTANT_FAN_IN.  Output order is fixed: columns ascend within a row, rows
 * ascend in active_rows, so the result is unique.  If every row is ablated, k = 0 and n_active = 0.
 */
cfi_status_t cfi_pack(const float* w_dense, const uint8_t* mask, int32_t out_features, int32_t in_features,
                      int32_t* k, int32_t* n_active, float* values, int32_t* indices, int32_t* active_rows);

/*
 * cfi_compact_producer / cfi_compact_consumer — the paper's own output form, host only.
 * (Algorithm 1 returns (batch, active_neurons): Sec. 4.4 removes ablated neurons from the layer altogether, where
 *  cfi_forward writes all out_features columns with act(bias) in the ablated ones.)
 *
 * A layer in compact form is an ordinary layer for cfi_create with out_features = n_active and
 * active_rows = 0 .. n_active-1; its output is the full-width output with the ablated columns deleted.
 * cfi_compact_producer writes that layer's bias and row list:
 *
 *   bias          host, float [out_features] or NULL (= zeros)
 *   active_rows   host, int32 [n_active], each in [0, out_features), no repeats
 *   bias_compact  host, float [n_active], written:  bias_compact[r] = bias[active_rows[r]]
 *   rows_compact  host, int32 [n_active], written:  0, 1, ..., n_active-1
 *
 * cfi_compact_consumer rewrites, in place, the layer that reads such an output (its in_features become the
 * producer's n_active):
 *
 *   prod_active_rows, prod_n_active, prod_out   the producer's row list (as above) and full width
 *   prod_const    host, float [prod_out] or NULL (= zeros): what the producer emits in each of its columns when
 *                 that column is ablated, i.e. act(bias) in the producer's storage precision; only ablated entries
 *                 are read
 *   values        host, float [n_active, k], in/out
 *   indices       host, int32 [n_active, k], in/out: full-width columns in, compact columns out
 *   active_rows   host, int32 [n_active]: the consumer's own row list (selects the bias entry of a row)
 *   bias          host, float [out_features], in/out
 *
 * An entry that reads an active column c of the producer gets the compact column (the rank of c in
 * prod_active_rows).  An entry that reads an ablated column multiplied a constant: values * prod_const[c] is added
 * (in fp32) to the bias of the entry's row, the value becomes 0 and the index the smallest compact column the row
 * does not use yet, so that fan-in stays constant and no column repeats.  The result equals the full-width pair of
 * layers up to the rounding of those bias updates.
 * CFI_ERR_NULL, CFI_ERR_SHAPE (negative sizes, k > prod_n_active), CFI_ERR_INDEX_RANGE (an index or row number out
 * of range, a repeated producer row).
 */
cfi_status_t cfi_compact_producer(const float* bias, const int32_t* active_rows, int32_t n_active, int32_t out_features,
                                  float* bias_compact, int32_t* rows_compact);
cfi_status_t cfi_compact_consumer(const int32_t* prod_active_rows, int32_t prod_n_active, int32_t prod_out,
                                  const float* prod_const, float* values, int32_t* indices, const int32_t* active_rows,
                                  int32_t n_active, int32_t k, float* bias, int32_t out_features);

/*
 * cfi_srigl_update — one SRigL mask update of one layer, on the device (Sec. 3.1, the seven steps "for each
 * layer": magnitudes and gradient magnitudes; K; salient weights per neuron; ablation below gamma_sal * k; the new
 * fan-in k'; global pruning of the K smallest; regrowth per neuron to k').  Outside the forward path: it produces
 * the masks that cfi_pack / cfi_create consume.
 *
 *   w       device, float [out_features, in_features], in/out: zero where masked; survivors keep their value,
 *           grown weights are 0
 *   mask    device, uint8 [out_features, in_features], in/out: 0/1, the same number k of ones in every non-empty row
 *   grad    device, float [out_features, in_features]: dense gradient of the loss with respect to w
 *   K       weights to prune and to grow (clipped to the number of active weights and of inactive positions)
 *   gamma_sal  ablation threshold in [0, 1]: a neuron with fewer than max(1, gamma_sal * k) salient weights is ablated
 *   workspace  device, 256-byte aligned, at least cfi_srigl_workspace_bytes(out_features, in_features) bytes
 *   k_new, n_active_new  host, written: the new fan-in k' = min(in, floor(k * live_before / live_after)) and the
 *           number of neurons that are still active
 *
 * Readings where the paper leaves a choice: ties in magnitude go to the smaller position (row-major); a weight is
 * salient if it is active and not among the K smallest of the layer, or inactive and among the K largest gradients
 * of the layer (live neurons only); neurons without weights stay ablated; regrowth may use any position of the
 * neuron that is not active at that moment, a weight pruned in this very update included, and grown weights start
 * at 0; a neuron left with more than k' weights after the global pruning loses its smallest down to k'.
 * Runs on `stream` and waits for it.  CFI_ERR_NULL, CFI_ERR_SHAPE (sizes < 1, more than 2^31 entries, gamma_sal
 * negative or NaN), CFI_ERR_ALIGNMENT, CFI_ERR_BUFFER_TOO_SMALL (workspace), CFI_ERR_CUDA.
 */
cfi_status_t cfi_srigl_workspace_bytes(int32_t out_features, int32_t in_features, size_t* bytes);
cfi_status_t cfi_srigl_update(float* w, uint8_t* mask, const float* grad, int32_t out_features, int32_t in_features,
                              int64_t K, float gamma_sal, void* workspace, size_t workspace_bytes, int32_t* k_new,
                              int32_t* n_active_new, cfi_stream_t stream);

/*
 * cfi_pack_device — cfi_pack for a weight and mask that live in device memory (e.g. right after cfi_srigl_update):
 * the same condensed arrays, the same order (columns ascending within a row, rows ascending), written to device
 * memory.  The mask is required and defines the structure.
 *
 *   w_dense, mask   device, [out_features, in_features] float / uint8
 *   workspace       device, 256-byte aligned, at least 8 * out_features + 256 bytes
 *   k, n_active     host, written on every successful call
 *   values, indices, active_rows   device, [n_active, k] / [n_active, k] / [n_active]; all three NULL: size query
 *
 * Runs on `stream` and waits for it.  CFI_ERR_NOT_CONSTANT_FAN_IN as for cfi_pack; CFI_ERR_NULL, CFI_ERR_SHAPE,
 * CFI_ERR_ALIGNMENT, CFI_ERR_BUFFER_TOO_SMALL, CFI_ERR_CUDA.
 */
cfi_status_t cfi_pack_device(const float* w_dense, const uint8_t* mask, int32_t out_features, int32_t in_features,
                             void* workspace, size_t workspace_bytes, int32_t* k, int32_t* n_active, float* values,
                             int32_t* indices, int32_t* active_rows, cfi_stream_t stream);

/*
 * cfi_create — build a device-resident layer from condensed arrays (the inputs w and indx of
 * Algorithm 1, plus the bias that Sec. 4.4 extracts with the weights).
 *
 *   values       host, float [n_active, k]; stored on the device as `dtype` (bf16: round to nearest even)
 *   indices      host, int32 [n_active, k], each in [0, in_features); any order; a repeated column in a
 *                row is allowed and simply adds, as Algorithm 1 would
 *   active_rows  host, int32 [n_active], distinct, each in [0, out_features); any order
 *   bias         host, float [out_features] or NULL (zero bias = Algorithm 1 as printed); kept in fp32
 *   dtype, act   see the enums
 *   layer        receives the new layer; destroy it with cfi_destroy
 *
 * Requires 0 <= n_active <= out_features, 0 <= k <= in_features (k >= 1 if n_active > 0),
 * in_features <= 2^20.  The arrays are copied; the caller may free them after the call.
 * The layer lives on the CUDA device that is current when cfi_create is called.  All three device layouts are
 * built (cfi_create_layouts builds fewer).
 */
cfi_status_t cfi_create(const float* values, const int32_t* indices, const int32_t* active_rows, const float* bias,
                        int32_t n_active, int32_t k, int32_t in_features, int32_t out_features,
                        cfi_dtype_t dtype, cfi_act_t act, cfi_layer_t** layer);

/*
 * cfi_create_layouts — cfi_create with the device layouts chosen by the caller (a bit set of cfi_layout_t;
 * cfi_create builds CFI_LAYOUT_ALL).  A layer used for online inference only needs CFI_LAYOUT_SMALL_BATCH and then
 * holds little more than the condensed arrays themselves: 4096 x 4096 at 99 % sparsity is 1.4 MB, against 67 MB with
 * the dense copy.  cfi_forward chooses among the kernels whose layout exists (a small batch runs on the dense or
 * gather layout if that is all there is, and the other way round); cfi_forward_variant with a variant whose layout is
 * missing returns CFI_ERR_SHAPE.  CFI_LAYOUT_DENSE is skipped silently where the tensor-core variant cannot address
 * the shapes (see CFI_VARIANT_DENSE_TC) unless it is the only layout asked for, which is CFI_ERR_SHAPE;
 * cfi_layer_info reports what was built.  CFI_ERR_DTYPE for an empty or unknown bit set.  The paper has no counterpart of the choice: its layer has the one condensed form.
 *
 * cfi_layer_add_layouts builds layouts the layer does not have yet (the layer keeps a host copy of its condensed
 * arrays for this).  No forward call may be running on the layer meanwhile.
 */
cfi_status_t cfi_create_layouts(const float* values, const int32_t* indices, const int32_t* active_rows, const float* bias,
                                int32_t n_active, int32_t k, int32_t in_features, int32_t out_features,
                                cfi_dtype_t dtype, cfi_act_t act, int32_t layouts, cfi_layer_t** layer);
cfi_status_t cfi_layer_add_layouts(cfi_layer_t* layer, int32_t layouts);

/*
 * cfi_forward — y = layer(x) for `batch` rows (Algorithm 1 with bias, ablated rows and activation).
 *
 *   x       device, [batch, in_features]  of the layer's dtype, 16-byte aligned
 *   y       device, [batch, out_features] of the layer's dtype, 16-byte aligned; must not overlap x
 *   stream  the work is enqueued on this stream; the call does not synchronise
 *
 * Every element of y is written (ablated columns too).  batch == 0 succeeds and launches nothing.
 * The return value reports argument and launch errors only.
 *
 * Non-finite inputs.  The condensed kernels (CFI_VARIANT_SIMPLE, SPLITK, BATCH) read only the columns a row
 * indexes, so an inf or NaN in a column that no row (or not this row) uses leaves that row's output alone.
 * CFI_VARIANT_DENSE_TC computes the dense masked product, in which such a column meets weights of 0 and
 * 0 * inf = NaN reaches every output of that batch row (for fp32 layers also through the operand split).  The two
 * agree for finite x, which is the equivalence the paper states (appendix "Condensed matrix multiplication").
 * cfi_forward picks by speed; a caller that needs the condensed behaviour for non-finite activations calls
 * cfi_forward_variant with one of the condensed variants.
 */
cfi_status_t cfi_forward(const cfi_layer_t* layer, const void* x, void* y, int32_t batch, cfi_stream_t stream);

/* As cfi_forward with the kernel chosen by the caller.  A variant that cannot run the given shape
 * (e.g. not enough shared memory) returns CFI_ERR_SHAPE rather than falling back. */
cfi_status_t cfi_forward_variant(const cfi_layer_t* layer, const void* x, void* y, int32_t batch,
                                 cfi_stream_t stream, cfi_variant_t variant);

/*
 * cfi_forward_dense — CFI_VARIANT_DENSE_TC with the launch shape chosen by the caller (tests and sweeps; the paper
 * has no counterpart).  0 leaves a value to the library.
 *
 *   fp32 layers   tile = batch rows per tile: 16, 32, 48, 64, 96 or 128;  cluster = CTAs that share one tile by splitting K
 *                 over a thread-block cluster, 1 .. 8
 *   bf16 layers   tile = outputs per tile: 128 (one tile per CTA; cluster 1 .. 8 as above) or 256 (persistent kernel;
 *                 cluster must be 0 or 1)
 *
 * CFI_ERR_SHAPE for a value outside these sets, for a cluster size the device cannot hold, or if the layer has no
 * dense copy.  Otherwise as cfi_forward.
 */
cfi_status_t cfi_forward_dense(const cfi_layer_t* layer, const void* x, void* y, int32_t batch, cfi_stream_t stream,
                               int32_t tile, int32_t cluster);

/*
 * cfi_forward_host — the same operation for a caller whose activations live in host memory.
 *
 *   x_host  host (pinned memory makes the copies asynchronous), [batch, in_features]  of the layer's dtype
 *   y_host  host, [batch, out_features] of the layer's dtype
 *
 * Copies x to a device staging buffer owned by the layer, runs cfi_forward, copies y back, all on
 * `stream`, then waits for the stream.  The staging buffers grow on demand (a cudaMalloc on the first
 * call and whenever batch exceeds every earlier batch), so this entry point is NOT safe to call
 * concurrently on the same layer.
 */
cfi_status_t cfi_forward_host(cfi_layer_t* layer, const void* x_host, void* y_host, int32_t batch,
                              cfi_stream_t stream);

/* Layer facts for reports: what the forward streams from memory. */
typedef struct {
    int32_t in_features, out_features, n_active, k;
    int32_t dtype, act;
    int32_t k_padded;            /* row length of the small-batch device layout (multiple of 4 or 8)    */
    int32_t batch_slab_columns;  /* columns of x per shared-memory slab in the large-batch kernel        */
    int32_t batch_row_stride;    /* padded row length of the large-batch device layout                   */
    int32_t reserved;
    int64_t weight_bytes_splitk; /* bytes of values+indices the small-batch kernel reads per pass        */
    int64_t weight_bytes_batch;  /* bytes of values+columns the large-batch kernel reads per batch tile  */
    int64_t device_bytes;        /* device memory held by the layer: the three below + bias, row map, status */
    int64_t bytes_small_batch;   /* CFI_LAYOUT_SMALL_BATCH                                               */
    int64_t bytes_gather;        /* CFI_LAYOUT_GATHER                                                    */
    int64_t bytes_dense;         /* CFI_LAYOUT_DENSE                                                     */
    int32_t layouts;             /* bit set of cfi_layout_t: what exists                                 */
    int32_t reserved2;
} cfi_layer_info_t;

cfi_status_t cfi_layer_info(const cfi_layer_t* layer, cfi_layer_info_t* info);

/* Which variant cfi_forward would run for this batch size (written to *variant). */
cfi_status_t cfi_choose_variant(const cfi_layer_t* layer, int32_t batch, int32_t* variant);

/*
 * Launch shape CFI_VARIANT_DENSE_TC would use for this batch size, in the terms of cfi_forward_dense: *tile_n = batch
 * rows per tile (16, 32, 48, 64, 96 or 128) for fp32 layers, outputs per tile (128, or 256 for the persistent kernel) for bf16
 * layers; *cluster = the number of CTAs that share one tile by splitting K over a thread-block cluster (1 .. 8).
 * An introspection call for tests and benchmarks; the paper has no counterpart.
 * CFI_ERR_SHAPE if the layer has no dense copy (see CFI_VARIANT_DENSE_TC), CFI_ERR_NULL on a NULL argument.
 */
cfi_status_t cfi_dense_tile_shape(const cfi_layer_t* layer, int32_t batch, int32_t* tile_n, int32_t* cluster);

/*
 * cfi_device_status — waits for `stream`, then reads the layer's device status word into *flag.
 * 0 means no kernel of this layer has recorded an error since creation; non-zero returns
 * CFI_ERR_DEVICE_FLAG as well.  Kernels never trap: a failed internal check records a code and returns.
 */
cfi_status_t cfi_device_status(const cfi_layer_t* layer, cfi_stream_t stream, int32_t* flag);

/* Frees the layer's device and host memory.  No work using the layer may still be in flight. NULL is OK. */
cfi_status_t cfi_destroy(cfi_layer_t* layer);

/*
 * cfi_stack_* — a chain of layers y = L_{n-1}( ... L_1(L_0(x)) ), e.g. the MLP blocks of a transformer
 * (768 -> 3072 with GELU, 3072 -> 768) whose linears are the layers the paper condenses (Sec. 4.4,
 * appendix "Condensed linear CPU benchmark details").  Layer i+1 consumes layer i's output directly:
 * no residual, normalisation or attention in between.
 *
 *   layers     host array of n_layers layer handles; out_features of layer i must equal in_features of
 *              layer i+1 and all dtypes must match, else CFI_ERR_DTYPE / CFI_ERR_SHAPE.  The stack
 *              borrows the layers: they must outlive it and are not destroyed with it.
 *   max_batch  the two intermediate activation buffers (device, owned by the stack) are sized for it
 *
 * cfi_stack_forward enqueues the n_layers forwards on `stream` without synchronising; batch above
 * max_batch returns CFI_ERR_BUFFER_TOO_SMALL.  One stack must not run on two streams at once (the
 * intermediates are shared).
 */
cfi_status_t cfi_stack_create(cfi_layer_t* const* layers, int32_t n_layers, int32_t max_batch, cfi_stack_t** stack);
cfi_status_t cfi_stack_forward(const cfi_stack_t* stack, const void* x, void* y, int32_t batch, cfi_stream_t stream);
cfi_status_t cfi_stack_destroy(cfi_stack_t* stack);

/*
 * cfi_stack_forward_static — the chain of cfi_stack_forward for callers that must not allocate device
 * memory: code running where cudaMalloc is off limits (a real-time or latency-critical serving loop that
 * may not take the allocator's locks or implicit synchronisation, a process working under a fixed memory
 * budget handed out at start-up, a plug-in whose host forbids allocations after initialisation).  The paper
 * has no counterpart of this entry point; it exists for deployment only.
 *
 * Nothing is created or destroyed: the layers are passed directly, and the intermediate activations live
 * in one fixed 8 MiB device array that is part of the library image (every GPU that loads the library
 * holds these 8 MiB until the process exits).  The array is split into two 4 MiB halves used alternately,
 * so the call requires
 *
 *     batch * max_i(out_features of layer i, i < n_layers - 1) * sizeof(dtype)  <=  4 MiB
 *
 * and returns CFI_ERR_BUFFER_TOO_SMALL otherwise (a single layer needs no intermediate and always fits).
 * Arguments and checks are those of cfi_stack_create + cfi_stack_forward: layers must chain and share
 * dtype and device; x and y are caller-owned device buffers, 16-byte aligned.  The work is enqueued on
 * `stream` without synchronising.  No cudaMalloc / cudaFree and no allocating library call is made.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that first
 * call outside any stream capture.  All calls in the process share the one array: two calls whose kernels
 * can overlap on the GPU (different streams) race on it and must be ordered by the caller.  The array keeps
 * whatever the last call left; nothing needs clearing, because every layer overwrites all batch * out
 * values it hands to the next.
 */
cfi_status_t cfi_stack_forward_static(cfi_layer_t* const* layers, int32_t n_layers, const void* x, void* y,
                                      int32_t batch, cfi_stream_t stream);

/*
 * cfi_probe_device — measures, on the current device, the ceilings the forward kernels are judged against
 * and that no vendor figure states: fp32 FMA rate (register-only chains on every SM), shared-memory load
 * bandwidth (conflict-free 16-byte loads), L2 read bandwidth (every SM streaming a resident 16 MB buffer,
 * and every SM streaming the same 768 KB, which is how the large-batch kernel reads x) and the time of an
 * empty kernel launch in a stream.  Takes a few milliseconds; allocates and frees 16 MB; synchronises
 * the device.  No counterpart in the paper: it reports timings only (Sec. 4.4, Fig. 4).
 */
typedef struct {
    int32_t sm_count;
    int32_t reserved;
    int64_t l2_bytes;
    int64_t smem_per_block_optin;
    double sm_clock_mhz_nominal;
    double fma_tflops;              /* 2 flops per FMA                                   */
    double smem_load_gbs;           /* all SMs together                                  */
    double l2_read_gbs;             /* distinct lines per SM at a time                   */
    double l2_read_same_lines_gbs;  /* all SMs reading the same lines at the same time   */
    double empty_launch_us;
} cfi_device_probe_t;

cfi_status_t cfi_probe_device(cfi_device_probe_t* probe);

/*
 * cfi_probe_floor_launch — enqueues one launch of a kernel that does none of the layer's work, for measuring what a
 * forward call costs at the very least.  It has the forward kernels' launch attributes (one CTA per SM, programmatic
 * dependent launch: it releases its successor at once and waits for its predecessor), so a chain of these launches
 * in a stream or a CUDA graph is timed exactly like a chain of cfi_forward calls.  No counterpart in the paper, which
 * reports wall-clock medians only (Sec. 4.4, Fig. 4).
 *
 *   kind     0: an empty kernel;  1: every CTA makes one dependent trip to DRAM (a 128-byte line of `buf` that no
 *            recent launch has read, chosen from a launch counter kept in `scratch`) and one store
 *   buf      device, 256-byte aligned, buf_bytes >= 1 MiB and best several times the L2 size (kind 1; ignored for 0)
 *   scratch  device, 256-byte aligned, at least 4 KiB, zeroed by the caller before the first launch
 *
 * Asynchronous on `stream`.  CFI_ERR_DTYPE (kind), CFI_ERR_NULL, CFI_ERR_ALIGNMENT, CFI_ERR_BUFFER_TOO_SMALL, CFI_ERR_CUDA.
 */
cfi_status_t cfi_probe_floor_launch(int32_t kind, const void* buf, size_t buf_bytes, void* scratch, cfi_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* CFI_H_ */
