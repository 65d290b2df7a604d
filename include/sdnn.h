/*
 * sdnn - sparse deep neural network SGD hot path on one NVIDIA B200 (sm_100a).
 *
 * C ABI of the shared library libsdnn.so.  The operations are those of the paper
 * "Partitioning Sparse Deep Neural Networks for Scalable Training and Inference"
 * (ICS '21), Section 3.2 and Algorithm 1, for a network of L square layers of N
 * neurons whose weight matrices W^k are sparse:
 *
 *   forward   x^k = f(W^k x^{k-1} + b^k),  k = 1..L          (feedforward equation)
 *   output    delta^L = grad_{x^L} J (.) f'(z^L)             (final-layer gradient equation)
 *   backward  delta^{k-1} = (W^k)^T delta^k (.) f'(z^{k-1})  (recursive formula)
 *   update    W^k(j,i) <- W^k(j,i) - eta * delta^k(j) x^{k-1}(i)  on stored entries only
 *                                                            (gradient update rule)
 *
 * W^k(j,i) is the weight of the link from neuron i of layer k to neuron j of
 * layer k+1: CSR row j of W^k lists the incoming links of output neuron j.
 * f(z) = min(max(z, 0), clamp); f'(z) = 1 for 0 < z < clamp, else 0 (activation 0), or the sigmoid of the
 * paper's experimental setup (Section 6), f(z) = 1/(1+exp(-z)), f'(z) = f(z)(1 - f(z)) (activation 1).
 * J = 1/(2B) sum_b ||x^L_b - y_b||^2 (mean squared error over a minibatch of B
 * inputs); a minibatch step is exact minibatch SGD: one delta per input, the
 * gradient averaged over the batch (B = 1 is Algorithm 1 verbatim).  The
 * transposed product of layer k uses W^k as it was before its own update, as in
 * Algorithm 1 (line computing delta^{k-1} precedes the update line).  delta^0 is
 * never formed.
 *
 * Conventions
 *  - Every function returns an sdnn_status (0 = success, negative = error) and
 *    never throws or aborts; sdnn_last_error() gives a message for the last failure.
 *  - The caller keeps ownership of every array it passes.  The handle owns all
 *    device memory it allocates and frees it in sdnn_destroy().
 *  - "host" / "device" below says where a pointer must live.  Device pointers must
 *    be on the handle's device.  All arithmetic is fp32 (fp32 accumulation, FMA).
 *  - Calls are issued on cfg->cuda_stream; a call that returns a scalar to the host
 *    (loss_out, nz_total_out) or uses host buffers synchronises that stream before
 *    returning, otherwise it returns after enqueueing.
 *  - A handle is not thread-safe.  There is no CPU fallback: without a CUDA device
 *    creation fails with SDNN_ERR_CUDA.
 */
#ifndef SDNN_H
#define SDNN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sdnn sdnn_t; /* opaque */

typedef enum {
    SDNN_OK = 0,
    SDNN_ERR_INVALID_ARG = -1,   /* NULL where not allowed, size out of range, batch > max_batch, capacity too small */
    SDNN_ERR_BAD_CSR = -2,       /* row_ptr not monotone from 0, column out of [0,N), unsorted/duplicate, non-finite value */
    SDNN_ERR_OOM = -3,           /* device or host allocation failed */
    SDNN_ERR_CUDA = -4,          /* CUDA runtime error (message in sdnn_last_error) */
    SDNN_ERR_STATE = -5,         /* call not valid in the handle's state (e.g. train step on an inference handle) */
    SDNN_ERR_UNIMPLEMENTED = -6
} sdnn_status;

/* cfg->flags */
#define SDNN_FLAG_BWD_ATOMICS 0x01u /* backward product by scatter with vector reductions into L2 (one pass, one   */
                                    /* copy of the weights)                                                        */
#define SDNN_FLAG_BWD_CSC     0x02u /* backward product by gather through a transposed copy of the layer (second   */
                                    /* index and value array, both copies updated; no atomics).  The default.      */
#define SDNN_FLAG_KEEP_DEBUG  0x04u /* train handles: also store delta^k and the gradient G^k of the last step     */
#define SDNN_FLAG_SKIP_DEAD   0x08u /* allow data-dependent skipping; default is dense mode: every layer streams   */
                                    /* its weights and processes every input.  Inference: inputs whose activation  */
                                    /* vector has become all zero are dropped from the tile (whole chunks of 256   */
                                    /* columns at a time); only done while no layer has a positive bias, because   */
                                    /* only then does an all-zero vector stay all zero.  Training: a unit of rows  */
                                    /* whose delta is zero for every input skips its entries (not for B <= 4,      */
                                    /* whose kernels have no such test).  Results are the same as in dense mode.   */
#define SDNN_FLAG_NO_GRAPH    0x10u /* launch the layer chain kernel by kernel instead of through a CUDA graph     */
#define SDNN_FLAG_BWD_ONE_LAUNCH 0x80u /* transposed realisation: column and row units of a layer in one launch.  By      */
                                    /* default the row units (the update of the row-major copy) are launches of their    */
                                    /* own on two more streams, beside the column units of the layers below; that keeps   */
                                    /* every delta^k of a step (N * padded(B) * 4 bytes per layer more) and is faster    */
#define SDNN_FLAG_NO_PDL      0x20u /* do not let a layer's kernel start its prologue under the previous layer's tail */
#define SDNN_FLAG_ONE_TILE    0x40u /* inference: one tile in flight at a time (see sdnn_infer_batch)               */
#define SDNN_FLAG_IDX32       0x400u /* keep 32-bit indices in the library's internal copies of the layers.  By default a     */
                                    /* net of at most 65536 neurons stores them in 16 bits (2 bytes less per stored entry  */
                                    /* and pass over it); results are identical either way                                */
#define SDNN_FLAG_REORDER     0x100u /* set-up (untimed): group the rows of every W^k by the columns they share and    */
                                    /* renumber the neurons of layer k-1 so that each group's columns are one            */
                                    /* contiguous window of at most 1536 neurons (the single-GPU counterpart of the      */
                                    /* paper's row partitioning, Section 5: rows that read the same x entries go         */
                                    /* together).  A layer for which such groups exist is stored group by group, so that */
                                    /* the rows worked on at any moment gather from a small window of the activation     */
                                    /* tile that the caches hold; a layer without that structure (a uniformly random     */
                                    /* pattern) is left as it is.  Everything                                             */
                                    /* the caller sees keeps the caller's numbering: inputs, outputs, id lists,           */
                                    /* sdnn_get_weights / sdnn_set_weights.  The layers are analysed in sdnn_finalize;   */
                                    /* until then the handle keeps a host copy of every loaded layer.  Inference and     */
                                    /* training handles (targets, activations, deltas and gradients keep the caller's   */
                                    /* numbering too).                                                                    */

#define SDNN_FLAG_SMEM_WINDOWS 0x200u /* with SDNN_FLAG_REORDER: run the layers for which groups were found with kernels   */
                                    /* that own a group: the group's window of the activation tile is copied into shared */
                                    /* memory once and gathered from there (forward_window32_kernel for chunks of 32     */
                                    /* inputs, forward_window_kernel for narrower ones) instead of out of L1/L2.         */
                                    /* Measured on B200: 13-20 % faster on a net of 64 blocks per layer (65536 neurons,  */
                                    /* windows of 1024), slower on a net that is one group (1024 neurons), hence opt-in. */
                                    /* Inference handles only (SDNN_ERR_UNIMPLEMENTED with train = 1); not together with */
                                    /* SDNN_FLAG_SKIP_DEAD (these kernels do not keep track of live inputs).             */

#define SDNN_ACT_CLAMPED_RELU 0
#define SDNN_ACT_SIGMOID      1

typedef struct {
    int32_t  activation;   /* SDNN_ACT_CLAMPED_RELU or SDNN_ACT_SIGMOID */
    float    clamp;        /* upper clamp of the clamped ReLU, e.g. 32.0f; must be > 0 (ignored by the sigmoid) */
    int32_t  max_batch;    /* train: largest minibatch B, at most 128 (the whole minibatch is one register tile of the
                              backward kernels; larger values are rejected with SDNN_ERR_INVALID_ARG);
                              inference: batch tile (inputs processed together), at most 2^30 */
    int32_t  train;        /* 0: inference only (no stored activations); 1: sdnn_train_step allowed.  A training
                              handle stores x^0..x^L of one minibatch and, unless SDNN_FLAG_BWD_ATOMICS is set, a second
                              (transposed) copy of the indices and values of every layer but the first */
    int32_t  update_bias;  /* 1: b^k <- b^k - eta * mean_b delta^k_b (bias read as a column of W^k); 0: bias frozen */
    uint32_t flags;        /* SDNN_FLAG_* */
    void*    cuda_stream;  /* cudaStream_t to issue work on; NULL = a stream the handle creates, which orders
                              itself against the legacy default stream like any blocking stream */
    int32_t  device;       /* CUDA device ordinal; -1 = the current device */
} sdnn_config;

/*
 * Problem statement of Section 3.2 / "Require" line of Algorithm 1: a network {W^k}, k = 1..L.
 * Creates a handle from per-layer CSR arrays (all host pointers; copied, caller keeps them).
 *   row_ptr[l] -> int32[n_neurons+1], monotone, row_ptr[l][0] == 0
 *   col_idx[l] -> int32[nnz_l], in [0,n_neurons), strictly ascending within each row
 *   values[l]  -> float[nnz_l], finite (explicit zeros are legal stored entries and stay in the pattern)
 *   bias[l]    -> float[n_neurons], finite
 * Errors: INVALID_ARG (NULL, sizes <= 0, bad cfg), BAD_CSR, OOM, CUDA.  On error *out is NULL.
 */
int sdnn_create(sdnn_t** out, int32_t n_layers, int32_t n_neurons,
                const int32_t* const* row_ptr, const int32_t* const* col_idx,
                const float* const* values, const float* const* bias, const sdnn_config* cfg);

/*
 * Same network, loaded layer by layer so that the host never holds more than one layer:
 * sdnn_create_deferred reserves device memory for nnz_per_layer[l] stored entries per layer
 * (host array of n_layers int64), sdnn_load_layer validates and uploads one layer (0-based,
 * any order, each exactly once), sdnn_finalize makes the handle usable.  sdnn_create is
 * these three in sequence.  Calling infer/train before finalize gives SDNN_ERR_STATE.
 */
int sdnn_create_deferred(sdnn_t** out, int32_t n_layers, int32_t n_neurons,
                         const int64_t* nnz_per_layer, const sdnn_config* cfg);
int sdnn_load_layer(sdnn_t* h, int32_t layer, const int32_t* row_ptr, const int32_t* col_idx,
                    const float* values, const float* bias);
int sdnn_finalize(sdnn_t* h);

/*
 * Inference (feedforward equation applied L times; minibatch form X^k = f(W^k X^{k-1}) of
 * Section 5's Discussion; inputs are independent of one another).
 *   x0            device float[n_inputs][N], row-major (one input vector per row)
 *   y_out         device float[n_inputs][N] = x^L per input, or NULL
 *   nz_count_out  device int32[n_inputs]: number of nonzero entries of x^L per input, or NULL
 *   nz_index_out  device int32[nz_index_capacity]: for input 0, 1, ... in turn, the ascending
 *                 neuron ids i with x^L(i) != 0, concatenated; or NULL
 *   nz_total_out  host int64*: total number of ids (sum of counts), or NULL
 * The batch is processed in tiles of at most cfg.max_batch inputs (narrower ones, a power of two >= 128, when two
 * activation tiles of max_batch inputs would not fit in the L2 cache and the sparsity pattern is not local: the
 * gathers of a layer then come out of L2 instead of HBM).  Tiles are independent; a batch of more than one tile
 * keeps two in flight, each on a stream of its own (the second stream and its two activation tiles are created at
 * the first such call), so that the start and tail of one tile's launches are filled by the other's;
 * SDNN_FLAG_ONE_TILE turns that off.  The call is ordered on the handle's stream either way:
 * work enqueued there before it is seen, and everything the call launched is complete once that stream has caught
 * up.  If nz_index_out is given and the
 * capacity is too small, only the ids at positions below the capacity are written, *nz_total_out
 * (if given) holds the needed capacity and the call returns SDNN_ERR_INVALID_ARG; y_out and
 * nz_count_out are still valid.  n_inputs == 0 is a valid no-op.
 */
int sdnn_infer_batch(sdnn_t* h, const float* x0, int64_t n_inputs, float* y_out,
                     int32_t* nz_count_out, int32_t* nz_index_out, int64_t nz_index_capacity,
                     int64_t* nz_total_out);

/* Inputs per tile that sdnn_infer_batch uses on this handle (see above); 0 before sdnn_finalize. */
int32_t sdnn_infer_tile_width(const sdnn_t* h);

/* Tiles that sdnn_infer_batch keeps in flight on this handle when a batch has more than one (1 or 2; see above);
 * 0 before sdnn_finalize. */
int32_t sdnn_infer_tiles_in_flight(const sdnn_t* h);

/* Same call with every array in HOST memory (pinned or pageable); the library stages the
 * copies itself, tile by tile, and returns when the outputs are in place. */
int sdnn_infer_batch_host(sdnn_t* h, const float* x0, int64_t n_inputs, float* y_out,
                          int32_t* nz_count_out, int32_t* nz_index_out, int64_t nz_index_capacity,
                          int64_t* nz_total_out);

/*
 * One minibatch SGD step (Algorithm 1 body for a batch of B inputs): forward through all
 * layers, output gradient, then for k = L..1 the transposed product, the masked gradient and
 * the in-place weight update, fused into one pass over the stored entries of each layer.
 *   x0, target  device float[B][N], row-major;  1 <= B <= cfg.max_batch
 *   eta         learning rate
 *   loss_out    host float*: J before the update, or NULL (no synchronisation then)
 * Needs cfg.train = 1 (else SDNN_ERR_STATE).  Weights persist across calls.
 */
int sdnn_train_step(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta,
                    float* loss_out);

/* Same step with x0 and target in HOST memory; copies are staged through pinned buffers. */
int sdnn_train_step_host(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta,
                         float* loss_out);

/*
 * The minibatch step in the averaged form that the Discussion of Section 5 describes: the forward pass runs
 * on all B inputs (X^k = f(W^k X^{k-1})), the final-layer gradient is the average over the batch,
 *     delta^L = (1/B) sum_b (x^L_b - y_b) (.) f'(x^L_b),
 * and that ONE vector is backpropagated, SpBP (Algorithm 3) running as for a single input with step eta.  The passage
 * does not say which x^{k-1} and f'(z^{k-1}) the single vector is paired with; this library takes the batch mean
 * xbar^{k-1} = (1/B) sum_b x^{k-1}_b for both (f' evaluated from xbar^{k-1} exactly as a single input's is from
 * x^{k-1}): W^k(i,j) -= eta * delta^k(i) * xbar^{k-1}(j) on the stored entries, delta^{k-1} = (W^k)^T delta^k (.) f'(xbar^{k-1}).
 * An approximation of sdnn_train_step (which averages the per-input gradients instead); identical to it at B = 1.
 * Arguments, return values and state as sdnn_train_step (device pointers; J is the same loss).  Afterwards
 * sdnn_get_delta returns the single backpropagated vector (float[1][N]) and sdnn_get_gradient delta^k (x) xbar^{k-1}.
 */
int sdnn_train_step_averaged(sdnn_t* h, const float* x0, const float* target, int32_t B, float eta,
                             float* loss_out);

/*
 * Current parameters of one layer (0-based), in the caller's original CSR order: the W^k that the update line
 * of Algorithm 1 (W^k <- W^k - eta * grad) has produced so far, and b^k.
 *   values_out  host float[nnz_l], or NULL;   bias_out  host float[N], or NULL
 * Synchronises the stream.  Creating a new handle from these arrays resumes training.
 */
int sdnn_get_weights(sdnn_t* h, int32_t layer, float* values_out, float* bias_out);

/*
 * Overwrites W^k and b^k, the state that the update line of Algorithm 1 carries from one input to the next, for
 * one layer (0-based) from host arrays in the caller's CSR order
 * (restore from a checkpoint without re-creating the handle; the pattern cannot change).
 *   values  host float[nnz_l], or NULL to keep;   bias  host float[N], or NULL to keep
 * Values must be finite (else SDNN_ERR_BAD_CSR).  Synchronises the stream.
 */
int sdnn_set_weights(sdnn_t* h, int32_t layer, const float* values, const float* bias);

/*
 * Inspection of the last train step (tests, diagnostics).  All outputs are host arrays,
 * input-major like x0: out[b*N + i].  layer is the paper's index k.
 *   sdnn_get_activations: x^k of the last step, k = 0..L                         float[B][N]
 *   sdnn_get_delta:       delta^k of the last step, k = 1..L  (needs KEEP_DEBUG) float[B][N]
 *   sdnn_get_gradient:    G^k = (1/B) sum_b delta^k_b (x) x^{k-1}_b on the stored
 *                         entries, CSR order, k = 1..L        (needs KEEP_DEBUG) float[nnz_k]
 * SDNN_ERR_STATE if no step has run or the flag is missing.
 */
int sdnn_get_activations(sdnn_t* h, int32_t layer, float* out);
int sdnn_get_delta(sdnn_t* h, int32_t layer, float* out);
int sdnn_get_gradient(sdnn_t* h, int32_t layer, float* out);

/*
 * Consistency of the two copies of a training layer's weights.  Without SDNN_FLAG_BWD_ATOMICS a training
 * handle keeps, beside the row-major copy of W^k that the forward product reads, a transposed copy (entries
 * by column, own value array) so that the transposed product of the recursive formula is a gather like the
 * forward product and needs no atomic adds.  Both copies receive the update of the gradient update rule with
 * bit-identical arithmetic.  count_out (host) = number of stored entries of `layer` (0-based) whose two values
 * differ in any bit; bit 32 and up count entries of the transposed pattern missing from the row-major one
 * (never set for a handle this library built).  0 for layers without a transposed copy (the first layer,
 * atomics handles, inference handles).  Synchronises the stream.
 */
int sdnn_mirror_mismatches(sdnn_t* h, int32_t layer, int64_t* count_out);

/*
 * Measures what bounds the layer kernels on the current device (diagnostic; the paper has no counterpart): the
 * rate at which an SM array can gather random rows of `row_bytes` bytes (16 .. 1024, a power of two; read with the
 * layer kernels' own 256-bit accesses, through L1 or past it, whichever is faster) out of a table
 * of `table_rows` rows (a power of two; at most 1 GiB in all) that sits in L2 or, if larger, in HBM, with nothing
 * else competing for the load pipe.  A layer with nnz stored entries and a padded batch of ld inputs gathers
 * nnz rows of 4*ld bytes in the forward product and 2*nnz in the backward launch (transposed realisation), so
 * nnz / rate is the floor of those launches whatever the HBM bandwidth.  Allocates and frees its own table and
 * stream, runs about a hundred microseconds of kernels, synchronises.  rows_per_second: host double*.
 */
int sdnn_probe_gather_rate(int32_t row_bytes, int64_t table_rows, double* rows_per_second);

/*
 * How the gather rate depends on the rows in flight (diagnostic; the paper has no counterpart).  The 64-byte random
 * rows of sdnn_probe_gather_rate, but in strict batches: every lane keeps exactly `loads_in_flight` (1, 2, 4, 8 or 16)
 * 256-bit loads in flight and starts its next batch only when the last of them has returned, with `threads_per_sm`
 * (a multiple of 128, at most 2048) resident threads per SM: threads_per_sm / 2 * loads_in_flight rows in flight per
 * SM.  rows_per_second (host double*) over that number is the latency-throughput curve of the path; rows in flight
 * divided by the rate per SM and clock is the round trip.  It tells whether a layer kernel that stays below the rate of
 * sdnn_probe_gather_rate lacks loads in flight or loses its time elsewhere.  SDNN_ERR_INVALID_ARG if the combination
 * does not fit an SM's registers (all CTAs must be resident for the figure to mean what it says).  table_rows as in
 * sdnn_probe_gather_rate.  Allocates and frees its own table and stream; synchronises.
 */
int sdnn_probe_gather_inflight(int64_t table_rows, int32_t threads_per_sm, int32_t loads_in_flight, double* rows_per_second);

/*
 * What a layer boundary costs on the current device (diagnostic; the paper has no counterpart).  Every layer of
 * Algorithm 1 needs all of the layer before it, so a layer ends with a device-wide hand-over.  barrier_us (host double*):
 * microseconds per grid-wide barrier inside ONE cooperative launch of ctas_per_sm (1..4) CTAs of `threads` threads per
 * SM (release-add on a counter, bounded acquire-spin): what a kernel looping over the layers itself would pay.
 * launch_us (host double*): microseconds per launch of a chain of dependent launches of the same shape under
 * programmatic dependent launch, captured into one graph: what the library's layer launches pay.  Each round / launch
 * writes one float per thread.  SDNN_ERR_INVALID_ARG if the grid cannot be resident as a whole; SDNN_ERR_CUDA with a
 * message if a barrier wait ran out (the kernel then leaves instead of spinning on).  Allocates and frees its own
 * buffers, stream and graph; synchronises.
 */
int sdnn_probe_layer_boundary(int32_t ctas_per_sm, int32_t threads, double* barrier_us, double* launch_us);

/*
 * Measures the alternative to keeping two copies of a training layer's values (diagnostic; the paper has no
 * counterpart): with ONE value array in row-major order, the column units of the transposed product would reach each
 * value through a position map, i.e. read (and, to apply the update, write) single 4-byte words at scattered places.
 * store = 0: scattered 4-byte loads; store = 1: scattered 4-byte stores; out of / into a table of `table_words` floats
 * (a power of two, 2^10 .. 2^28).  words_per_second (host double*): accesses per second by the whole device.  To be
 * compared with sdnn_probe_gather_rate: a scattered word costs the load/store pipe as much as a gathered row of up
 * to 64 bytes, so sharing one value array would trade one row gather per stored entry for one (loads) or two (update)
 * scattered words.  Allocates and frees its own table and stream; synchronises.
 */
int sdnn_probe_word_rate(int32_t store, int64_t table_words, double* words_per_second);

/*
 * The same measurement with the rows fetched by the copy engine (TMA) into shared memory instead of by load
 * instructions into registers (diagnostic; the paper has no counterpart).  gather4 = 0: one bulk copy
 * (cp.async.bulk) per row; gather4 = 1: four rows of a two-dimensional tensor map per instruction
 * (cp.async.bulk.tensor ... tile::gather4).  row_bytes 16 .. 256 (a power of two), table as in sdnn_probe_gather_rate.
 * No cluster multicast; the tensor map covers this device's own table only.  Every wait of the kernel is bounded;
 * if one runs out the call returns SDNN_ERR_CUDA with a message instead of a rate.  Allocates and frees its own
 * table; synchronises.
 */
int sdnn_probe_tma_gather_rate(int32_t row_bytes, int64_t table_rows, int32_t gather4, double* rows_per_second);

/*
 * Do the two gather paths add up?  (Diagnostic; the paper has no counterpart.)  One CTA of 1024 threads per SM: four
 * warps fetch random rows with tile::gather4 into shared memory (tma_rounds rounds each), 28 warps gather random rows
 * with 256-bit loads into registers (lsu_per_group rows per lane group, a multiple of 8), out of the same table; either
 * part may be given no work.  row_bytes 64 or 256.  seconds (host double*): device time of one launch; rows (host
 * double*): rows gathered by one launch over both paths.  Comparing a launch of both parts with launches of each part
 * alone says whether the copy engine could carry gathers BESIDE the load instructions.  Waits bounded as in
 * sdnn_probe_tma_gather_rate; allocates and frees its own table; synchronises.
 */
int sdnn_probe_mixed_gather(int32_t row_bytes, int64_t table_rows, int32_t tma_rounds, int32_t lsu_per_group,
                            double* seconds, double* rows);

/*
 * The same measurement for operand tiles staged on chip (diagnostic; the paper has no counterpart): random rows of
 * `row_bytes` bytes (32, 64, 128 or 256; read with 128-bit accesses) out of a table of 128 KiB per CTA held in shared
 * memory.  cluster_size 1: every CTA reads its own shared memory; 2, 4, 8 or 16: the table is spread over the shared
 * memories of a thread-block cluster and read with ld.shared::cluster (distributed shared memory), every CTA of the
 * cluster reading the whole cluster's table.  One CTA of 1024 threads per SM, as many whole clusters as the device holds
 * at once.  rows_per_second (host double*): rows gathered per second by all of them together; ctas_out (host int32*, may
 * be NULL): CTAs (= SMs) that took part.  Compared with sdnn_probe_gather_rate this says whether staging a tile in a
 * cluster's shared memories could beat gathering it out of L2.  Errors: INVALID_ARG (sizes), CUDA (a cluster of that
 * size does not fit the device).  Synchronises.
 */
int sdnn_probe_smem_gather_rate(int32_t row_bytes, int32_t cluster_size, double* rows_per_second, int32_t* ctas_out);

/* Layers for which SDNN_FLAG_REORDER found groups of rows sharing a window of columns (0 without the flag or before
 * sdnn_finalize), and how many of them run with the window staged in shared memory (SDNN_FLAG_SMEM_WINDOWS). */
int32_t sdnn_grouped_layers(const sdnn_t* h);
int32_t sdnn_windowed_layers(const sdnn_t* h);

/*
 * The grouping step of SDNN_FLAG_REORDER on one layer, on the host (no device needed; for tests and studies):
 * greedy column-net clustering of the rows of an n x n CSR pattern (row_ptr host int32[n+1], col_idx host int32[nnz])
 * into groups of at most row_cap rows whose columns span at most col_cap neurons after renumbering.
 *   group_of_row  host int32[n]: group of each row (rows without entries: the last group)
 *   col_label     host int32[n]: new number of each column (a permutation of 0..n-1)
 *   n_groups      host int32*: number of groups, or 0 when the pattern has no such structure (the other outputs are
 *                 then untouched)
 *   max_window    host int32*: widest window (new column numbers spanned by one group)
 * Errors: INVALID_ARG (NULL, n < 1, caps < 1).
 */
int sdnn_cluster_layer(int32_t n, const int32_t* row_ptr, const int32_t* col_idx, int32_t col_cap, int32_t row_cap,
                       int32_t* group_of_row, int32_t* col_label, int32_t* n_groups, int32_t* max_window);

/* Counters since creation: kernels launched by this handle (graph nodes count one each);
 * device bytes it holds. */
int64_t sdnn_kernel_launches(const sdnn_t* h);
int64_t sdnn_device_bytes(const sdnn_t* h);

/* Device time of the two kernel chains of the most recent train step, from events recorded on the
 * handle's stream around them (inside the graph when one is used): fwd_ms covers the L forward
 * launches, bwd_ms the L backward+update launches.  Synchronises the stream.  SDNN_ERR_STATE if no
 * step has run. */
int sdnn_get_phase_times(sdnn_t* h, float* fwd_ms, float* bwd_ms);

/* Per-layer liveness of the most recent inference tile run with SDNN_FLAG_SKIP_DEAD in effect (see the flag):
 * live_inputs_out host int32[L] = inputs of that tile whose activation vector is not all zero after each layer.
 * Synchronises the stream.  SDNN_ERR_STATE if no such tile has run. */
int sdnn_get_liveness(sdnn_t* h, int32_t* live_inputs_out);

/*
 * Inference without any allocation (the paper has no counterpart: this entry point exists for
 * callers that cannot allocate device memory when they call us - for example a host application
 * whose own allocator has already reserved the whole device so that a raw cudaMalloc would fail,
 * a latency-critical loop that cannot afford the device-wide synchronisation an allocation may
 * imply, or a plug-in interface that forbids allocating after initialisation).
 *
 * Same arithmetic as sdnn_infer_batch with y_out only (L forward layers, one tile), but with no
 * handle: the network stays in the caller's device arrays and the two ping-pong activation tiles
 * live in a fixed array inside the library (SDNN_NOALLOC_SCRATCH_BYTES, held by every GPU that
 * loads the library until the process exits).  The call makes no cudaMalloc / cudaFree and uses
 * no allocating library routine; it only launches kernels on `cuda_stream` (NULL = legacy default
 * stream) and returns without synchronising.
 *   row_ptr       device int32[n_layers][n_neurons+1], offsets local to each layer
 *   col_idx       device int32[], values device float[]: the layers' stored entries; layer l
 *                 starts at element layer_offset[l] (host int64[n_layers], each a multiple of 4;
 *                 both base pointers 16-byte aligned).  The arrays are NOT validated: they must
 *                 satisfy the rules of sdnn_create.
 *   bias          device float[n_layers][n_neurons]
 *   x0            device float[n_inputs][n_neurons];  y_out  device float[n_inputs][n_neurons]
 * Limit: n_neurons * padded(n_inputs) <= SDNN_NOALLOC_MAX_TILE_FLOATS, where padded() rounds the
 * batch up to 4, 8, .., 128 and then to multiples of 128; larger problems are rejected with
 * SDNN_ERR_INVALID_ARG and a message (sdnn_last_error(NULL)) before anything is launched.
 * The first call on each device looks up the address of the library's scratch array (once per
 * device, with that device current); make that first call outside any stream capture.
 * All calls share the one scratch array, which keeps whatever the previous call left in it; every
 * call overwrites the part it reads, so nothing needs clearing, but two calls whose kernels may
 * overlap on the GPU (different streams, or different host threads) race on it and must be
 * serialised by the caller.
 */
#define SDNN_NOALLOC_MAX_TILE_FLOATS (1 << 20)
#define SDNN_NOALLOC_SCRATCH_BYTES   (2 * SDNN_NOALLOC_MAX_TILE_FLOATS * 4)
int sdnn_infer_noalloc(int32_t n_layers, int32_t n_neurons, const int32_t* row_ptr, const int32_t* col_idx,
                       const float* values, const int64_t* layer_offset, const float* bias,
                       const float* x0, int32_t n_inputs, float* y_out, float clamp, void* cuda_stream);

/*
 * sdnn_infer_noalloc cannot validate the caller's device arrays on the host.  Its kernel checks the one thing it can
 * without knowing the arrays' lengths: a column index outside [0, n_neurons) is not followed (the entry contributes
 * nothing) and is counted.  count_out (host int64*): such indices met on the current device since the library was
 * loaded; nonzero means the results of some call are not those of the network.  Waits for the device (a copy on
 * the legacy default stream); allocates nothing.
 */
int sdnn_infer_noalloc_bad_columns(int64_t* count_out);

void sdnn_destroy(sdnn_t* h);                 /* NULL is a no-op */
const char* sdnn_last_error(const sdnn_t* h); /* h may be NULL: last creation error of this thread */
const char* sdnn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SDNN_H */
