/*
 * libist — one round of Independent Subnet Training (IST, arXiv 1910.02120) on one GPU.
 *
 * A round (Sec. 2.1 "Methodology" of the paper): the hidden neurons of a fully connected
 * network are randomly partitioned into S disjoint groups ("Constructing Subnets"), every
 * subnet takes the weight slices its neurons select, trains for K iterations of local SGD
 * without talking to the others ("Training Subnets"; K is the paper's J), and the slices are
 * copied back into the full network.  The paper places the S subnets on S machines; here they
 * are S groups of one grouped computation on a single device.
 *
 * Conventions
 *   - C ABI, no exceptions.  Every call returns ist_status (0 = IST_OK, < 0 = error) unless
 *     stated otherwise; ist_last_error() gives a human-readable message for the last failure.
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *   - The library allocates no device memory.  The caller owns the full network, the inputs,
 *     the outputs and one workspace blob (size from ist_workspace_bytes) that must stay alive
 *     and untouched from ist_create to ist_destroy.
 *   - All device work is enqueued on the stream given to ist_create, in call order, and is
 *     asynchronous to the host.  Only ist_sync_status() synchronises.
 *   - Network layout: layer_dims = {N_0, ..., N_t}; layer l (1..t) has W_l row-major
 *     [N_{l-1}][N_l] fp32 (y = x * W_l + b_l) and b_l [N_l] fp32.  Hidden layers use ReLU;
 *     the loss is the softmax cross-entropy averaged over the minibatch.  (The paper fixes
 *     neither the loss nor biases; these are this library's reading.)
 *   - Call order: ist_create -> ist_bind_weights -> { ist_partition -> ist_local_steps* ->
 *     ist_reassemble }* ; ist_eval any time the network is bound and not partitioned.
 *     Between ist_partition and ist_reassemble the caller must not write the bound weights.
 *   - One process drives one device (kernel attributes and launch limits are looked up once
 *     per process, on the device current at the first call); several contexts on that device
 *     are fine, and calls on one context must not overlap in time.  Calls may come from any
 *     host thread, including one that has made no CUDA call before.
 */
#ifndef IST_H_
#define IST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ist_ctx ist_ctx; /* opaque, host object */
typedef int32_t ist_status;

enum {
  IST_OK = 0,
  IST_ERR_ARG = -1,            /* null pointer, size out of range, misaligned pointer */
  IST_ERR_STATE = -2,          /* call out of order */
  IST_ERR_WORKSPACE = -3,      /* workspace too small or misaligned */
  IST_ERR_CUDA = -4,           /* a CUDA runtime call failed */
  IST_ERR_DEVICE_CHECK = -5,   /* a device-side bounds check tripped (label / column / index) */
  IST_ERR_DEVICE_TIMEOUT = -6, /* a bounded device-side wait gave up */
  IST_ERR_UNSUPPORTED = -7     /* valid request this build cannot serve */
};

/* Operand precision of the local steps.  Master weights are fp32 in both modes. */
enum { IST_FP32 = 0, IST_BF16 = 1 };

/* Input kinds. */
enum { IST_X_DENSE_F32 = 0, IST_X_DENSE_BF16 = 1, IST_X_CSR = 2 };

/*
 * Minibatches for ist_local_steps / ist_eval.  X is logically [S][K][batch][N_0]: subnet s at
 * local step k reads rows  r0 = s*stride_subnet + k*stride_step ... r0 + batch - 1  (strides in
 * rows; 0 means "the same rows again").  The paper gives every site its own data and draws a
 * minibatch per iteration (Sec. 2.1); the two strides express that.
 *   dense : `dense` points at row-major rows of N_0 elements (fp32 or bf16), device memory.
 *           bf16 rows need N_0 % 8 == 0 and a 16-byte aligned base.
 *   CSR   : row_ptr [rows+1] (absolute offsets into col/val), col [nnz] (0 <= col < N_0,
 *           distinct inside a row), val [nnz] fp32; all device memory.
 * ist_eval ignores the strides and reads rows 0..n-1.
 */
typedef struct ist_input {
  int32_t kind;
  int32_t batch;
  const void* dense;
  const int32_t* row_ptr;
  const int32_t* col;
  const float* val;
  int64_t stride_subnet;
  int64_t stride_step;
} ist_input;

/*
 * Bytes of device workspace a context of this shape needs (0 on invalid arguments).
 * layer_dims: host, n_dims = t+1 entries, each >= 1.  S >= 1 subnets (S = 1 if t = 1),
 * S <= every hidden N_l.  1 <= max_batch <= 65535: largest `batch` later passed in ist_input
 * (ist_eval processes its rows in chunks of max_batch).
 */
size_t ist_workspace_bytes(const int64_t* layer_dims, int n_dims, int S, int precision,
                           int max_batch, int input_is_csr);

/*
 * Sec. 2.1 "Constructing Subnets" says only that each hidden neuron is assigned uniformly at
 * random to one of the n sites; it does not say whether group sizes are fixed.  Two readings:
 * IST_PART_BALANCED (what ist_workspace_bytes / ist_create use): the rule stated at ist_partition,
 * equal group sizes.  IST_PART_IID: every neuron picks its subnet independently (App. A:
 * probability 1/n each): group of neuron i = floor(key_i * S / 2^64) with the same keys, indices
 * ascending inside a group; group sizes are Binomial(N_l, 1/S) and a group may be empty.  The
 * packed layout then has room for ceil(N_l/S) + ceil(7 * sqrt(N_l (1/S)(1 - 1/S))) + 8 neurons
 * per subnet and hidden layer (at most N_l); ist_partition returns IST_ERR_UNSUPPORTED, without
 * enqueueing anything, for a seed whose draw does not fit (probability below 1e-11 per group), and
 * computes the group sizes on the host (N_l hash evaluations per hidden layer and call).
 */
#define IST_PART_BALANCED 0
#define IST_PART_IID 1
size_t ist_workspace_bytes2(const int64_t* layer_dims, int n_dims, int S, int precision,
                            int max_batch, int input_is_csr, int partition_rule);
ist_status ist_create2(ist_ctx** out, const int64_t* layer_dims, int n_dims, int S, int precision,
                       int max_batch, int input_is_csr, int partition_rule, void* workspace_dev,
                       size_t workspace_bytes, void* cuda_stream);

/*
 * Creates a context for a network of the paper's form (Sec. 2: an input layer, t - 1 hidden
 * layers and an output layer with weight matrices between consecutive layers, trained at n = S
 * sites).  Contexts and workspaces themselves have no counterpart in the paper.
 * workspace_dev: device, 256-byte aligned, >= ist_workspace_bytes(...).
 * cuda_stream: a cudaStream_t (NULL = legacy default stream), borrowed.  The workspace is
 * cleared on this stream.  *out is set only on success; free it with ist_destroy.
 */
ist_status ist_create(ist_ctx** out, const int64_t* layer_dims, int n_dims, int S, int precision,
                      int max_batch, int input_is_csr, void* workspace_dev, size_t workspace_bytes,
                      void* cuda_stream);

/*
 * The full network the rounds act on (Sec. 2.1: the model the subnets are cut from and copied
 * back into).  W_dev / b_dev: host arrays of t device pointers
 * (W_l [N_{l-1}][N_l] fp32, b_l [N_l] fp32), borrowed until ist_destroy or the next bind.
 */
ist_status ist_bind_weights(ist_ctx* ctx, float* const* W_dev, float* const* b_dev);

/*
 * Sec. 2.1 "Constructing Subnets" + distribution of the slices.  Draws a fresh partition of
 * every hidden layer from `seed` and gathers each subnet's slices into the workspace:
 * subnet s owns W_1[:, G_1^s], W_l[G_{l-1}^s, G_l^s] for 1 < l < t, W_t[G_{t-1}^s, :], the
 * hidden biases of its neurons and its own copy of the output bias (App. A: each neuron in
 * exactly one subnet; its footnote: a subnet's weight slices leave out everything that belongs
 * to neurons the subnet does not own).
 * Partition rule (the paper states only that the assignment is uniform): neuron i of hidden layer l
 * gets the i-th output of a SplitMix64 generator seeded with the l-th output of a SplitMix64
 * generator seeded with `seed`; neurons are ranked by (key, index); group g takes the next
 * floor(N_l/S) (+1 if g < N_l mod S) ranks; indices are ascending inside a group.
 */
ist_status ist_partition(ist_ctx* ctx, uint64_t seed);

/*
 * Copies the current partition of hidden layer `hidden_layer` (1..t-1) out, i.e. the membership
 * indicators of App. A as index lists (group s = the neurons j with m^(s)_{l,j} = 1):
 * idx_out_dev [N_l] int32 (group-major, ascending inside a group), off_out_dev [S+1] int32.
 */
ist_status ist_get_partition(ist_ctx* ctx, int hidden_layer, int32_t* idx_out_dev,
                             int32_t* off_out_dev);

/*
 * Copies subnet s's current fp32 master slice of layer l (1..t) out, densely:
 * W_out_dev [rows][cols] with rows = |G_{l-1}^s| (N_0 for l = 1), cols = |G_l^s| (N_t for
 * l = t); b_out_dev [cols].  Either pointer may be NULL.  Needs a partition in place.
 */
ist_status ist_get_subnet_params(ist_ctx* ctx, int layer, int s, float* W_out_dev,
                                 float* b_out_dev);

/*
 * Shape of subnet s's slice of layer l (1..t) under the partition in place (Sec. 2.1; Sec. 2.3
 * counts these sizes): *rows_out_host = |G_{l-1}^s| (N_0 for l = 1), *cols_out_host = |G_l^s|
 * (N_t for l = t).  Host outputs, either may be NULL.  These are the extents
 * ist_get_subnet_params writes.  Needs a partition in place (IST_ERR_STATE otherwise).
 */
ist_status ist_subnet_slice_shape(ist_ctx* ctx, int layer, int s, int64_t* rows_out_host,
                                  int64_t* cols_out_host);

/*
 * Sec. 2.1 "Training Subnets": K iterations of local SGD on every subnet, no exchange.
 * Step k of subnet s: forward (App. A Eq. (2) on the slice, without the n^2 factor, as
 * Sec. 2.2 removes it), mean softmax cross-entropy against y, backward, w <- w - lr * grad
 * with all gradients taken at the pre-update weights.
 * y_dev: int32 labels addressed like X rows (row r -> y_dev[r]), 0 <= y < N_t.
 * loss_out_dev: [S*K] fp32, loss_out[s*K + k] = loss of subnet s before the update of step k
 * (may be NULL).  1 <= K.  X->batch <= max_batch.
 */
ist_status ist_local_steps(ist_ctx* ctx, const ist_input* X, const int32_t* y_dev, float lr, int K,
                           float* loss_out_dev);

/*
 * Sec. 2.2, "IST for other architectures": when only the fully connected part of a network is
 * partitioned, the part in front of it (a convolutional trunk, which every site holds whole and
 * trains by local SGD) needs the gradient of each subnet's loss with respect to that subnet's
 * inputs.  Same as ist_local_steps, and in addition
 * dx_out_dev (device, fp32, not NULL): rows addressed exactly like the rows of X (row r of X ->
 * row r of dx_out_dev, N_0 floats each, so the buffer spans as many rows as X does); the row of
 * subnet s, step k, sample b receives d(loss[s][k]) / d(that input row) = delta_1 W_1^T on the
 * subnet's slice, taken at the weights step k starts from.  Rows of X that no step reads are not
 * written.  Dense inputs only (IST_ERR_UNSUPPORTED for CSR); on the bf16 path N_0 must be a
 * multiple of 4.  With K > 1 the later steps' gradients belong to inputs the trunk produced
 * before its own update: the usual call has K = 1.
 */
ist_status ist_local_steps_dx(ist_ctx* ctx, const ist_input* X, const int32_t* y_dev, float lr, int K,
                              float* loss_out_dev, float* dx_out_dev);

/*
 * Training the S subnets at several sites (Sec. 2.1 "Distributing Subnets": every subnet goes to
 * its own compute node; Sec. 2.3: only the slices travel).  A context may own only subnets
 * first .. first + count - 1: ist_partition then draws the whole partition (it is cheap and every
 * site needs the same one) but gathers only the owned subnets' slices, and ist_local_steps trains
 * only those; the other subnets are trained by other contexts (other GPUs, one process each) that
 * hold a copy of the same full network and draw the same partition (same seed).  Before
 * ist_reassemble every context must hold all S trained slices: ist_packed_layer gives the device
 * address of layer l's packed fp32 slices ([S][*master_bytes_per_subnet], subnet s at byte
 * offset s * bytes) and of its packed biases, so that the caller can exchange them (one
 * all-gather per layer over the subnet dimension, each site contributing its own `count` slabs).
 * ist_reassemble writes all S slabs back, whoever trained them.
 * In ist_local_steps the inputs and losses are then addressed by the local subnet index
 * (0 .. count-1): rows start at i * stride_subnet, loss_out_dev holds count * K values.
 * Default range: all S subnets.  Not allowed while a partition is in place.
 */
ist_status ist_set_subnet_range(ist_ctx* ctx, int first, int count);
ist_status ist_packed_layer(ist_ctx* ctx, int layer, void** master_dev, size_t* master_bytes_per_subnet,
                            void** bias_dev, size_t* bias_bytes_per_subnet);

/*
 * Sec. 2.1 "Training Subnets", last step: the trained slices go back into the full network; the
 * groups are disjoint, so no two subnets write the same entry.
 * Writes every trained slice to the positions it was gathered from; entries of middle layers
 * whose row group differs from their column group are not written.  The output bias, the one
 * parameter all subnets hold, becomes b + (sum_s (b^(s) - b)) / S (its mean over the copies).
 * Afterwards the context is back in the "bound" state.
 */
ist_status ist_reassemble(ist_ctx* ctx);

/*
 * Full-width forward pass of the bound network (the deployed model, Sec. 2.2) over n rows:
 * mean softmax cross-entropy -> *mean_loss_out_dev (fp32), number of rows whose arg-max
 * (lowest index on ties) equals the label -> *n_correct_out_dev (int64).  Computed in fp32.
 */
ist_status ist_eval(ist_ctx* ctx, const ist_input* X, const int32_t* y_dev, int64_t n,
                    float* mean_loss_out_dev, int64_t* n_correct_out_dev);

/*
 * Sec. 2.2 "Correcting Distributional Shift", second remedy: every hidden neuron's input is
 * standardised over the minibatch before the non-linearity,
 *   zh = (z - mean_b z) / sqrt(var_b z + eps),  a = max(zh, 0),
 * per subnet and neuron, with the biased (1/batch) variance and no learned scale or shift (the
 * paper fixes neither eps nor the variance estimator), and the backward pass differentiates
 * through it:  d_z = (d_zh - mean_b d_zh - zh * mean_b(d_zh * zh)) / sigma.
 *
 * ist_norm_workspace_bytes: bytes of a second device blob that holds the fp32 pre-activations
 * of the hidden layers ([S][max_batch][n_l] per layer) and the statistics.
 * ist_enable_normalization: switches the context to this mode for all later calls (there is no
 * way back).  norm_workspace_dev: device, 256-byte aligned, at least that many bytes, borrowed
 * until ist_destroy; it is cleared on the context's stream.  eps > 0.  Not allowed while a
 * partition is in place.
 * ist_calibrate: the deployment statistics of Sec. 2.2: mean and standard deviation of every
 * hidden neuron's input over rows 0..n-1 of X (1 <= n <= max_batch, fp32 or CSR rows), computed
 * with the bound full network layer by layer in fp32.  ist_eval then standardises with these
 * stored values.  ist_reassemble and ist_bind_weights discard the statistics (they belong to the
 * weights they were taken with); in this mode ist_eval without valid statistics returns
 * IST_ERR_STATE.
 */
size_t ist_norm_workspace_bytes(const ist_ctx* ctx);
ist_status ist_enable_normalization(ist_ctx* ctx, float eps, void* norm_workspace_dev,
                                    size_t norm_workspace_bytes);
ist_status ist_calibrate(ist_ctx* ctx, const ist_input* X, int64_t n);

/* Waits for the stream and returns the sticky device status (IST_OK, IST_ERR_DEVICE_CHECK,
 * IST_ERR_DEVICE_TIMEOUT or IST_ERR_CUDA). */
ist_status ist_sync_status(ist_ctx* ctx);

/*
 * Self-test of the device-side error path (no counterpart in the paper).  Every wait inside the
 * tensor-core kernels is bounded: after its limit it records IST_ERR_DEVICE_TIMEOUT in the status
 * word and the kernel returns.  This call enqueues, on the context's stream, a one-block kernel that
 * waits with the same routine on a barrier nothing ever signals, for limit_cycles SM clock cycles
 * (1 .. 2e9, i.e. at most about a second), so that the wait must give up.  Afterwards
 * ist_sync_status returns IST_ERR_DEVICE_TIMEOUT for this context (the status word is sticky: create
 * a new context to go on); the stream and the device stay usable.  Returns IST_ERR_ARG for a limit
 * outside the range, IST_ERR_CUDA if the launch fails.
 */
ist_status ist_selftest_wait_expiry(ist_ctx* ctx, int64_t limit_cycles);

/*
 * Measurement aid (no counterpart in the paper).  Kernel classes of a round, in the order a
 * round runs them.  With profiling enabled every group of launches of one class is bracketed
 * by a pair of CUDA events on the context's stream; ist_profile_read synchronises and returns
 * the number of kernels launched and the summed device time of that class since profiling was
 * enabled.  Enabling clears earlier records.  The events cost a few microseconds each, so
 * throughput should be timed with profiling off.
 */
enum {
  IST_K_PARTITION = 0, /* keys, ranks, index lists */
  IST_K_GATHER = 1,    /* full network -> packed slices (+ bf16 copies) */
  IST_K_STAGE = 2,     /* fp32 input rows -> bf16 staging */
  IST_K_FWD = 3,       /* forward GEMMs with bias / ReLU / logits epilogues */
  IST_K_LOSS = 4,      /* softmax cross-entropy, loss reduction */
  IST_K_DX = 5,        /* delta_{l-1} GEMMs with the ReLU mask epilogue */
  IST_K_DW_SGD = 6,    /* weight-gradient GEMMs with the fused SGD update */
  IST_K_BIAS_SGD = 7,  /* bias gradient and update */
  IST_K_SPMM = 8,      /* sparse first layer: forward, backward + update */
  IST_K_SCATTER = 9,   /* packed slices -> full network */
  IST_K_EVAL = 10,     /* full-width evaluation */
  IST_K_NORM = 11,     /* batch standardisation, forward and backward (Sec. 2.2) */
  IST_K_COUNT = 12
};
ist_status ist_profile(ist_ctx* ctx, int enable);
ist_status ist_profile_read(ist_ctx* ctx, int kernel_class, int64_t* launches_out_host,
                            double* ms_out_host);

/*
 * Partition of one hidden layer without a context, a workspace or any allocation.  (The paper
 * has no counterpart; this is a service entry point of the library.)
 *
 * For callers that cannot obtain device memory at the time they need a partition: code running
 * inside a host application that gave out its device-memory budget at start-up and forbids
 * allocation afterwards, or a process that only wants the index lists (for example to decide
 * which weight slices to fetch) and has no room for an ist_ctx workspace.  The caller passes
 * only its own outputs; the kernels' intermediate arrays live in a device array that is part of
 * the library image, 2 MB that every GPU loading the library holds until exit.
 *
 * Result: exactly the partition ist_partition(seed) draws for hidden layer `hidden_layer`
 * (1-based) when that layer has n_neurons neurons and the network is split into S subnets:
 * idx_out_dev [n_neurons] int32 (group-major, ascending inside a group), off_out_dev [S+1].
 * Work is enqueued on cuda_stream (a cudaStream_t, NULL = default stream), asynchronously.
 *
 * Limits: n_neurons <= IST_STATIC_MAX_NEURONS and S <= IST_STATIC_MAX_SUBNETS, otherwise
 * IST_ERR_UNSUPPORTED and nothing is enqueued.  IST_ERR_ARG for null outputs, S < 1,
 * S > n_neurons or hidden_layer outside 1..62.  The call performs no cudaMalloc / cudaFree and
 * calls no allocating routine.
 *
 * The first call on a device looks up the device address of the built-in array (a host-side
 * set-up step): make that first call before starting any stream capture.
 * All calls on a device share the one array, which keeps the previous call's contents; the
 * entry point clears what has to start at zero.  Two calls whose kernels can overlap on the
 * GPU (different streams without an ordering between them) race on it: order them.
 */
#define IST_STATIC_MAX_NEURONS 65536
#define IST_STATIC_MAX_SUBNETS 64
ist_status ist_partition_layer_static(uint64_t seed, int hidden_layer, int64_t n_neurons, int S,
                                      int32_t* idx_out_dev, int32_t* off_out_dev, void* cuda_stream);

/*
 * Device-side status of ist_partition_layer_static on the current device (no counterpart in the
 * paper).  Its kernels check every index they emit against [0, n_neurons) and record a failure
 * in a status word at the start of the built-in array; each call of the entry point clears the
 * word first, so this reports on the most recent call.  Waits for cuda_stream (the stream that
 * call used), copies the word to the host and returns IST_OK or IST_ERR_DEVICE_CHECK
 * (IST_ERR_CUDA if the copy fails).  Allocates nothing.  Before the first
 * ist_partition_layer_static call on the device it returns IST_OK.
 */
ist_status ist_static_partition_status(void* cuda_stream);

/* Number of kernels this context has launched so far (host counter). */
int64_t ist_kernel_launches(const ist_ctx* ctx);

/* Message for the most recent failing call on this context ("" if none).  ctx may be NULL,
 * in which case the message of the last failing ist_create on this thread is returned. */
const char* ist_last_error(const ist_ctx* ctx);

/* Frees the host object.  Does not touch device memory; pending work keeps running. */
void ist_destroy(ist_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* IST_H_ */
