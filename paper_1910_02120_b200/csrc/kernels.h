// Host-side launchers of the IST library's kernels (internal; the public boundary is ist.h).
#pragma once

#include "common.cuh"

namespace ist {

struct Launch {
  cudaStream_t stream;
  int64_t* counter;  // host counter of kernels launched
  void count(int n = 1) const { if (counter) *counter += n; }
};

// ---- partition.cu -----------------------------------------------------------------------
// Balanced random partition of {0..N-1} into S groups from SplitMix64 keys (see ist.h).
// Outputs: idx [N] (group-major, ascending inside a group), off [S+1].  Scratch arrays live in
// caller-provided memory laid out by partition_scratch_carve.
struct PartitionScratch {
  int log_buckets, n_buckets;
  uint64_t* keys;     // [N]
  uint64_t* skey;     // [N] keys grouped by bucket
  int32_t* sidx;      // [N] their neuron indices
  int32_t* hist;      // [n_buckets]
  int32_t* start;     // [n_buckets + 1]
  int32_t* cursor;    // [n_buckets]
  int32_t* grp;       // [N]
  int32_t* lp;        // [N] position among the block's members of the same group
  int32_t* blkcnt;    // [ceil(N/1024)][S]
};
size_t partition_scratch_carve(void* base, int N, int S, PartitionScratch* out);
size_t partition_scratch_bytes(int N, int S);
// Returns false if S is too large for the kernels' shared-memory counters (S > 768).
bool partition_layer(const Launch& L, uint64_t layer_seed, int N, int S, const PartitionScratch& sc,
                     int32_t* idx, int32_t* off, DeviceStatus* st);
// Independent uniform assignment: group_i = floor(key_i * S / 2^64); same outputs.
bool partition_layer_iid(const Launch& L, uint64_t layer_seed, int N, int S, const PartitionScratch& sc, int32_t* idx,
                         int32_t* off, DeviceStatus* st);
void partition_iid_counts_host(uint64_t layer_seed, int N, int S, int64_t* counts);

// ---- gather_scatter.cu ------------------------------------------------------------------
// A slice map describes how packed element (s, i, j) of a layer relates to the full matrix:
// full row = row_idx ? row_idx[row_off[s] + i] : i, full col likewise.
struct SliceMap {
  const int32_t* row_idx;
  const int32_t* row_off;
  const int32_t* col_idx;
  const int32_t* col_off;
  int64_t full_rows, full_cols;  // N_{l-1}, N_l (row stride of the full matrix = full_cols)
  int64_t rows_pad, ld;          // packed slice: [S][rows_pad][ld]
  int s_first;                   // first subnet a launch covers (it covers S consecutive ones)
};
// S = number of subnets moved, starting at m.s_first; master / opw point at subnet 0's slab.
void gather_slices(const Launch& L, const float* W, const SliceMap& m, int S, float* master,
                   bf16* opw, DeviceStatus* st);
void scatter_slices(const Launch& L, float* W, const SliceMap& m, int S, const float* master,
                    DeviceStatus* st);
// b[j] += (sum_s (packed[s][j] - b[j])) / S for the output bias.
void scatter_mean_bias(const Launch& L, float* b, int64_t n, int S, const float* packed,
                       int64_t ld);
// Dense copy-out of a packed slice (ist_get_subnet_params).
void copy_out_slice(const Launch& L, const float* packed, int64_t ld, int64_t rows, int64_t cols,
                    float* out);

// ---- grouped GEMM -----------------------------------------------------------------------
// C[g](m, n) = sum_k A[g](m, k) * B[g](n, k), fp32 accumulation, followed by an epilogue.
enum Epilogue : int {
  EPI_BIAS_RELU = 0,  // out = T(max(C + bias[n], 0))
  EPI_BIAS_F32 = 1,   // outf = C + bias[n]                     (logits)
  EPI_RELU_MASK = 2,  // out = T(mask > 0 ? C : 0)              (delta through ReLU)
  EPI_SGD = 3,        // outf -= lr * C; opw = bf16(outf) if opw (fused weight update)
  EPI_STORE = 4,      // out = T(C)
  // Softmax cross-entropy over a very wide output layer without storing the logits (two passes
  // over the same product):
  EPI_LSE_PART = 5,   // per row and column tile: (max, sum exp(z - max)) of z = C + bias -> lse_part
  EPI_SOFTMAX_DELTA = 6  // out = T((exp(z - lse[m]) - [n == label[m]]) * inv_rows); z[m][label[m]] -> label_logit
};

template <typename T>
struct GemmArgs {
  int M, N, K, G;
  int N_store;  // columns the epilogue may write (>= N, the padded row length); 0 = N
  int k_splits; // > 1: cut the k range into this many slices; slice s of group g writes its fp32
                // partial product to outf slab g * k_splits + s (EPI_BIAS_F32 without bias only)
  const T* A; int64_t a_sm, a_sk, a_sg;
  const T* B; int64_t b_sn, b_sk, b_sg;
  // Per-group extents (tensor-core path; device pointers or null): group g really has
  // off[g + 1] - off[g] rows (m_off), columns (n_off) or contraction entries (k_off); M, N, K are
  // then the capacity every group is laid out for, and the rest of a slab holds zeros.  Tiles
  // that lie wholly beyond a group's rows or columns are skipped and contractions stop at the
  // group's depth (unequal subnets: work follows the true shapes, not the padded ones).
  const int32_t* m_off; const int32_t* n_off; const int32_t* k_off;
  // EPI_SGD on the tensor-core path, launches on single CTAs only (gemm_tc_update_sums_bias): the
  // launch also updates the layer's bias from the B operand (the deltas) it streams anyway:
  // bias_upd[g * bias_upd_sg + n] -= lr * sum_k B[g](n, k), n < bias_n.
  // bias_upd_from_memory: the deltas are read from memory (any launch shape; meant for deltas that are
  // still in L2) instead of from the operand stages.
  float* bias_upd; int64_t bias_upd_sg; int bias_n; int bias_upd_from_memory;
  int epi;
  const float* bias; int64_t bias_sg;
  T* out; int64_t out_ld, out_sg;
  float* outf; int64_t outf_ld, outf_sg;
  const T* mask; int64_t mask_ld, mask_sg;
  bf16* opw;
  float lr;
  // wide softmax head.  lse_part: [G][gemm_tc_lse_parts(N_store)][M] float2 (a few partials per
  // 256-column tile); lse / label_logit: [G][lse_sg]; labels: labels[g * labels_sg + m].
  float* lse_part;
  const float* lse; int64_t lse_sg;
  const int32_t* labels; int64_t labels_sg;
  float* label_logit;
  float inv_rows;
};
template <typename T> void gemm_simt(const Launch& L, const GemmArgs<T>& a);
// Tensor-core path (tcgen05 + TMA) for bf16 operands.  Returns false if the shape cannot be
// described to TMA (misaligned strides) or the operand layouts do not fit an epilogue.
bool gemm_tc(const Launch& L, const GemmArgs<bf16>& a, DeviceStatus* st);
// Several products with the same operand layouts and epilogue (bias + ReLU, ReLU mask, or SGD
// update) as tiles of one launch; at most gemm_tc_max_batch() of them, none k-split.  With a
// chain, problem i + 1 must read problem i's output (A == out, same M and G) and its tiles wait for
// the rows they read.  counters: device, [n - 1][stride] unsigned, stride >= G * ceil(M / 128);
// totals: host, [n - 1], running sums this call advances.  The caller clears counters and totals
// together (once at start, and whenever the batch's shape changes).  A chain must not be used
// from two streams at once.
struct GemmChain {
  unsigned* counters;
  size_t stride;
  unsigned* totals;
};
// loss (weight-update launches only, may be null): the step's mean losses are reduced by the launch.
struct LossReduce;
bool gemm_tc_batch(const Launch& L, const GemmArgs<bf16>* a, int n, const GemmChain* chain, const LossReduce* loss,
                   DeviceStatus* st);
int gemm_tc_max_batch();
bool gemm_tc_update_sums_bias(const GemmArgs<bf16>* a, int n);
// Launches a one-block kernel whose bounded barrier wait must expire after limit_cycles (see
// ist_selftest_wait_expiry).
bool gemm_tc_wait_selftest(const Launch& L, DeviceStatus* st, long long limit_cycles);
int gemm_tc_splits(int K, int want);
int gemm_tc_lse_parts(int64_t n_store);

// ---- rowops.cu --------------------------------------------------------------------------
// Row-wise softmax cross-entropy of logits [G][B][ld] against labels; writes
// delta = (softmax - onehot)/B (zero in columns Nt..ld_d) and row_loss [G][B].
template <typename T>
void softmax_xent(const Launch& L, const float* logits, int64_t ld, int64_t sg, int G, int B, int Nt,
                  const int32_t* y, int64_t y_sg, T* delta, int64_t ld_d, int64_t sg_d,
                  float* row_loss, DeviceStatus* st);
// out[g][b][n] = T(mask[g][b][n] > 0 ? sum_s part[(g * ks + s)][b][n] : 0): closes a k-split
// delta GEMM (fp32 partial slabs of B rows x ld columns each).
template <typename T>
void splitk_mask_reduce(const Launch& L, const float* part, int ks, int G, int B, int64_t ld, const T* mask,
                        int64_t mask_sg, T* out, int64_t out_sg);
// Narrow output layer (Nt <= 64): softmax cross-entropy of logits given as ks partial slabs
// ([G * ks][B][ld] fp32) plus bias; same outputs as softmax_xent.
template <typename T>
void softmax_xent_small(const Launch& L, const float* part, int ks, int64_t ld, int G, int B, int Nt,
                        const float* bias, int64_t bias_sg, const int32_t* y, int64_t y_sg, T* delta, int64_t ld_d,
                        int64_t sg_d, float* row_loss, DeviceStatus* st);
// Wide head, between the two passes: lse[g][b] = log sum_n exp(z[g][b][n]) from the per-tile
// partials ([G][parts][B] float2), labels checked against [0, Nt).  After the second pass:
// row_loss[g][b] = lse[g][b] - label_logit[g][b].
void lse_combine(const Launch& L, const float* lse_part, int parts, int G, int B, int64_t lse_sg, float* lse,
                 const int32_t* y, int64_t y_sg, int Nt, DeviceStatus* st);
void lse_row_loss(const Launch& L, const float* lse, const float* label_logit, int G, int B, int64_t lse_sg,
                  float* row_loss);
// loss_out[g * out_stride + k] = (1/B) sum_b row_loss[g][b]  (fixed summation order); rides on
// the bias update's launch (see bias_sgd) so that it costs no launch of its own.
struct LossReduce {
  const float* row_loss;   // [G][B]
  float* loss_out;         // null: no loss wanted
  int64_t out_stride;
  int k;
};
// bias[g][n] -= lr * sum_b delta[g][b][n] for up to kMaxBiasLayers layers in one launch.
// delta rows are ld elements long (ld a multiple of 8, 16-byte aligned); n <= ld.  If
// loss.loss_out is set, G extra blocks of the same launch reduce the step's row losses.
constexpr int kMaxBiasLayers = 8;
template <typename T> struct BiasSgdLayer {
  const T* delta; int64_t ld, sg;
  float* bias; int64_t bias_sg;
  int n;
};
template <typename T> struct BiasSgdArgs {
  BiasSgdLayer<T> layer[kMaxBiasLayers];
  int xstart[kMaxBiasLayers + 1];   // filled in by bias_sgd: first block of each layer
};
template <typename T>
void bias_sgd(const Launch& L, const BiasSgdArgs<T>& a, int n_layers, int G, int B, float lr, const LossReduce& loss);
// fp32 rows -> T rows with leading dimension ld (pad columns zero), per group row offsets.
template <typename T>
void stage_rows(const Launch& L, const float* X, int64_t N0, int64_t group_row_stride, int G, int B,
                T* out, int64_t ld, int64_t sg);
// eval accumulators: loss_sum += sum of row losses, correct += #argmax hits
void eval_rows(const Launch& L, const float* logits, int64_t ld, int rows, int Nt, const int32_t* y,
               double* loss_sum, long long* correct, DeviceStatus* st);
void eval_finalize(const Launch& L, const double* loss_sum, const long long* correct, int64_t n,
                   float* mean_loss_out, int64_t* correct_out);

// ---- colnorm.cu -------------------------------------------------------------------------
// Batch standardisation of hidden pre-activations (Sec. 2.2).  z [G][B][ld] fp32, statistics
// [G][ld] (stat_sg apart), act / delta [G][B][ld] in operand precision.  n live columns.
template <typename T>
void colnorm_forward(const Launch& L, const float* z, int64_t ld, int64_t z_sg, int G, int B, int n, float eps,
                     float* mu, float* rstd, int64_t stat_sg, T* act, int64_t act_sg);
template <typename T>
void colnorm_backward(const Launch& L, T* delta, int64_t ld, int64_t d_sg, const float* z, int64_t z_sg, const float* mu,
                      const float* rstd, int64_t stat_sg, int G, int B, int n);
void colnorm_apply(const Launch& L, float* z, int64_t ld, int rows, int n, const float* mu, const float* rstd);

// ---- spmm.cu ----------------------------------------------------------------------------
// out[g][b][:] = relu(sum_nz val * P[g][col][:] + bias[g][:]) for rows r0_g + b of a CSR matrix.
template <typename T, typename TO>
void spmm_forward(const Launch& L, const int32_t* row_ptr, const int32_t* col, const float* val,
                  int64_t row0, int64_t group_row_stride, int G, int B, int64_t N0, const T* P,
                  int64_t p_ld, int64_t p_sg, const float* bias, int64_t bias_sg, int n1, TO* out,
                  int64_t out_ld, int64_t out_sg, DeviceStatus* st, bool relu = true);
// master[g][col][:] -= lr * val * delta[g][b][:] over stored nonzeros (atomic adds), then
// refresh the bf16 copy of the touched rows (opw may be null).
template <typename T>
void spmm_backward_sgd(const Launch& L, const int32_t* row_ptr, const int32_t* col, const float* val,
                       int64_t row0, int64_t group_row_stride, int G, int B, int64_t N0,
                       const T* delta, int64_t d_ld, int64_t d_sg, int n1, float* master, bf16* opw,
                       int64_t p_ld, int64_t p_sg, float lr);

}  // namespace ist
