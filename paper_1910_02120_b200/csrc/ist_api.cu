// C-ABI boundary of the IST library (see include/ist.h): argument checks, workspace carving,
// the call-order state machine, and the sequence of kernels each call enqueues.  Every step
// of a round runs in this library's kernels; the host only validates and enqueues.
#include "../../include/ist.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <string>
#include <vector>

#include "kernels.h"

using namespace ist;

namespace {

enum State { ST_CREATED = 0, ST_BOUND = 1, ST_PARTITIONED = 2 };

thread_local std::string g_create_error;

struct Region {
  size_t offset = 0;
  template <typename T> T* at(void* base) const { return reinterpret_cast<T*>((char*)base + offset); }
};

// Placement of everything that lives in the caller's workspace blob.
struct Plan {
  size_t total = 0;
  Region status, part, row_loss, logits, ev_a, ev_b, ev_acc, splitk, lse, label_logit, chain_fwd, chain_dx;
  std::vector<Region> idx, off;             // hidden layer l at [l]  (1..t-1)
  std::vector<Region> master, bias, opw;    // layer l at [l]         (1..t)
  std::vector<Region> act, delta;           // act [0..t-1], delta [1..t]
  Region take(size_t bytes) {
    Region r;
    r.offset = total;
    total += (size_t)round_up((int64_t)bytes, 256);
    return r;
  }
};

// Placement of the buffers of the optional batch standardisation (a second caller-owned blob).
struct NormPlan {
  size_t total = 0;
  std::vector<Region> z, mu, rstd;          // training: hidden layer l at [l], per subnet
  std::vector<Region> ev_mu, ev_rstd;       // deployment statistics of the full network
  Region take(size_t bytes) {
    Region r;
    r.offset = total;
    total += (size_t)round_up((int64_t)bytes, 256);
    return r;
  }
};

}  // namespace

struct ist_ctx {
  int t = 0, S = 1, precision = IST_FP32, max_batch = 0, csr = 0;
  std::vector<int64_t> N;    // layer widths N_0..N_t
  std::vector<int64_t> np;   // per-subnet width: N_0, ceil(N_l/S) for hidden l, N_t
  std::vector<int64_t> ld;   // np rounded up to 8 elements (16-byte rows for bf16)
  cudaStream_t stream = nullptr;
  void* ws = nullptr;
  Plan plan;
  int state = ST_CREATED;
  std::vector<float*> W, b;  // bound full network, index l-1
  int64_t launches = 0;
  uint64_t seed = 0;
  std::string err;

  // partition rule and, for the independent rule, the group sizes of the partition in place
  int rule = IST_PART_BALANCED;
  std::vector<std::vector<int64_t>> group_count;   // [hidden layer][subnet]

  // subnets this context trains in ist_local_steps (all S unless ist_set_subnet_range narrowed it)
  int sub_first = 0, sub_count = 0;

  // chained launches: running totals of the row-block counters (index = layer), and the batch size
  // and subnet count they were accumulated with (a change clears counters and totals)
  std::vector<unsigned> fwd_totals, dx_totals;
  int chain_B = -1, chain_S = -1;
  size_t chain_stride() const { return (size_t)S * ceil_div((int64_t)max_batch, 128); }

  // batch standardisation of hidden pre-activations (off unless ist_enable_normalization ran)
  bool norm = false, calibrated = false;
  float norm_eps = 0.f;
  void* nws = nullptr;
  NormPlan nplan;
  float* zbuf(int l) const { return nplan.z[l].at<float>(nws); }
  float* nmu(int l) const { return nplan.mu[l].at<float>(nws); }
  float* nrstd(int l) const { return nplan.rstd[l].at<float>(nws); }
  float* ev_mu(int l) const { return nplan.ev_mu[l].at<float>(nws); }
  float* ev_rstd(int l) const { return nplan.ev_rstd[l].at<float>(nws); }

  // profiling: event pairs around groups of launches of one kernel class
  struct Span { int cls; int64_t kernels; cudaEvent_t a, b; };
  bool profiling = false;
  std::vector<Span> spans;
  std::vector<cudaEvent_t> event_pool;
  cudaEvent_t new_event() {
    cudaEvent_t e = nullptr;
    if (!event_pool.empty()) { e = event_pool.back(); event_pool.pop_back(); }
    else cudaEventCreate(&e);
    return e;
  }
  void clear_spans() {
    for (auto& s : spans) { event_pool.push_back(s.a); event_pool.push_back(s.b); }
    spans.clear();
  }
  ~ist_ctx() {
    clear_spans();
    for (auto e : event_pool) cudaEventDestroy(e);
  }

  size_t esize() const { return precision == IST_BF16 ? 2 : 4; }
  Launch launch() { return Launch{stream, &launches}; }
  DeviceStatus* status() const { return plan.status.at<DeviceStatus>(ws); }
  int32_t* idx(int l) const { return plan.idx[l].at<int32_t>(ws); }
  int32_t* off(int l) const { return plan.off[l].at<int32_t>(ws); }
  float* master(int l) const { return plan.master[l].at<float>(ws); }
  float* bias(int l) const { return plan.bias[l].at<float>(ws); }
  bf16* opw(int l) const { return precision == IST_BF16 ? plan.opw[l].at<bf16>(ws) : nullptr; }
  int64_t rows_pad(int l) const { return np[l - 1]; }              // packed rows of layer l
  int64_t slice_elems(int l) const { return np[l - 1] * ld[l]; }   // per subnet
};

namespace {

// Brackets the launches made during its lifetime when profiling is on.
struct Scope {
  ist_ctx* c;
  int cls;
  int64_t before;
  cudaEvent_t a = nullptr;
  Scope(ist_ctx* ctx, int k) : c(ctx), cls(k), before(ctx->launches) {
    if (c->profiling) {
      a = c->new_event();
      cudaEventRecord(a, c->stream);
    }
  }
  ~Scope() {
    if (a) {
      cudaEvent_t b = c->new_event();
      cudaEventRecord(b, c->stream);
      c->spans.push_back({cls, c->launches - before, a, b});
    }
  }
};

ist_status fail(ist_ctx* c, ist_status code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_create_error = buf;
  return code;
}

bool valid_shape(const int64_t* dims, int n_dims, int S, int precision, int max_batch, std::string* why) {
  if (!dims || n_dims < 2 || n_dims > 64) { *why = "layer_dims must hold 2..64 entries"; return false; }
  if (precision != IST_FP32 && precision != IST_BF16) { *why = "precision must be IST_FP32 or IST_BF16"; return false; }
  // a minibatch runs along the y dimension of several launch grids, which holds 65535 blocks
  if (max_batch < 1 || max_batch > 65535) { *why = "max_batch must be in 1..65535"; return false; }
  if (S < 1) { *why = "S must be >= 1"; return false; }
  for (int i = 0; i < n_dims; ++i)
    if (dims[i] < 1 || dims[i] > (int64_t)1 << 30) { *why = "every layer width must be in 1..2^30"; return false; }
  if (n_dims == 2 && S != 1) { *why = "a network without hidden layers cannot be partitioned: S must be 1"; return false; }
  for (int i = 1; i + 1 < n_dims; ++i)
    if (S > dims[i]) { *why = "S exceeds a hidden layer's width"; return false; }
  return true;
}

// A narrow output layer (bf16 operands, at most 64 padded classes) is handled specially: its
// logits GEMM is cut into k slices (more tiles, shorter pipelines) that the softmax kernel sums.
constexpr int kHeadSplitsMax = 8;
bool narrow_head(const ist_ctx* c) { return c->precision == IST_BF16 && c->t >= 2 && c->ld[c->t] <= 64; }
int head_splits(const ist_ctx* c) {
  const int64_t nkb = ceil_div(c->np[c->t - 1], 64);
  return (int)std::max<int64_t>(1, std::min<int64_t>(kHeadSplitsMax, nkb / 4));
}

// A very wide output layer (bf16 operands): the logits are never stored.  The product is formed
// twice, once for per-row log-sum-exp partials and once for delta = (softmax - onehot) / B.
bool wide_head(const ist_ctx* c) { return c->precision == IST_BF16 && c->ld[c->t] > 8192; }

// delta_{l-1} = delta_l * W_l^T contracts over the width of layer l.  When that width is huge
// (hundreds of thousands of classes) and the output small, the product has too few tiles to
// fill the machine, so the contraction is cut into slices that run as separate tiles.  A product
// that already has a 256 x 256 tile for every pair of SMs is left whole: slices would only add
// fp32 partial slabs to write and read back.
int wanted_k_splits(int64_t K, int64_t out_cols, int S, int B) {
  if (K < 16384) return 1;
  const int64_t tiles = ceil_div(B, 256) * ceil_div(out_cols, 256) * S;
  if (tiles >= 74) return 1;
  return (int)std::min<int64_t>(64, ceil_div(K, 8192));
}

void make_plan(ist_ctx* c) {
  Plan& p = c->plan;
  const int t = c->t, S = c->S;
  const int64_t Bm = c->max_batch;
  p = Plan();
  p.idx.resize(t + 1); p.off.resize(t + 1);
  p.master.resize(t + 1); p.bias.resize(t + 1); p.opw.resize(t + 1);
  p.act.resize(t + 1); p.delta.resize(t + 1);
  p.status = p.take(sizeof(DeviceStatus));
  int64_t maxH = 1, maxN = 0;
  for (int l = 1; l < t; ++l) maxH = std::max(maxH, c->N[l]);
  for (int l = 0; l <= t; ++l) maxN = std::max(maxN, c->N[l]);
  p.part = p.take(partition_scratch_bytes((int)maxH, S));
  for (int l = 1; l < t; ++l) {
    p.idx[l] = p.take(c->N[l] * 4);
    p.off[l] = p.take((S + 1) * 4);
  }
  for (int l = 1; l <= t; ++l) {
    p.master[l] = p.take((size_t)S * c->slice_elems(l) * 4);
    p.bias[l] = p.take((size_t)S * c->ld[l] * 4);
    if (c->precision == IST_BF16) p.opw[l] = p.take((size_t)S * c->slice_elems(l) * 2);
  }
  const size_t es = c->esize();
  if (!c->csr) p.act[0] = p.take((size_t)S * Bm * c->ld[0] * es);   // staging of fp32 inputs
  for (int l = 1; l < t; ++l) p.act[l] = p.take((size_t)S * Bm * c->ld[l] * es);
  for (int l = 1; l <= t; ++l) p.delta[l] = p.take((size_t)S * Bm * c->ld[l] * es);
  if (wide_head(c))   // (max, sum) partials per row and 128 columns instead of the logits themselves
    p.logits = p.take((size_t)S * Bm * gemm_tc_lse_parts(c->ld[t]) * 8);
  else
    p.logits = p.take((size_t)S * Bm * c->ld[t] * 4 * (narrow_head(c) ? kHeadSplitsMax : 1));
  p.row_loss = p.take((size_t)S * Bm * 4);
  p.lse = p.take((size_t)S * Bm * 4);
  p.label_logit = p.take((size_t)S * Bm * 4);
  p.ev_a = p.take((size_t)Bm * maxN * 4);
  p.ev_b = p.take((size_t)Bm * maxN * 4);
  p.ev_acc = p.take(64);
  // fp32 partial products of k-split delta GEMMs (very wide layers only)
  size_t sk = 0;
  if (c->precision == IST_BF16)
    for (int l = 2; l <= t; ++l) {   // batch 1 has the fewest tiles, hence the most slices any batch can ask for
      const int ks = wanted_k_splits(c->np[l], c->np[l - 1], S, 1);
      sk = std::max(sk, (size_t)(ks > 1 ? ks : 0) * S * Bm * c->ld[l - 1] * 4);
    }
  p.splitk = p.take(sk);
  // row-block counters of chained launches (forward chain, delta chain): one set per layer
  const size_t chain_words = (size_t)(t + 1) * S * ceil_div(Bm, 128);
  p.chain_fwd = p.take(c->precision == IST_BF16 ? chain_words * 4 : 0);
  p.chain_dx = p.take(c->precision == IST_BF16 ? chain_words * 4 : 0);
}

void make_norm_plan(ist_ctx* c) {
  NormPlan& p = c->nplan;
  const int t = c->t;
  p = NormPlan();
  p.z.resize(t + 1); p.mu.resize(t + 1); p.rstd.resize(t + 1);
  p.ev_mu.resize(t + 1); p.ev_rstd.resize(t + 1);
  for (int l = 1; l < t; ++l) {
    p.z[l] = p.take((size_t)c->S * c->max_batch * c->ld[l] * 4);
    p.mu[l] = p.take((size_t)c->S * c->ld[l] * 4);
    p.rstd[l] = p.take((size_t)c->S * c->ld[l] * 4);
    p.ev_mu[l] = p.take((size_t)c->N[l] * 4);
    p.ev_rstd[l] = p.take((size_t)c->N[l] * 4);
  }
}

// Rows / columns a subnet's slice of a hidden layer is laid out for.  Balanced groups hold
// ceil(N/S) neurons at most.  Independent assignment gives Binomial(N, 1/S) sizes: the layout has
// room for the mean plus seven standard deviations (a larger draw, probability < 1e-11 per group,
// is refused by ist_partition).
int64_t slice_capacity(int64_t N, int S, int rule) {
  const int64_t mean = ceil_div(N, (int64_t)S);
  if (rule != IST_PART_IID || S == 1) return mean;
  const double sd = std::sqrt((double)N * (1.0 / S) * (1.0 - 1.0 / S));
  return std::min<int64_t>(N, mean + (int64_t)std::ceil(7.0 * sd) + 8);
}

void fill_shape(ist_ctx* c, const int64_t* dims, int n_dims, int S, int precision, int max_batch, int csr,
                int rule = IST_PART_BALANCED) {
  c->rule = rule;
  c->t = n_dims - 1;
  c->S = S;
  c->sub_first = 0;
  c->sub_count = S;
  c->precision = precision;
  c->max_batch = max_batch;
  c->csr = csr ? 1 : 0;
  c->N.assign(dims, dims + n_dims);
  c->np.resize(n_dims);
  c->ld.resize(n_dims);
  for (int l = 0; l <= c->t; ++l) {
    c->np[l] = (l == 0 || l == c->t) ? dims[l] : slice_capacity(dims[l], S, rule);
    c->ld[l] = round_up(c->np[l], 8);
  }
  make_plan(c);
  make_norm_plan(c);
}

ist_status cuda_fail(ist_ctx* c, cudaError_t e, const char* what) {
  return fail(c, IST_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define IST_CUDA(c, call)                                   \
  do {                                                      \
    cudaError_t e_ = (call);                                \
    if (e_ != cudaSuccess) return cuda_fail(c, e_, #call);  \
  } while (0)

uint64_t splitmix64_next(uint64_t* state) {
  uint64_t z = (*state += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Slice map of layer l (1..t): rows follow hidden layer l-1's partition, columns layer l's.
SliceMap slice_map(const ist_ctx* c, int l, int s_first = 0) {
  SliceMap m{};
  m.s_first = s_first;
  const bool rows_indexed = l > 1, cols_indexed = l < c->t;
  m.row_idx = rows_indexed ? c->idx(l - 1) : nullptr;
  m.row_off = rows_indexed ? c->off(l - 1) : nullptr;
  m.col_idx = cols_indexed ? c->idx(l) : nullptr;
  m.col_off = cols_indexed ? c->off(l) : nullptr;
  m.full_rows = c->N[l - 1];
  m.full_cols = c->N[l];
  m.rows_pad = c->np[l - 1];
  m.ld = c->ld[l];
  return m;
}

SliceMap bias_map(const ist_ctx* c, int l, int s_first = 0) {
  SliceMap m{};
  m.s_first = s_first;
  const bool cols_indexed = l < c->t;
  m.col_idx = cols_indexed ? c->idx(l) : nullptr;
  m.col_off = cols_indexed ? c->off(l) : nullptr;
  m.full_rows = 1;
  m.full_cols = c->N[l];
  m.rows_pad = 1;
  m.ld = c->ld[l];
  return m;
}

ist_status check_input(ist_ctx* c, const ist_input* X, const int32_t* y, bool training) {
  if (!X || !y) return fail(c, IST_ERR_ARG, "X and y_dev must not be null");
  if (X->kind != IST_X_DENSE_F32 && X->kind != IST_X_DENSE_BF16 && X->kind != IST_X_CSR)
    return fail(c, IST_ERR_ARG, "unknown input kind %d", X->kind);
  if ((X->kind == IST_X_CSR) != (c->csr != 0))
    return fail(c, IST_ERR_ARG, "input kind does not match input_is_csr given to ist_create");
  if (X->kind == IST_X_CSR) {
    if (!X->row_ptr || !X->col || !X->val) return fail(c, IST_ERR_ARG, "CSR input needs row_ptr, col and val");
  } else {
    if (!X->dense) return fail(c, IST_ERR_ARG, "dense input pointer is null");
    if (X->kind == IST_X_DENSE_BF16) {
      if (c->precision != IST_BF16 && training)
        return fail(c, IST_ERR_UNSUPPORTED, "bf16 inputs need a bf16-precision context");
      if (c->N[0] % 8 != 0 || ((uintptr_t)X->dense & 15))
        return fail(c, IST_ERR_ARG, "bf16 rows need N_0 %% 8 == 0 and a 16-byte aligned base");
    }
  }
  if (training) {
    if (X->batch < 1 || X->batch > c->max_batch)
      return fail(c, IST_ERR_ARG, "batch %d outside 1..max_batch (%d)", X->batch, c->max_batch);
    if (X->stride_subnet < 0 || X->stride_step < 0) return fail(c, IST_ERR_ARG, "negative row stride");
  }
  return IST_OK;
}

// ---- grouped GEMM dispatch ------------------------------------------------------------------
// fp32 operands run on the CUDA cores, bf16 operands on the tensor cores.
bool gemm(ist_ctx* c, const GemmArgs<float>& a) {
  gemm_simt<float>(c->launch(), a);
  return true;
}
bool gemm(ist_ctx* c, const GemmArgs<bf16>& a) { return gemm_tc(c->launch(), a, c->status()); }

// Several products of one kind in as few launches as possible.  fp32 operands: one CUDA-core
// launch each.  bf16 operands: tiles of one tensor-core launch per gemm_tc_max_batch() problems;
// with `chained`, every problem reads the output of the one before it and the launch orders
// their tiles through the row-block counters of `region` (one set per problem, indexed by
// `layer0 + i`; `totals` are the context's running sums for that region).
bool gemm_list(ist_ctx* c, const std::vector<GemmArgs<float>>& v, bool, Region, std::vector<unsigned>*, int,
               const LossReduce* = nullptr) {
  for (auto& g : v) gemm_simt<float>(c->launch(), g);
  return true;
}
// Whether every launch a weight-update list is cut into can sum the deltas for the bias update.
bool update_sums_bias(const std::vector<GemmArgs<float>>&) { return false; }
bool update_sums_bias(const std::vector<GemmArgs<bf16>>& v) {
  const int cap = gemm_tc_max_batch();
  for (size_t i0 = 0; i0 < v.size(); i0 += cap)
    if (!gemm_tc_update_sums_bias(v.data() + i0, (int)std::min<size_t>(cap, v.size() - i0))) return false;
  return !v.empty();
}
// `loss` (weight-update lists only): the first launch also reduces the step's mean losses.
bool gemm_list(ist_ctx* c, const std::vector<GemmArgs<bf16>>& v, bool chained, Region region,
               std::vector<unsigned>* totals, int layer0, const LossReduce* loss = nullptr) {
  const int cap = gemm_tc_max_batch();
  for (size_t i0 = 0; i0 < v.size(); i0 += cap) {
    const int n = (int)std::min<size_t>(cap, v.size() - i0);
    if (chained && n > 1) {
      GemmChain ch{region.at<unsigned>(c->ws) + (size_t)(layer0 + i0) * c->chain_stride(), c->chain_stride(),
                   totals->data() + layer0 + i0};
      if (!gemm_tc_batch(c->launch(), v.data() + i0, n, &ch, nullptr, c->status())) return false;
    } else if (!gemm_tc_batch(c->launch(), v.data() + i0, n, nullptr, i0 == 0 ? loss : nullptr, c->status())) {
      return false;
    }
  }
  return true;
}

// delta GEMM with the contraction cut into slices: fp32 partial slabs, then sum + ReLU mask.
bool split_delta_gemm(ist_ctx*, const GemmArgs<float>&, int, int) { return false; }
bool split_delta_gemm(ist_ctx* c, const GemmArgs<bf16>& masked, int want, int B) {
  const int ks = gemm_tc_splits(masked.K, want);
  float* part = c->plan.splitk.at<float>(c->ws);
  GemmArgs<bf16> g = masked;
  g.epi = EPI_BIAS_F32;
  g.bias = nullptr;
  g.k_splits = ks;
  g.n_off = nullptr; g.k_off = nullptr;   // every slice writes its whole slab: the reduction reads all of it
  g.outf = part; g.outf_ld = masked.out_ld; g.outf_sg = (int64_t)B * masked.out_ld;
  g.out = nullptr; g.mask = nullptr;
  if (!gemm_tc(c->launch(), g, c->status())) return false;
  splitk_mask_reduce<bf16>(c->launch(), part, ks, masked.G, B, masked.out_ld, masked.mask, masked.mask_sg, masked.out,
                           masked.out_sg);
  return true;
}

// Type-dispatch shims: the narrow-head kernels exist for bf16 operands only.
int gemm_splits(int want, int K, const float*) { return 1; }
int gemm_splits(int want, int K, const bf16*) { return gemm_tc_splits(K, want); }
void small_softmax(const Launch&, const float*, int, int64_t, int, int, int, const float*, int64_t, const int32_t*,
                   int64_t, float*, int64_t, int64_t, float*, DeviceStatus*) {}
void small_softmax(const Launch& L, const float* part, int ks, int64_t ld, int G, int B, int Nt, const float* bias,
                   int64_t bias_sg, const int32_t* y, int64_t y_sg, bf16* delta, int64_t ld_d, int64_t sg_d,
                   float* row_loss, DeviceStatus* st) {
  softmax_xent_small<bf16>(L, part, ks, ld, G, B, Nt, bias, bias_sg, y, y_sg, delta, ld_d, sg_d, row_loss, st);
}
// A product written as plain fp32: on the tensor-core path the fp32 epilogue without a bias, on
// the CUDA-core path (operands and output of the same type) a plain store.
void set_plain_fp32_output(GemmArgs<bf16>& g, float* out, int64_t ld, int64_t sg) {
  g.epi = EPI_BIAS_F32; g.bias = nullptr; g.outf = out; g.outf_ld = ld; g.outf_sg = sg;
}
void set_plain_fp32_output(GemmArgs<float>& g, float* out, int64_t ld, int64_t sg) {
  g.epi = EPI_STORE; g.out = out; g.out_ld = ld; g.out_sg = sg;
}
// Working sets up to this size are taken to survive in the 126 MB L2 between two kernels.
constexpr size_t kL2ResidentBytes = 64u << 20;
// One call of ist_local_steps in operand type T.
// dx_out (may be null): fp32 rows addressed like the rows of X; row r receives d(loss)/d(row r).
template <typename T>
ist_status run_local_steps(ist_ctx* c, const ist_input* X, const int32_t* y, float lr, int K,
                           float* loss_out, float* dx_out) {
  // S here is the number of subnets this context trains: slabs s0 .. s0 + S - 1 of the packed
  // weights; activations, deltas and the other scratch buffers use their first S slabs.
  const int t = c->t, S = c->sub_count, s0 = c->sub_first, B = X->batch;
  const int64_t Bm = c->max_batch;
  const bool bf = c->precision == IST_BF16;
  auto act = [&](int l) { return c->plan.act[l].at<T>(c->ws); };
  auto delta = [&](int l) { return c->plan.delta[l].at<T>(c->ws); };
  auto master = [&](int l) { return c->master(l) + (int64_t)s0 * c->slice_elems(l); };
  auto opw = [&](int l) -> bf16* { return bf ? c->opw(l) + (int64_t)s0 * c->slice_elems(l) : nullptr; };
  auto bias_of = [&](int l) { return c->bias(l) + (int64_t)s0 * c->ld[l]; };
  auto weights = [&](int l) -> const T* {       // operand copy of layer l's slices
    return bf ? reinterpret_cast<const T*>(opw(l)) : reinterpret_cast<const T*>(master(l));
  };
  float* logits = c->plan.logits.at<float>(c->ws);
  float* row_loss = c->plan.row_loss.at<float>(c->ws);
  // Unequal subnets (independent assignment): the group offsets of hidden layer l tell the
  // tensor-core launches each group's true extent; null for the input / output layers and under the
  // balanced rule, where every group fills its slab (up to one neuron).
  const bool ragged = c->rule == IST_PART_IID && bf;
  auto off_of = [&](int l) -> const int32_t* { return (ragged && l >= 1 && l < t) ? c->off(l) + s0 : nullptr; };
  DeviceStatus* st = c->status();
  Launch L = c->launch();
  if (bf && (c->chain_B != B || c->chain_S != S)) {
    // the counters' per-launch increments depend on the tile shape, which follows the batch
    if (c->plan.chain_dx.offset > c->plan.chain_fwd.offset)
      IST_CUDA(c, cudaMemsetAsync(c->plan.chain_fwd.at<char>(c->ws), 0,
                                  2 * (c->plan.chain_dx.offset - c->plan.chain_fwd.offset), c->stream));
    c->fwd_totals.assign(t + 2, 0u);
    c->dx_totals.assign(t + 2, 0u);
    c->chain_B = B;
    c->chain_S = S;
  }

  for (int k = 0; k < K; ++k) {
    const int64_t row0 = (int64_t)k * X->stride_step;
    // ---- layer-0 activations ---------------------------------------------------------------
    const T* a0 = nullptr;
    int64_t a0_ld = 0, a0_sg = 0;
    if (X->kind != IST_X_CSR) {
      const bool direct = (X->kind == IST_X_DENSE_BF16) == bf;
      if (direct) {
        a0 = reinterpret_cast<const T*>(X->dense) + row0 * c->N[0];
        a0_ld = c->N[0];
        a0_sg = X->stride_subnet * c->N[0];
      } else {  // fp32 rows into a bf16 context: round into the staging buffer
        Scope sc(c, IST_K_STAGE);
        stage_rows<T>(L, reinterpret_cast<const float*>(X->dense) + row0 * c->N[0], c->N[0],
                      X->stride_subnet, S, B, act(0), c->ld[0], Bm * c->ld[0]);
        a0 = act(0);
        a0_ld = c->ld[0];
        a0_sg = Bm * c->ld[0];
      }
    }
    auto in_ptr = [&](int l) { return l == 0 ? a0 : act(l); };
    auto in_ld = [&](int l) { return l == 0 ? a0_ld : c->ld[l]; };
    auto in_sg = [&](int l) { return l == 0 ? a0_sg : Bm * c->ld[l]; };

    const bool head = narrow_head(c), wide = wide_head(c);
    float* lse = c->plan.lse.at<float>(c->ws);
    float* label_logit = c->plan.label_logit.at<float>(c->ws);
    const int head_ks = head ? gemm_splits(head_splits(c), (int)c->np[t - 1], (const T*)nullptr) : 1;
    // Sec. 2.2: a_l = max((z_l - mean_b z_l) / sigma_b, 0) per subnet and neuron
    auto standardise = [&](int l) {
      Scope sc(c, IST_K_NORM);
      colnorm_forward<T>(L, c->zbuf(l), c->ld[l], Bm * c->ld[l], S, B, (int)c->np[l], c->norm_eps, c->nmu(l),
                         c->nrstd(l), c->ld[l], act(l), Bm * c->ld[l]);
    };
    // ---- forward ---------------------------------------------------------------------------
    // Hidden layers without standardisation form a chain a_l = relu(a_{l-1} W_l + b_l): they are
    // collected and go out together (tiles of one launch, see gemm_list).
    std::vector<GemmArgs<T>> fwd_chain;
    int fwd_chain_l0 = 0;
    auto flush_fwd = [&]() -> bool {
      if (fwd_chain.empty()) return true;
      Scope sc(c, IST_K_FWD);
      const bool ok = gemm_list(c, fwd_chain, true, c->plan.chain_fwd, &c->fwd_totals, fwd_chain_l0);
      fwd_chain.clear();
      return ok;
    };
    for (int l = 1; l <= t; ++l) {
      if (l == 1 && X->kind == IST_X_CSR && t > 1) {
        {
          Scope sc(c, IST_K_SPMM);
          if (c->norm)
            spmm_forward<T, float>(L, X->row_ptr, X->col, X->val, row0, X->stride_subnet, S, B, c->N[0],
                                   weights(1), c->ld[1], c->slice_elems(1), bias_of(1), c->ld[1],
                                   (int)c->np[1], c->zbuf(1), c->ld[1], Bm * c->ld[1], st, false);
          else
            spmm_forward<T, T>(L, X->row_ptr, X->col, X->val, row0, X->stride_subnet, S, B, c->N[0],
                               weights(1), c->ld[1], c->slice_elems(1), bias_of(1), c->ld[1],
                               (int)c->np[1], act(1), c->ld[1], Bm * c->ld[1], st);
        }
        if (c->norm) standardise(1);
        continue;
      }
      GemmArgs<T> g{};
      g.M = B; g.N = (int)c->np[l]; g.K = (int)c->np[l - 1]; g.G = S;
      g.N_store = (int)c->ld[l];
      g.A = in_ptr(l - 1); g.a_sm = in_ld(l - 1); g.a_sk = 1; g.a_sg = in_sg(l - 1);
      g.B = weights(l); g.b_sn = 1; g.b_sk = c->ld[l]; g.b_sg = c->slice_elems(l);
      g.bias = bias_of(l); g.bias_sg = c->ld[l];
      g.n_off = off_of(l); g.k_off = off_of(l - 1);
      if (l < t && c->norm) {
        g.epi = EPI_BIAS_F32;        // fp32 pre-activations; standardisation and ReLU follow
        g.outf = c->zbuf(l); g.outf_ld = c->ld[l]; g.outf_sg = Bm * c->ld[l];
      } else if (l < t) {
        g.epi = EPI_BIAS_RELU;
        g.out = act(l); g.out_ld = c->ld[l]; g.out_sg = Bm * c->ld[l];
      } else if (wide) {
        g.epi = EPI_LSE_PART;        // first pass over the output layer: log-sum-exp partials per row
        g.lse_part = logits;
      } else if (head) {
        g.epi = EPI_BIAS_F32;        // k slices of the logits; bias and the sum happen in the softmax kernel
        g.bias = nullptr;
        g.k_splits = head_ks;
        if (head_ks > 1) g.k_off = nullptr;
        g.outf = logits; g.outf_ld = c->ld[t]; g.outf_sg = (int64_t)B * c->ld[t];
      } else {
        g.epi = EPI_BIAS_F32;
        g.outf = logits; g.outf_ld = c->ld[t]; g.outf_sg = Bm * c->ld[t];
      }
      if (g.epi == EPI_BIAS_RELU) {
        if (fwd_chain.empty()) fwd_chain_l0 = l;
        fwd_chain.push_back(g);
        continue;
      }
      // the k slices of a narrow output layer ride on the hidden layers' launch when there is room
      if (bf && l == t && head && !fwd_chain.empty() && (int)fwd_chain.size() < gemm_tc_max_batch()) {
        fwd_chain.push_back(g);
        if (!flush_fwd()) return fail(c, IST_ERR_UNSUPPORTED, "forward GEMMs cannot be launched");
        continue;
      }
      if (!flush_fwd()) return fail(c, IST_ERR_UNSUPPORTED, "forward GEMMs below layer %d cannot be launched", l);
      {
        Scope sc(c, IST_K_FWD);
        if (!gemm(c, g)) return fail(c, IST_ERR_UNSUPPORTED, "forward GEMM of layer %d cannot be launched", l);
      }
      if (l < t && c->norm) standardise(l);
    }
    if (!flush_fwd()) return fail(c, IST_ERR_UNSUPPORTED, "forward GEMMs cannot be launched");
    // ---- loss and its gradient -------------------------------------------------------------
    {
      Scope sc(c, IST_K_LOSS);
      if (wide) {
        lse_combine(L, logits, gemm_tc_lse_parts(c->ld[t]), S, B, Bm, lse, y + row0, X->stride_subnet, (int)c->N[t], st);
        GemmArgs<T> g{};             // second pass: the same product, written out as delta_t
        g.M = B; g.N = (int)c->np[t]; g.K = (int)c->np[t - 1]; g.G = S;
        g.N_store = (int)c->ld[t];
        g.A = in_ptr(t - 1); g.a_sm = in_ld(t - 1); g.a_sk = 1; g.a_sg = in_sg(t - 1);
        g.B = weights(t); g.b_sn = 1; g.b_sk = c->ld[t]; g.b_sg = c->slice_elems(t);
        g.bias = bias_of(t); g.bias_sg = c->ld[t];
        g.k_off = off_of(t - 1);
        g.epi = EPI_SOFTMAX_DELTA;
        g.out = delta(t); g.out_ld = c->ld[t]; g.out_sg = Bm * c->ld[t];
        g.lse = lse; g.lse_sg = Bm;
        g.labels = y + row0; g.labels_sg = X->stride_subnet;
        g.label_logit = label_logit;
        g.inv_rows = 1.f / (float)B;
        if (!gemm(c, g)) return fail(c, IST_ERR_UNSUPPORTED, "softmax pass of the output layer cannot be launched");
        lse_row_loss(L, lse, label_logit, S, B, Bm, row_loss);
      } else if (head)
        small_softmax(L, logits, head_ks, c->ld[t], S, B, (int)c->N[t], bias_of(t), c->ld[t], y + row0,
                      X->stride_subnet, delta(t), c->ld[t], Bm * c->ld[t], row_loss, st);
      else
      softmax_xent<T>(L, logits, c->ld[t], Bm * c->ld[t], S, B, (int)c->N[t], y + row0,
                      X->stride_subnet, delta(t), c->ld[t], Bm * c->ld[t], row_loss, st);
    }
    // ---- backward + SGD, last layer first --------------------------------------------------
    // db_l = sum_b delta_l, layers l_lo..l_hi; the step's mean losses are reduced by the same launch
    auto update_biases = [&](int l_hi, int l_lo, bool with_loss = true) {
      Scope sc(c, IST_K_BIAS_SGD);
      BiasSgdArgs<T> ba{};
      LossReduce lo{row_loss, with_loss ? loss_out : nullptr, K, k};
      int n = 0;
      for (int l = l_hi; l >= l_lo; --l) {
        ba.layer[n++] = BiasSgdLayer<T>{delta(l), c->ld[l], Bm * c->ld[l], bias_of(l), c->ld[l], (int)c->np[l]};
        if (n == kMaxBiasLayers || l == l_lo) {
          bias_sgd<T>(L, ba, n, S, B, lr, lo);
          lo.loss_out = nullptr;
          n = 0;
        }
      }
    };
    // Every delta is formed from the weights as they stood at the start of the step, so all of
    // them are computed first; the bias update follows at once, while the deltas it sums are still
    // in L2 (after the weight updates have streamed the masters through, they no longer are).
    std::vector<GemmArgs<T>> dx_chain;      // delta_{l-1} = (delta_l W_l^T) * mask, l descending
    int dx_chain_l0 = 0;
    auto flush_dx = [&]() -> bool {
      if (dx_chain.empty()) return true;
      Scope sc(c, IST_K_DX);
      const bool ok = gemm_list(c, dx_chain, true, c->plan.chain_dx, &c->dx_totals, dx_chain_l0);
      dx_chain.clear();
      return ok;
    };
    for (int l = t; l > 1; --l) {
      {
        GemmArgs<T> g{};
        g.M = B; g.N = (int)c->np[l - 1]; g.K = (int)c->np[l]; g.G = S;
        g.N_store = (int)c->ld[l - 1];
        g.A = delta(l); g.a_sm = c->ld[l]; g.a_sk = 1; g.a_sg = Bm * c->ld[l];
        g.B = weights(l); g.b_sn = c->ld[l]; g.b_sk = 1; g.b_sg = c->slice_elems(l);
        g.n_off = off_of(l - 1); g.k_off = off_of(l);
        g.epi = EPI_RELU_MASK;
        g.mask = act(l - 1); g.mask_ld = c->ld[l - 1]; g.mask_sg = Bm * c->ld[l - 1];
        g.out = delta(l - 1); g.out_ld = c->ld[l - 1]; g.out_sg = Bm * c->ld[l - 1];
        const int want = bf ? wanted_k_splits(c->np[l], c->np[l - 1], S, B) : 1;
        if (want > 1) {
          if (!flush_dx()) return fail(c, IST_ERR_UNSUPPORTED, "delta GEMMs above layer %d cannot be launched", l);
          Scope sc(c, IST_K_DX);
          if (!split_delta_gemm(c, g, want, B))
            return fail(c, IST_ERR_UNSUPPORTED, "k-split delta GEMM of layer %d cannot be launched", l);
        } else {
          if (dx_chain.empty()) dx_chain_l0 = t - l;
          dx_chain.push_back(g);
          if (c->norm && !flush_dx())
            return fail(c, IST_ERR_UNSUPPORTED, "delta GEMM of layer %d cannot be launched", l);
        }
      }
      if (c->norm) {   // the masked product is d_zh; carry it through the standardisation
        Scope sc(c, IST_K_NORM);
        colnorm_backward<T>(L, delta(l - 1), c->ld[l - 1], Bm * c->ld[l - 1], c->zbuf(l - 1), Bm * c->ld[l - 1],
                            c->nmu(l - 1), c->nrstd(l - 1), c->ld[l - 1], S, B, (int)c->np[l - 1]);
      }
    }
    if (!flush_dx()) return fail(c, IST_ERR_UNSUPPORTED, "delta GEMMs cannot be launched");
    if (dx_out) {
      // Sec. 2.2, "IST for other architectures": the gradient with respect to the step's inputs,
      // delta_1 W_1^T on every subnet's slice, taken like all gradients at the weights the step
      // started from (the update below has not touched them yet).  This is what a trunk in front
      // of the partitioned layers (held whole at every site) is trained from.
      Scope sc(c, IST_K_DX);
      GemmArgs<T> g{};
      g.M = B; g.N = (int)c->N[0]; g.K = (int)c->np[1]; g.G = S;
      g.N_store = (int)c->N[0];
      g.A = delta(1); g.a_sm = c->ld[1]; g.a_sk = 1; g.a_sg = Bm * c->ld[1];
      g.B = weights(1); g.b_sn = c->ld[1]; g.b_sk = 1; g.b_sg = c->slice_elems(1);
      g.k_off = t > 1 ? off_of(1) : nullptr;
      float* out = dx_out + row0 * c->N[0];
      set_plain_fp32_output(g, out, c->N[0], X->stride_subnet * c->N[0]);
      if (!gemm(c, g)) return fail(c, IST_ERR_UNSUPPORTED, "input-gradient GEMM cannot be launched (N_0 must be a multiple of 4)");
    }
    // the weight updates of the dense layers do not depend on one another: tiles of one launch
    std::vector<GemmArgs<T>> upd;
    for (int l = t; l >= 1; --l) {
      if (l == 1 && X->kind == IST_X_CSR && t > 1) continue;
      GemmArgs<T> g{};
      g.M = (int)c->np[l - 1]; g.N = (int)c->np[l]; g.K = B; g.G = S;
      g.N_store = (int)c->ld[l];
      g.A = in_ptr(l - 1); g.a_sm = 1; g.a_sk = in_ld(l - 1); g.a_sg = in_sg(l - 1);
      g.B = delta(l); g.b_sn = 1; g.b_sk = c->ld[l]; g.b_sg = Bm * c->ld[l];
      g.m_off = off_of(l - 1); g.n_off = off_of(l);
      g.epi = EPI_SGD;
      g.outf = master(l); g.outf_ld = c->ld[l]; g.outf_sg = c->slice_elems(l);
      g.opw = opw(l);
      g.lr = lr;
      upd.push_back(g);
    }
    // Biases are not read by the backward pass, so their update may come before or after the
    // weight updates.  With bf16 operands the weight-update launch does it on the side, in two
    // warps per CTA that sum the deltas and also reduce the step's mean losses: out of the operand
    // stages it streams anyway when the deltas of a step are too large to be still in L2 and the
    // launch runs on single CTAs (a very wide output layer), from memory otherwise (from L2 as a
    // rule; deltas beyond its size come from DRAM a second time there, as they would for the bias
    // kernel, but in the shadow of the update).  What is left for the bias kernel is a sparse
    // first layer's bias and the fp32 path, where it runs first if the deltas fit in L2 and last
    // otherwise.
    const bool sparse_first = X->kind == IST_X_CSR && t > 1;
    size_t delta_bytes = 0;
    for (int l = 1; l <= t; ++l) delta_bytes += (size_t)S * B * c->ld[l] * sizeof(T);
    const bool bias_first = delta_bytes <= kL2ResidentBytes;
    const bool bias_in_gemm = bf;
    const bool from_stages = bias_in_gemm && !bias_first && update_sums_bias(upd);
    if (bias_in_gemm) {
      for (auto& g : upd) {
        const int l = t - (int)(&g - upd.data());   // upd[i] is layer t - i
        g.bias_upd = bias_of(l); g.bias_upd_sg = c->ld[l]; g.bias_n = (int)c->np[l];
        g.bias_upd_from_memory = from_stages ? 0 : 1;
      }
      if (sparse_first) update_biases(1, 1, false);
    } else if (bias_first) {
      update_biases(t, 1);
    }
    {
      Scope sc(c, IST_K_DW_SGD);
      LossReduce lo{row_loss, loss_out, K, k};
      if (!gemm_list(c, upd, false, Region(), nullptr, 0, (bias_in_gemm && loss_out) ? &lo : nullptr))
        return fail(c, IST_ERR_UNSUPPORTED, "weight-gradient GEMMs cannot be launched");
    }
    if (X->kind == IST_X_CSR && t > 1) {
      Scope sc(c, IST_K_SPMM);
      spmm_backward_sgd<T>(L, X->row_ptr, X->col, X->val, row0, X->stride_subnet, S, B, c->N[0],
                           delta(1), c->ld[1], Bm * c->ld[1], (int)c->np[1], master(1), opw(1),
                           c->ld[1], c->slice_elems(1), lr);
    }
    if (!bias_in_gemm && !bias_first) update_biases(t, 1);
  }
  IST_CUDA(c, cudaGetLastError());
  return IST_OK;
}

}  // namespace

// ================================= public entry points =======================================

extern "C" size_t ist_workspace_bytes2(const int64_t* layer_dims, int n_dims, int S, int precision,
                                       int max_batch, int input_is_csr, int partition_rule) {
  std::string why;
  if (!valid_shape(layer_dims, n_dims, S, precision, max_batch, &why)) {
    g_create_error = why;
    return 0;
  }
  if (partition_rule != IST_PART_BALANCED && partition_rule != IST_PART_IID) {
    g_create_error = "unknown partition rule";
    return 0;
  }
  ist_ctx tmp;
  fill_shape(&tmp, layer_dims, n_dims, S, precision, max_batch, input_is_csr, partition_rule);
  return tmp.plan.total;
}

extern "C" size_t ist_workspace_bytes(const int64_t* layer_dims, int n_dims, int S, int precision,
                                      int max_batch, int input_is_csr) {
  return ist_workspace_bytes2(layer_dims, n_dims, S, precision, max_batch, input_is_csr, IST_PART_BALANCED);
}

extern "C" ist_status ist_create2(ist_ctx** out, const int64_t* layer_dims, int n_dims, int S,
                                  int precision, int max_batch, int input_is_csr, int partition_rule,
                                  void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return fail(nullptr, IST_ERR_ARG, "out must not be null");
  std::string why;
  if (!valid_shape(layer_dims, n_dims, S, precision, max_batch, &why))
    return fail(nullptr, IST_ERR_ARG, "%s", why.c_str());
  if (partition_rule != IST_PART_BALANCED && partition_rule != IST_PART_IID)
    return fail(nullptr, IST_ERR_ARG, "unknown partition rule %d", partition_rule);
  if (input_is_csr && n_dims < 3)
    return fail(nullptr, IST_ERR_UNSUPPORTED, "CSR inputs need at least one hidden layer");
  ist_ctx* c = new ist_ctx();
  fill_shape(c, layer_dims, n_dims, S, precision, max_batch, input_is_csr, partition_rule);
  if (!workspace_dev || ((uintptr_t)workspace_dev & 255)) {
    delete c;
    return fail(nullptr, IST_ERR_WORKSPACE, "workspace must be a 256-byte aligned device pointer");
  }
  if (workspace_bytes < c->plan.total) {
    size_t need = c->plan.total;
    delete c;
    return fail(nullptr, IST_ERR_WORKSPACE, "workspace holds %zu bytes, %zu needed", workspace_bytes, need);
  }
  c->ws = workspace_dev;
  c->stream = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaMemsetAsync(workspace_dev, 0, c->plan.total, c->stream);
  if (e != cudaSuccess) {
    delete c;
    return fail(nullptr, IST_ERR_CUDA, "clearing the workspace: %s", cudaGetErrorString(e));
  }
  *out = c;
  return IST_OK;
}

extern "C" ist_status ist_create(ist_ctx** out, const int64_t* layer_dims, int n_dims, int S,
                                 int precision, int max_batch, int input_is_csr, void* workspace_dev,
                                 size_t workspace_bytes, void* cuda_stream) {
  return ist_create2(out, layer_dims, n_dims, S, precision, max_batch, input_is_csr, IST_PART_BALANCED,
                     workspace_dev, workspace_bytes, cuda_stream);
}

extern "C" ist_status ist_bind_weights(ist_ctx* c, float* const* W_dev, float* const* b_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state == ST_PARTITIONED) return fail(c, IST_ERR_STATE, "cannot rebind between ist_partition and ist_reassemble");
  if (!W_dev || !b_dev) return fail(c, IST_ERR_ARG, "W_dev and b_dev must not be null");
  for (int l = 0; l < c->t; ++l) {
    if (!W_dev[l] || !b_dev[l]) return fail(c, IST_ERR_ARG, "layer %d: null weight or bias pointer", l + 1);
    if (((uintptr_t)W_dev[l] & 15) || ((uintptr_t)b_dev[l] & 3))
      return fail(c, IST_ERR_ARG, "layer %d: weights must be 16-byte aligned", l + 1);
  }
  c->W.assign(W_dev, W_dev + c->t);
  c->b.assign(b_dev, b_dev + c->t);
  c->calibrated = false;
  c->state = ST_BOUND;
  return IST_OK;
}

extern "C" ist_status ist_partition(ist_ctx* c, uint64_t seed) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_BOUND) return fail(c, IST_ERR_STATE, "ist_partition needs bound weights and no partition in place");
  Launch L = c->launch();
  const int t = c->t, S = c->S;
  c->seed = seed;
  uint64_t round_state = seed;
  if (c->rule == IST_PART_IID) {
    // group sizes of this draw, from the same rule on the host: nothing is enqueued if a group
    // does not fit the layout the workspace was sized for
    uint64_t st = seed;
    c->group_count.assign(t, std::vector<int64_t>(S, 0));
    for (int l = 1; l < t; ++l) {
      const uint64_t layer_seed = splitmix64_next(&st);
      partition_iid_counts_host(layer_seed, (int)c->N[l], S, c->group_count[l].data());
      for (int s = 0; s < S; ++s)
        if (c->group_count[l][s] > c->np[l])
          return fail(c, IST_ERR_UNSUPPORTED,
                      "seed %llu puts %lld neurons of hidden layer %d into subnet %d; the layout holds %lld",
                      (unsigned long long)seed, (long long)c->group_count[l][s], l, s, (long long)c->np[l]);
    }
  }
  for (int l = 1; l < t; ++l) {
    Scope sc(c, IST_K_PARTITION);
    uint64_t layer_seed = splitmix64_next(&round_state);
    PartitionScratch ps{};
    partition_scratch_carve(c->plan.part.at<char>(c->ws), (int)c->N[l], S, &ps);
    const bool ok = c->rule == IST_PART_IID
                        ? partition_layer_iid(L, layer_seed, (int)c->N[l], S, ps, c->idx(l), c->off(l), c->status())
                        : partition_layer(L, layer_seed, (int)c->N[l], S, ps, c->idx(l), c->off(l), c->status());
    if (!ok) return fail(c, IST_ERR_UNSUPPORTED, "S = %d exceeds what the partition kernels support (768)", S);
  }
  // only the subnets this context trains are gathered (Sec. 2.3: a site receives its own slices)
  for (int l = 1; l <= t; ++l) {
    Scope sc(c, IST_K_GATHER);
    gather_slices(L, c->W[l - 1], slice_map(c, l, c->sub_first), c->sub_count, c->master(l), c->opw(l), c->status());
    gather_slices(L, c->b[l - 1], bias_map(c, l, c->sub_first), c->sub_count, c->bias(l), nullptr, c->status());
  }
  IST_CUDA(c, cudaGetLastError());
  c->state = ST_PARTITIONED;
  return IST_OK;
}

extern "C" ist_status ist_get_partition(ist_ctx* c, int hidden_layer, int32_t* idx_out_dev,
                                        int32_t* off_out_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "no partition in place");
  if (hidden_layer < 1 || hidden_layer >= c->t) return fail(c, IST_ERR_ARG, "hidden_layer outside 1..t-1");
  if (idx_out_dev)
    IST_CUDA(c, cudaMemcpyAsync(idx_out_dev, c->idx(hidden_layer), c->N[hidden_layer] * 4,
                                cudaMemcpyDeviceToDevice, c->stream));
  if (off_out_dev)
    IST_CUDA(c, cudaMemcpyAsync(off_out_dev, c->off(hidden_layer), (c->S + 1) * 4,
                                cudaMemcpyDeviceToDevice, c->stream));
  return IST_OK;
}

namespace {
// |G_l^s| under the partition in place; the input and output layers belong to every subnet whole
int64_t group_size(const ist_ctx* c, int l, int s) {
  if (l == 0 || l == c->t) return c->N[l];
  if (c->rule == IST_PART_IID) return c->group_count[l][s];
  return c->N[l] / c->S + (s < c->N[l] % c->S ? 1 : 0);
}
}  // namespace

extern "C" ist_status ist_subnet_slice_shape(ist_ctx* c, int layer, int s, int64_t* rows_out_host,
                                             int64_t* cols_out_host) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "no partition in place");
  if (layer < 1 || layer > c->t || s < 0 || s >= c->S) return fail(c, IST_ERR_ARG, "layer or subnet out of range");
  if (rows_out_host) *rows_out_host = group_size(c, layer - 1, s);
  if (cols_out_host) *cols_out_host = group_size(c, layer, s);
  return IST_OK;
}

extern "C" ist_status ist_get_subnet_params(ist_ctx* c, int layer, int s, float* W_out_dev,
                                            float* b_out_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "no partition in place");
  if (layer < 1 || layer > c->t || s < 0 || s >= c->S) return fail(c, IST_ERR_ARG, "layer or subnet out of range");
  auto count = [&](int l) { return group_size(c, l, s); };
  Launch L = c->launch();
  if (W_out_dev)
    copy_out_slice(L, c->master(layer) + (int64_t)s * c->slice_elems(layer), c->ld[layer],
                   count(layer - 1), count(layer), W_out_dev);
  if (b_out_dev)
    copy_out_slice(L, c->bias(layer) + (int64_t)s * c->ld[layer], c->ld[layer], 1, count(layer), b_out_dev);
  IST_CUDA(c, cudaGetLastError());
  return IST_OK;
}

extern "C" ist_status ist_local_steps(ist_ctx* c, const ist_input* X, const int32_t* y_dev, float lr,
                                      int K, float* loss_out_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "ist_local_steps needs a partition in place");
  if (K < 1) return fail(c, IST_ERR_ARG, "K must be >= 1");
  if (!(lr == lr)) return fail(c, IST_ERR_ARG, "lr is NaN");
  ist_status s = check_input(c, X, y_dev, true);
  if (s != IST_OK) return s;
  if (c->precision == IST_BF16) return run_local_steps<bf16>(c, X, y_dev, lr, K, loss_out_dev, nullptr);
  return run_local_steps<float>(c, X, y_dev, lr, K, loss_out_dev, nullptr);
}

extern "C" ist_status ist_local_steps_dx(ist_ctx* c, const ist_input* X, const int32_t* y_dev, float lr,
                                         int K, float* loss_out_dev, float* dx_out_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "ist_local_steps_dx needs a partition in place");
  if (K < 1) return fail(c, IST_ERR_ARG, "K must be >= 1");
  if (!(lr == lr)) return fail(c, IST_ERR_ARG, "lr is NaN");
  if (!dx_out_dev) return fail(c, IST_ERR_ARG, "dx_out_dev must not be null");
  ist_status s = check_input(c, X, y_dev, true);
  if (s != IST_OK) return s;
  if (X->kind == IST_X_CSR) return fail(c, IST_ERR_UNSUPPORTED, "the input gradient is defined for dense inputs only");
  if (c->precision == IST_BF16 && c->N[0] % 4 != 0)
    return fail(c, IST_ERR_UNSUPPORTED, "the input gradient on the bf16 path needs N_0 to be a multiple of 4");
  if (c->precision == IST_BF16) return run_local_steps<bf16>(c, X, y_dev, lr, K, loss_out_dev, dx_out_dev);
  return run_local_steps<float>(c, X, y_dev, lr, K, loss_out_dev, dx_out_dev);
}

extern "C" ist_status ist_set_subnet_range(ist_ctx* c, int first, int count) {
  if (!c) return IST_ERR_ARG;
  if (c->state == ST_PARTITIONED)
    return fail(c, IST_ERR_STATE, "the subnet range cannot change between ist_partition and ist_reassemble");
  if (first < 0 || count < 1 || first > c->S - count)
    return fail(c, IST_ERR_ARG, "subnet range [%d, %d) outside [0, %d)", first, first + count, c->S);
  c->sub_first = first;
  c->sub_count = count;
  return IST_OK;
}

extern "C" ist_status ist_packed_layer(ist_ctx* c, int layer, void** master_dev, size_t* master_bytes_per_subnet,
                                       void** bias_dev, size_t* bias_bytes_per_subnet) {
  if (!c) return IST_ERR_ARG;
  if (layer < 1 || layer > c->t) return fail(c, IST_ERR_ARG, "layer outside 1..t");
  if (master_dev) *master_dev = c->master(layer);
  if (master_bytes_per_subnet) *master_bytes_per_subnet = (size_t)c->slice_elems(layer) * 4;
  if (bias_dev) *bias_dev = c->bias(layer);
  if (bias_bytes_per_subnet) *bias_bytes_per_subnet = (size_t)c->ld[layer] * 4;
  return IST_OK;
}

extern "C" ist_status ist_reassemble(ist_ctx* c) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_PARTITIONED) return fail(c, IST_ERR_STATE, "ist_reassemble needs a partition in place");
  Launch L = c->launch();
  const int t = c->t, S = c->S;
  for (int l = 1; l <= t; ++l) {
    Scope sc(c, IST_K_SCATTER);
    scatter_slices(L, c->W[l - 1], slice_map(c, l), S, c->master(l), c->status());
    if (l < t) scatter_slices(L, c->b[l - 1], bias_map(c, l), S, c->bias(l), c->status());
  }
  {
    Scope sc(c, IST_K_SCATTER);
    scatter_mean_bias(L, c->b[t - 1], c->N[t], S, c->bias(t), c->ld[t]);
  }
  IST_CUDA(c, cudaGetLastError());
  c->state = ST_BOUND;
  c->calibrated = false;   // deployment statistics belong to the weights they were taken with
  return IST_OK;
}

namespace {

// Full-width forward of rows r0..r0+rows-1 in fp32.  Hidden layers apply ReLU directly, or, in
// normalisation mode, the stored statistics (measure = false) or statistics taken over these
// very rows, which are then stored (measure = true).  Returns the buffer holding layer
// `last`'s output (row stride N_last).
const float* full_forward(ist_ctx* c, const ist_input* X, int64_t r0, int rows, int last, bool measure) {
  Launch L = c->launch();
  float* buf[2] = {c->plan.ev_a.at<float>(c->ws), c->plan.ev_b.at<float>(c->ws)};
  const float* in = nullptr;
  int64_t in_ld = 0;
  int cur = 0;
  for (int l = 1; l <= last; ++l) {
    float* o = buf[cur];
    const bool hidden = l < c->t;
    if (l == 1 && X->kind == IST_X_CSR) {
      spmm_forward<float, float>(L, X->row_ptr, X->col, X->val, r0, 0, 1, rows, c->N[0], c->W[0], c->N[1],
                                 0, c->b[0], 0, (int)c->N[1], o, c->N[1], 0, c->status(), !c->norm);
    } else {
      GemmArgs<float> g{};
      g.M = rows; g.N = (int)c->N[l]; g.K = (int)c->N[l - 1]; g.G = 1;
      if (l == 1) { g.A = reinterpret_cast<const float*>(X->dense) + r0 * c->N[0]; g.a_sm = c->N[0]; }
      else { g.A = in; g.a_sm = in_ld; }
      g.a_sk = 1;
      g.B = c->W[l - 1]; g.b_sn = 1; g.b_sk = c->N[l];
      g.bias = c->b[l - 1];
      if (hidden && !c->norm) { g.epi = EPI_BIAS_RELU; g.out = o; g.out_ld = c->N[l]; }
      else { g.epi = EPI_BIAS_F32; g.outf = o; g.outf_ld = c->N[l]; }
      gemm_simt<float>(L, g);
    }
    if (hidden && c->norm) {
      if (measure)
        colnorm_forward<float>(L, o, c->N[l], 0, 1, rows, (int)c->N[l], c->norm_eps, c->ev_mu(l), c->ev_rstd(l), 0,
                               o, 0);
      else
        colnorm_apply(L, o, c->N[l], rows, (int)c->N[l], c->ev_mu(l), c->ev_rstd(l));
    }
    in = o;
    in_ld = c->N[l];
    cur ^= 1;
  }
  return in;
}

}  // namespace

extern "C" ist_status ist_eval(ist_ctx* c, const ist_input* X, const int32_t* y_dev, int64_t n,
                               float* mean_loss_out_dev, int64_t* n_correct_out_dev) {
  if (!c) return IST_ERR_ARG;
  if (c->state != ST_BOUND) return fail(c, IST_ERR_STATE, "ist_eval needs bound weights and no partition in place");
  if (c->norm && c->t > 1 && !c->calibrated)
    return fail(c, IST_ERR_STATE, "normalisation is enabled: ist_calibrate must run before ist_eval");
  if (n < 1) return fail(c, IST_ERR_ARG, "n must be >= 1");
  if (!mean_loss_out_dev || !n_correct_out_dev) return fail(c, IST_ERR_ARG, "output pointers must not be null");
  ist_status s = check_input(c, X, y_dev, false);
  if (s != IST_OK) return s;
  if (X->kind == IST_X_DENSE_BF16) return fail(c, IST_ERR_UNSUPPORTED, "ist_eval takes fp32 or CSR rows");
  Launch L = c->launch();
  double* loss_sum = c->plan.ev_acc.at<double>(c->ws);
  long long* correct = reinterpret_cast<long long*>(loss_sum + 1);
  IST_CUDA(c, cudaMemsetAsync(loss_sum, 0, 16, c->stream));
  Scope sc(c, IST_K_EVAL);
  for (int64_t r0 = 0; r0 < n; r0 += c->max_batch) {
    const int rows = (int)std::min<int64_t>(c->max_batch, n - r0);
    const float* logits = full_forward(c, X, r0, rows, c->t, false);
    eval_rows(L, logits, c->N[c->t], rows, (int)c->N[c->t], y_dev + r0, loss_sum, correct, c->status());
  }
  eval_finalize(L, loss_sum, correct, n, mean_loss_out_dev, n_correct_out_dev);
  IST_CUDA(c, cudaGetLastError());
  return IST_OK;
}

extern "C" size_t ist_norm_workspace_bytes(const ist_ctx* c) { return c ? std::max<size_t>(c->nplan.total, 256) : 0; }

extern "C" ist_status ist_enable_normalization(ist_ctx* c, float eps, void* norm_workspace_dev,
                                               size_t norm_workspace_bytes) {
  if (!c) return IST_ERR_ARG;
  if (c->state == ST_PARTITIONED)
    return fail(c, IST_ERR_STATE, "normalisation cannot be switched on between ist_partition and ist_reassemble");
  if (c->norm) return fail(c, IST_ERR_STATE, "normalisation is already enabled");
  if (!(eps > 0.f) || !(eps < 1e30f)) return fail(c, IST_ERR_ARG, "eps must be a positive finite number");
  if (!norm_workspace_dev || ((uintptr_t)norm_workspace_dev & 255))
    return fail(c, IST_ERR_WORKSPACE, "normalisation workspace must be a 256-byte aligned device pointer");
  if (norm_workspace_bytes < c->nplan.total)
    return fail(c, IST_ERR_WORKSPACE, "normalisation workspace holds %zu bytes, %zu needed", norm_workspace_bytes,
                c->nplan.total);
  if (c->nplan.total) IST_CUDA(c, cudaMemsetAsync(norm_workspace_dev, 0, c->nplan.total, c->stream));
  c->nws = norm_workspace_dev;
  c->norm_eps = eps;
  c->norm = true;
  c->calibrated = false;
  return IST_OK;
}

extern "C" ist_status ist_calibrate(ist_ctx* c, const ist_input* X, int64_t n) {
  if (!c) return IST_ERR_ARG;
  if (!c->norm) return fail(c, IST_ERR_STATE, "ist_calibrate needs ist_enable_normalization first");
  if (c->state != ST_BOUND) return fail(c, IST_ERR_STATE, "ist_calibrate needs bound weights and no partition in place");
  if (n < 1 || n > c->max_batch) return fail(c, IST_ERR_ARG, "n must be in 1..max_batch (%d)", c->max_batch);
  if (!X) return fail(c, IST_ERR_ARG, "X must not be null");
  const int32_t dummy = 0;
  ist_status s = check_input(c, X, &dummy, false);
  if (s != IST_OK) return s;
  if (X->kind == IST_X_DENSE_BF16) return fail(c, IST_ERR_UNSUPPORTED, "ist_calibrate takes fp32 or CSR rows");
  {
    Scope sc(c, IST_K_EVAL);
    full_forward(c, X, 0, (int)n, c->t - 1, true);
  }
  IST_CUDA(c, cudaGetLastError());
  c->calibrated = true;
  return IST_OK;
}

extern "C" ist_status ist_sync_status(ist_ctx* c) {
  if (!c) return IST_ERR_ARG;
  DeviceStatus h{};
  IST_CUDA(c, cudaMemcpyAsync(&h, c->status(), sizeof h, cudaMemcpyDeviceToHost, c->stream));
  IST_CUDA(c, cudaStreamSynchronize(c->stream));
  if (h.code != 0) {
    static const char* sites[] = {"", "label out of range", "CSR column out of range",
                                  "partition index out of range", "tensor-core pipeline wait expired",
                                  "CSR row_ptr not monotone"};
    const char* w = (h.site >= 0 && h.site <= 5) ? sites[h.site] : "?";
    return fail(c, (ist_status)h.code, "device status %d: %s (detail %lld)", h.code, w, h.detail);
  }
  return IST_OK;
}

extern "C" ist_status ist_selftest_wait_expiry(ist_ctx* c, int64_t limit_cycles) {
  if (!c) return IST_ERR_ARG;
  if (limit_cycles < 1 || limit_cycles > 2000000000ll)
    return fail(c, IST_ERR_ARG, "limit_cycles must be in 1..2e9 (about a second)");
  if (!gemm_tc_wait_selftest(c->launch(), c->status(), limit_cycles))
    return fail(c, IST_ERR_CUDA, "the self-test kernel could not be launched");
  return IST_OK;
}

extern "C" ist_status ist_profile(ist_ctx* c, int enable) {
  if (!c) return IST_ERR_ARG;
  IST_CUDA(c, cudaStreamSynchronize(c->stream));
  if (enable) c->clear_spans();
  c->profiling = enable != 0;
  return IST_OK;
}

extern "C" ist_status ist_profile_read(ist_ctx* c, int kernel_class, int64_t* launches_out_host,
                                       double* ms_out_host) {
  if (!c) return IST_ERR_ARG;
  if (kernel_class < 0 || kernel_class >= IST_K_COUNT) return fail(c, IST_ERR_ARG, "unknown kernel class");
  IST_CUDA(c, cudaStreamSynchronize(c->stream));
  int64_t n = 0;
  double ms = 0.0;
  for (auto& s : c->spans) {
    if (s.cls != kernel_class) continue;
    float t = 0.f;
    IST_CUDA(c, cudaEventElapsedTime(&t, s.a, s.b));
    ms += t;
    n += s.kernels;
  }
  if (launches_out_host) *launches_out_host = n;
  if (ms_out_host) *ms_out_host = ms;
  return IST_OK;
}

extern "C" int64_t ist_kernel_launches(const ist_ctx* c) { return c ? c->launches : 0; }

extern "C" const char* ist_last_error(const ist_ctx* c) {
  return c ? c->err.c_str() : g_create_error.c_str();
}

extern "C" void ist_destroy(ist_ctx* c) { delete c; }
