// Host-side logic of libpipe: descriptor validation, blob layout, status word, small utilities.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "pipe_common.cuh"
#include "pipe_diag.h"

namespace pipe {

__device__ int g_status_word = 0;

static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_kernel_choice{0};

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }
int kernel_choice() { return g_kernel_choice.load(); }

namespace {
std::mutex g_mark_mutex;
constexpr int kMaxMarked = 64;
cudaStream_t g_marked[kMaxMarked];
int g_num_marked = 0;
bool g_mark_overflow = false;   // more streams than the table holds: every call is then treated as following an expansion
}  // namespace

void mark_expansion(cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_mark_mutex);
  for (int i = 0; i < g_num_marked; ++i)
    if (g_marked[i] == stream) return;
  if (g_num_marked < kMaxMarked) g_marked[g_num_marked++] = stream;
  else g_mark_overflow = true;
}

bool take_expansion_mark(cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_mark_mutex);
  if (g_mark_overflow) return true;
  for (int i = 0; i < g_num_marked; ++i)
    if (g_marked[i] == stream) {
      g_marked[i] = g_marked[--g_num_marked];
      return true;
    }
  return false;
}

bool expansion_marked(cudaStream_t stream) {
  std::lock_guard<std::mutex> lock(g_mark_mutex);
  if (g_mark_overflow) return true;
  for (int i = 0; i < g_num_marked; ++i)
    if (g_marked[i] == stream) return true;
  return false;
}

int* device_status_word() {
  // The symbol is per device; its address is looked up once for whichever device is current and kept.
  constexpr int kMaxDevices = 64;
  static std::atomic<int*> cached[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int* p = cached[dev].load(std::memory_order_acquire);
  if (p) return p;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word) != cudaSuccess) return nullptr;
  cached[dev].store(p, std::memory_order_release);
  return p;
}

static uint64_t align_up64(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

static pipe_status resolve_layer_uncached(const pipe_layer_desc* d, LayerInfo* out);

// Every entry point resolves its descriptor; a serving loop passes the same few descriptors again and again, so
// each host thread keeps the last ones it resolved (the result is a pure function of the descriptor's bytes).
pipe_status resolve_layer(const pipe_layer_desc* d, LayerInfo* out) {
  if (!d || !out) return PIPE_ERR_INVALID_ARG;
  constexpr int kKept = 4;
  struct Entry {
    pipe_layer_desc desc;
    LayerInfo info;
    bool valid;
  };
  thread_local Entry kept[kKept] = {};
  thread_local int next = 0;
  for (int i = 0; i < kKept; ++i)
    if (kept[i].valid && std::memcmp(&kept[i].desc, d, sizeof(pipe_layer_desc)) == 0) {
      *out = kept[i].info;
      return PIPE_OK;
    }
  const pipe_status st = resolve_layer_uncached(d, out);
  if (st == PIPE_OK) {
    Entry& e = kept[next];
    next = (next + 1) % kKept;
    e.desc = *d;
    e.info = *out;
    e.valid = true;
  }
  return st;
}

static pipe_status resolve_layer_uncached(const pipe_layer_desc* d, LayerInfo* out) {
  if (d->out_features <= 0 || d->in_features <= 0) return PIPE_ERR_INVALID_ARG;
  if (!(d->weight_bits == 8 || d->weight_bits == 6 || d->weight_bits == 4 || d->weight_bits == 3 || d->weight_bits == 2))
    return PIPE_ERR_INVALID_ARG;
  if (d->score_mode != PIPE_SCORE_MAXABS && d->score_mode != PIPE_SCORE_L2) return PIPE_ERR_INVALID_ARG;
  if (d->keep_elems < 0 || d->keep_elems > d->in_features) return PIPE_ERR_INVALID_ARG;
  if (d->int8_copy != 0 && d->int8_copy != 1) return PIPE_ERR_INVALID_ARG;
  if (d->num_orders < 1 || d->num_orders > PIPE_MAX_ORDERS) return PIPE_ERR_INVALID_ARG;
  if (d->group_size < 1) return PIPE_ERR_INVALID_ARG;
  if (d->out_features % d->group_size != 0) return PIPE_ERR_SHAPE;
  if (d->int8_copy && d->group_size % 8 != 0) return PIPE_ERR_SHAPE;   // kept-row runs must keep the 8-row swizzle atoms whole
  const int container = d->weight_bits == 2 ? 2 : (d->weight_bits <= 4 ? 4 : 8);   // storage format of the codes
  const int per_byte = 8 / container;
  if (d->in_features % per_byte != 0) return PIPE_ERR_SHAPE;
  LayerInfo L;
  std::memset(&L, 0, sizeof(L));
  L.O = d->out_features;
  L.I = d->in_features;
  L.bits = container;
  L.wbits = d->weight_bits;
  L.score_mode = d->score_mode;
  L.keep_elems = d->keep_elems;
  L.K = d->num_orders;
  L.g = d->group_size;
  L.G = L.O / L.g;
  L.n_keep = d->keep_groups;
  L.M = d->num_branches;
  L.qmax = (1 << (L.wbits - 1)) - 1;
  if (L.n_keep < 1 || L.n_keep > L.G) return PIPE_ERR_INVALID_ARG;
  if (L.keep_elems > 0 && L.n_keep != L.G) return PIPE_ERR_SHAPE;
  if (L.M < 1 || L.M > L.K) return PIPE_ERR_SHAPE;
  // int32 partial sums (Eq. 9 is exact integer work).  The tensor-core and decode kernels accumulate sub-byte
  // codes as code * 2^(8-b) and shift back at the end, so the bound that keeps every kernel exact is
  // 127 * qmax * 2^(8-b) * I < 2^31: I <= 133144 (b = 8), 150976 (b = 4), 264208 (b = 2).
  if ((static_cast<int64_t>(127) * L.qmax * L.I << (8 - L.bits)) >= (static_cast<int64_t>(1) << 31)) return PIPE_ERR_ACC_OVERFLOW;

  int32_t bo[PIPE_MAX_ORDERS] = {0};
  bool all_zero = true;
  for (int m = 0; m < PIPE_MAX_ORDERS; ++m) all_zero = all_zero && d->branch_orders[m] == 0;
  if (all_zero) {
    for (int m = 0; m < L.M; ++m) bo[m] = L.K / L.M + (m < L.K % L.M ? 1 : 0);
  } else {
    int sum = 0;
    for (int m = 0; m < PIPE_MAX_ORDERS; ++m) {
      if (m < L.M) {
        if (d->branch_orders[m] < 1) return PIPE_ERR_SHAPE;
        bo[m] = d->branch_orders[m];
        sum += bo[m];
      } else if (d->branch_orders[m] != 0) {
        return PIPE_ERR_SHAPE;
      }
    }
    if (sum != L.K) return PIPE_ERR_SHAPE;
  }
  L.branch_begin[0] = 0;
  for (int m = 0; m < L.M; ++m) L.branch_begin[m + 1] = L.branch_begin[m] + bo[m];

  pipe_layer_layout& y = L.lay;
  y.num_groups = L.G;
  y.canon_row_bytes = static_cast<int32_t>(static_cast<int64_t>(L.I) * L.bits / 8);
  y.kernel_row_bytes = static_cast<int32_t>(static_cast<int64_t>(round_up(L.I, kKernelKAlign)) * L.bits / 8);
  for (int m = 0; m < L.M; ++m) y.branch_orders[m] = bo[m];
  uint64_t off = kHeaderBytes;
  int64_t total = 0;
  for (int k = 0; k < L.K; ++k) {
    const int kept = (k == 0) ? L.G : L.n_keep;
    y.kept_groups[k] = kept;
    y.rows[k] = kept * L.g;
    total += y.rows[k];
    y.codes_off[k] = off;
    off = align_up64(off + static_cast<uint64_t>(y.rows[k]) * y.canon_row_bytes, 256);
    y.scales_off[k] = off;
    off = align_up64(off + static_cast<uint64_t>(y.rows[k]) * 4, 256);
    y.kept_off[k] = off;
    off = align_up64(off + static_cast<uint64_t>(kept) * 4, 256);
    y.cum_off[k] = off;
    off = align_up64(off + static_cast<uint64_t>(L.G + 1) * 4, 1024);
    y.kcodes_off[k] = off;
    off = align_up64(off + static_cast<uint64_t>(y.rows[k]) * y.kernel_row_bytes, 1024);
    y.wcodes_off[k] = 0;
    if (d->int8_copy) {
      y.wcodes_off[k] = off;
      off = align_up64(off + static_cast<uint64_t>(y.rows[k]) * round_up(L.I, kKernelKAlign), 1024);
    }
  }
  // channel-block tables: predictors 0..M-1, then the cluster of all K orders
  for (int m = 0; m <= L.M; ++m) {
    const int nk = (m < L.M) ? bo[m] : L.K;
    y.blk_off[m] = 0;
    y.blk_cap[m] = 0;
    y.rec_off[m] = 0;
    y.rec_cap[m] = 0;
    if (nk > 8 || static_cast<int64_t>(nk) * L.g > PIPE_BLOCK_ROWS) continue;
    y.blk_cap[m] = L.G;   // a block holds at least one group
    y.blk_off[m] = off;
    off = align_up64(off + static_cast<uint64_t>(y.blk_cap[m] + 2) * 4, 256);
    int64_t R = 0;
    for (int k = (m < L.M ? L.branch_begin[m] : 0); k < (m < L.M ? L.branch_begin[m + 1] : L.K); ++k) R += y.rows[k];
    y.rec_cap[m] = block_count_bound(R, L.O, L.G, nk, L.g);
    y.rec_off[m] = off;
    off = align_up64(off + static_cast<uint64_t>(y.rec_cap[m]) * kRecBytes, 256);
  }
  // decode-unit tables: the clusters that run together share the SMs.  For c CTAs per unit the sets get units in
  // proportion to their rows; a unit's rows (rounded to the MMA's granularity, plus one group of every order of slack)
  // must fit the 256 accumulator columns; the cost of a split is the reduction steps of one CTA times the MMAs of a
  // step, each of which takes its tensor time (N / 2 cycles) but never less than the issue time of an instruction.
  auto plan = [&](int m_begin, int m_end, int32_t* split_out) {
    int64_t Rsum = 0;
    int64_t R[PIPE_MAX_ORDERS + 1];
    int nk[PIPE_MAX_ORDERS + 1];
    bool ok = true;
    for (int m = m_begin; m < m_end; ++m) {
      const int k0 = (m < L.M) ? L.branch_begin[m] : 0, k1 = (m < L.M) ? L.branch_begin[m + 1] : L.K;
      nk[m] = k1 - k0;
      R[m] = 0;
      for (int k = k0; k < k1; ++k) R[m] += (k == 0) ? L.O : static_cast<int64_t>(L.n_keep) * L.g;
      Rsum += R[m];
      if (nk[m] > 8 || static_cast<int64_t>(nk[m]) * L.g > PIPE_BLOCK_ROWS / 2) ok = false;
    }
    *split_out = 0;
    for (int m = m_begin; m < m_end; ++m) y.dec_off[m] = 0, y.dec_limit[m] = 0;
    if (!ok) return;
    const int kblocks = ceil_div(L.I, kKernelKAlign);
    double best = 1e300;
    int best_c = 0;
    int best_limit[PIPE_MAX_ORDERS + 1];
    for (int c = 1; c <= 4 && c <= kblocks; ++c) {
      const int units_total = kPlanSMs / c;
      int limit[PIPE_MAX_ORDERS + 1];
      int max_n = 0;
      for (int m = m_begin; m < m_end; ++m) {
        int64_t units = static_cast<int64_t>(units_total) * R[m] / Rsum;
        if (units < 1) units = 1;
        int64_t n = round_up<int64_t>(ceil_div<int64_t>(R[m], units), 16) + static_cast<int64_t>(nk[m]) * L.g;
        if (n > PIPE_BLOCK_ROWS) n = PIPE_BLOCK_ROWS;   // more units than SMs: the CTAs go round them
        limit[m] = static_cast<int>(n);
        max_n = n > max_n ? static_cast<int>(n) : max_n;
      }
      const double per_mma = max_n / 2.0 > 86.0 ? max_n / 2.0 : 86.0;
      int64_t waves = 0;   // units beyond one per CTA cost whole extra rounds
      for (int m = m_begin; m < m_end; ++m) waves += ceil_div<int64_t>(R[m], limit[m] - nk[m] * L.g);
      const double rounds = static_cast<double>(ceil_div<int64_t>(waves, units_total));
      const double cost = rounds * ceil_div(kblocks, c) * 4.0 * per_mma + (c > 1 ? 3000.0 : 0.0);
      if (cost < best) {
        best = cost;
        best_c = c;
        for (int m = m_begin; m < m_end; ++m) best_limit[m] = limit[m];
      }
    }
    *split_out = best_c;
    for (int m = m_begin; m < m_end; ++m) {
      y.dec_limit[m] = best_limit[m];
      y.dec_off[m] = off;
      off = align_up64(off + static_cast<uint64_t>(L.G + 2) * 4, 256);
    }
  };
  plan(0, L.M, &y.decode_split);
  plan(L.M, L.M + 1, &y.decode_split_all);
  if (total > INT32_MAX) return PIPE_ERR_SHAPE;
  y.total_rows = static_cast<int32_t>(total);
  y.blob_bytes = off;
  // expansion workspace: residual [O, I4] float + absmax [O] + group score [G] (double) + keep flag [G]
  // (+ the rows' sums of squares [O] double for the L2 score)
  const uint64_t I4 = round_up(L.I, 4);
  y.expand_ws_bytes = align_up64(static_cast<uint64_t>(L.O) * I4 * 4, 256) + align_up64(static_cast<uint64_t>(L.O) * 4, 256) +
                      align_up64(static_cast<uint64_t>(L.G) * 8, 256) + align_up64(static_cast<uint64_t>(L.G) * 4, 256) +
                      (L.score_mode == PIPE_SCORE_L2 ? align_up64(static_cast<uint64_t>(L.O) * 8, 256) : 0) +
                      (L.keep_elems > 0 ? 2 * align_up64(static_cast<uint64_t>(L.O) * 4, 256) : 0);
  y.quantize_ws_bytes = 256;
  *out = L;
  return PIPE_OK;
}

}  // namespace pipe

using namespace pipe;

extern "C" {

int32_t pipe_keep_groups_from_gamma(int32_t num_groups, double gamma) {
  if (num_groups < 1) return 0;
  double v = std::ceil(gamma * static_cast<double>(num_groups) - 1e-9);
  if (!(v >= 1.0)) v = 1.0;
  if (v > static_cast<double>(num_groups)) v = static_cast<double>(num_groups);
  return static_cast<int32_t>(v);
}

pipe_status pipe_default_branches(int32_t K, int32_t M, int32_t* h_out) {
  if (!h_out || K < 1 || K > PIPE_MAX_ORDERS) return PIPE_ERR_INVALID_ARG;
  if (M < 1 || M > K) return PIPE_ERR_SHAPE;
  for (int m = 0; m < M; ++m) h_out[m] = K / M + (m < K % M ? 1 : 0);
  return PIPE_OK;
}

static bool shape_ok(const pipe_op_shape* sh) {
  return sh && sh->kernel_size >= 1 && sh->feature_size >= 1 && sh->in_channels >= 1 && sh->out_channels >= 1 && sh->stride >= 1;
}
// products per output position summed over the layer: D^2 d^2 n_i n_o / s^2
static double products_of(const pipe_op_shape* sh) {
  const double D = sh->feature_size, d = sh->kernel_size, s = sh->stride;
  return D * D * d * d * static_cast<double>(sh->in_channels) * static_cast<double>(sh->out_channels) / (s * s);
}
static double digit_cost(int bits) { return static_cast<double>(bits) * std::log2(static_cast<double>(bits)); }

double pipe_bit_ops_original(const pipe_op_shape* shape) {
  if (!shape_ok(shape)) return -1.0;
  return products_of(shape) * digit_cost(32);
}

double pipe_bit_ops_expanded(const pipe_op_shape* shape, int32_t weight_bits, double orders) {
  if (!shape_ok(shape) || weight_bits < 2 || weight_bits > 32 || !(orders >= 0.0)) return -1.0;
  const double D = shape->feature_size, s = shape->stride;
  const double rescale = D * D * (static_cast<double>(shape->in_channels) + static_cast<double>(shape->out_channels) / (s * s)) * digit_cost(32);
  return rescale + orders * products_of(shape) * digit_cost(weight_bits);
}

int32_t pipe_max_orders_within_original(const pipe_op_shape* shape, int32_t weight_bits) {
  if (!shape_ok(shape) || weight_bits < 2 || weight_bits > 32) return -1;
  const double budget = pipe_bit_ops_original(shape);
  int32_t k = 0;
  while (k < (1 << 20) && pipe_bit_ops_expanded(shape, weight_bits, static_cast<double>(k + 1)) <= budget) ++k;
  return k;
}

pipe_status pipe_gamma_from_budget(double beta, int32_t K, double* h_gamma) {
  if (!h_gamma || K < 1 || K > PIPE_MAX_ORDERS || !(beta >= 1.0) || beta > static_cast<double>(K)) return PIPE_ERR_INVALID_ARG;
  *h_gamma = K == 1 ? 1.0 : (beta - 1.0) / static_cast<double>(K - 1);
  return PIPE_OK;
}

double pipe_bound_network(const double* h_s, const double* h_u, int32_t L) {
  if (!h_s || !h_u || L < 1) return -1.0;
  double prod = 1.0, sum = 0.0;
  for (int l = 0; l < L; ++l) {
    if (!(h_s[l] >= 0.0) || !(h_u[l] >= 0.0)) return -1.0;
    sum += h_s[l] * h_u[l];
    prod *= sum + 1.0;
  }
  return prod - 1.0;
}

double pipe_bound_step_dense(int32_t weight_bits, int32_t K, double first_scale_max) {
  if (weight_bits < 2 || weight_bits > 8 || K < 1 || K > PIPE_MAX_ORDERS || !(first_scale_max >= 0.0)) return -1.0;
  const double qmax = static_cast<double>((1 << (weight_bits - 1)) - 1);
  return std::pow(1.0 / qmax, K - 1) * first_scale_max / 2.0;
}

double pipe_bound_step_rows(const float* h_last_scale, int32_t O) {
  if (!h_last_scale || O < 1) return -1.0;
  double m = 0.0;
  for (int o = 0; o < O; ++o) {
    const double v = static_cast<double>(h_last_scale[o]);
    if (!(v >= 0.0)) return -1.0;
    if (v > m) m = v;
  }
  return m / 2.0;
}

pipe_status pipe_spectral_norm(const float* h_W, int32_t O, int32_t I, int64_t ldw, int32_t max_iters, double tol, double* h_sigma) {
  if (!h_W || !h_sigma || O < 1 || I < 1 || ldw < I || max_iters < 1 || !(tol >= 0.0)) return PIPE_ERR_INVALID_ARG;
  double* v = new double[I];
  double* w = new double[O];
  for (int i = 0; i < I; ++i) v[i] = 1.0 / std::sqrt(static_cast<double>(I));
  double sigma = 0.0;
  for (int it = 0; it < max_iters; ++it) {
    double nw = 0.0;
    for (int o = 0; o < O; ++o) {   // w = W v
      const float* row = h_W + static_cast<int64_t>(o) * ldw;
      double s = 0.0;
      for (int i = 0; i < I; ++i) s += static_cast<double>(row[i]) * v[i];
      w[o] = s;
      nw += s * s;
    }
    const double est = std::sqrt(nw);   // |W v| with |v| = 1
    for (int i = 0; i < I; ++i) v[i] = 0.0;
    for (int o = 0; o < O; ++o) {   // v = W^T w
      const float* row = h_W + static_cast<int64_t>(o) * ldw;
      for (int i = 0; i < I; ++i) v[i] += static_cast<double>(row[i]) * w[o];
    }
    double nv = 0.0;
    for (int i = 0; i < I; ++i) nv += v[i] * v[i];
    nv = std::sqrt(nv);
    const bool done = nv == 0.0 || std::fabs(est - sigma) <= tol * est;
    sigma = est;
    if (nv == 0.0) break;
    for (int i = 0; i < I; ++i) v[i] /= nv;
    if (done && it > 0) break;
  }
  *h_sigma = sigma;
  delete[] v;
  delete[] w;
  return PIPE_OK;
}

pipe_status pipe_choose_expansion(const pipe_op_shape* shape, int32_t weight_bits, double bit_ops_budget, int32_t max_orders,
                                  double min_gamma, int32_t num_branches, int32_t* h_K, double* h_gamma, int32_t* h_M,
                                  int32_t* h_branch_orders) {
  if (!shape_ok(shape) || !h_K || !h_gamma || !h_M || !h_branch_orders) return PIPE_ERR_INVALID_ARG;
  if (weight_bits < 2 || weight_bits > 8 || max_orders < 1 || max_orders > PIPE_MAX_ORDERS || num_branches < 1) return PIPE_ERR_INVALID_ARG;
  if (!(min_gamma > 0.0) || min_gamma > 1.0 || !(bit_ops_budget > 0.0)) return PIPE_ERR_INVALID_ARG;
  const double rescale = pipe_bit_ops_expanded(shape, weight_bits, 0.0);
  const double one_order = pipe_bit_ops_expanded(shape, weight_bits, 1.0) - rescale;
  double beta = (bit_ops_budget - rescale) / one_order;
  if (!(beta >= 1.0)) return PIPE_ERR_INVALID_ARG;
  if (beta > static_cast<double>(max_orders)) beta = static_cast<double>(max_orders);
  int K = 1 + static_cast<int>(std::floor((beta - 1.0) / min_gamma + 1e-9));
  if (K > max_orders) K = max_orders;
  if (K < 1) K = 1;
  double gamma = K == 1 ? 1.0 : (beta - 1.0) / static_cast<double>(K - 1);
  if (gamma > 1.0) gamma = 1.0;
  *h_K = K;
  *h_gamma = gamma;
  const int M = num_branches < K ? num_branches : K;
  *h_M = M;
  for (int m = 0; m < PIPE_MAX_ORDERS; ++m) h_branch_orders[m] = 0;
  return pipe_default_branches(K, M, h_branch_orders);
}

pipe_status pipe_layout(const pipe_layer_desc* desc, pipe_layer_layout* h_out) {
  if (!h_out) return PIPE_ERR_INVALID_ARG;
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  *h_out = L.lay;
  return PIPE_OK;
}

pipe_status pipe_diag_select_kernel(int32_t which) {
  if (which < 0 || which > 5) return PIPE_ERR_INVALID_ARG;
  g_kernel_choice.store(which);
  return PIPE_OK;
}

uint64_t pipe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

pipe_status pipe_poll_status(void* stream, int32_t* h_status) {
  if (!h_status) return PIPE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int* word = device_status_word();
  if (!word) return PIPE_ERR_CUDA;
  int v = 0;
  if (cudaMemcpyAsync(&v, word, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return PIPE_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PIPE_ERR_CUDA;
  if (v != 0 && cudaMemsetAsync(word, 0, sizeof(int), s) != cudaSuccess) return PIPE_ERR_CUDA;
  if (v != 0 && cudaStreamSynchronize(s) != cudaSuccess) return PIPE_ERR_CUDA;
  *h_status = v;
  return PIPE_OK;
}

const char* pipe_status_string(pipe_status s) {
  switch (s) {
    case PIPE_OK: return "ok";
    case PIPE_ERR_INVALID_ARG: return "invalid argument";
    case PIPE_ERR_SHAPE: return "inconsistent shape";
    case PIPE_ERR_ALIGNMENT: return "misaligned pointer or pitch";
    case PIPE_ERR_UNSUPPORTED: return "unsupported request";
    case PIPE_ERR_WORKSPACE: return "blob or workspace too small";
    case PIPE_ERR_NONFINITE: return "non-finite value in weights or activations";
    case PIPE_ERR_ACC_OVERFLOW: return "int32 partial sum could overflow";
    case PIPE_ERR_TIMEOUT: return "bounded device wait expired";
    case PIPE_ERR_CUDA: return "CUDA call failed";
  }
  return "unknown status";
}

}  // extern "C"
