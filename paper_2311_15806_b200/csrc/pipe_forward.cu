// pipe_expanded_linear / pipe_ensemble_forward: argument checks and kernel selection.
#include "pipe_common.cuh"

namespace pipe {

// Channel-block table m of the blob (m < L.M: predictor m; m = L.M: all K orders), or nullptr.
static const int32_t* block_table(const LayerInfo& L, const void* d_blob, int m) {
  return L.lay.blk_off[m] ? reinterpret_cast<const int32_t*>(static_cast<const uint8_t*>(d_blob) + L.lay.blk_off[m]) : nullptr;
}

static pipe_status dispatch_forward(const ForwardArgs& a, const LayerInfo& L, int M, int64_t T, const int32_t* const* zp,
                                    cudaStream_t stream);

static pipe_status run_forward(const LayerInfo& L, const void* d_blob, int M, const int8_t* const* xq,
                               const float* const* sx, float* const* y, const int* k_begin, const int* k_end,
                               int64_t T, int64_t ldxq, int64_t ldy, const float* d_bias, int sum_branches,
                               int32_t* d_partials, cudaStream_t stream, int8_t* const* yq = nullptr,
                               const float* const* out_scale = nullptr, int64_t ldyq = 0, int relu = 0,
                               const int32_t* const* zp = nullptr) {
  // yq != nullptr: the fused inner-layer epilogue; y and ldy are unused then
  const bool q8 = yq != nullptr;
  if (!d_blob || relu < 0 || relu > 4) return PIPE_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(d_blob) & (PIPE_BLOB_ALIGN - 1)) return PIPE_ERR_ALIGNMENT;
  if (T < 0 || ldxq < L.I) return PIPE_ERR_INVALID_ARG;
  if (q8 ? (ldyq < L.O || !out_scale || sum_branches) : (ldy < L.O)) return PIPE_ERR_INVALID_ARG;
  for (int m = 0; m < M; ++m) {
    if (!sx[m]) return PIPE_ERR_INVALID_ARG;
    if (T > 0 && !xq[m]) return PIPE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(sx[m]) & 3) return PIPE_ERR_ALIGNMENT;
    if (q8) {
      if (!out_scale[m] || (T > 0 && !yq[m])) return PIPE_ERR_INVALID_ARG;
      if (reinterpret_cast<uintptr_t>(out_scale[m]) & 3) return PIPE_ERR_ALIGNMENT;
      continue;
    }
    if (T > 0 && (m == 0 || !sum_branches) && !y[m]) return PIPE_ERR_INVALID_ARG;
    if ((m == 0 || !sum_branches) && (reinterpret_cast<uintptr_t>(y[m]) & 3)) return PIPE_ERR_ALIGNMENT;
  }
  if ((reinterpret_cast<uintptr_t>(d_bias) & 3) || (reinterpret_cast<uintptr_t>(d_partials) & 3)) return PIPE_ERR_ALIGNMENT;
  if (T == 0) return PIPE_OK;

  ForwardArgs a;
  for (int k = 0; k < L.K; ++k) a.order[k] = order_view(L, d_blob, k);
  a.num_branches = M;
  for (int m = 0; m < M; ++m) {
    BranchArgs& b = a.branch[m];
    b.xq = xq[m];
    b.sx = sx[m];
    b.zp = zp ? zp[m] : nullptr;
    b.y = q8 ? nullptr : (sum_branches ? y[0] : y[m]);
    b.yq = q8 ? yq[m] : nullptr;
    b.out_scale = q8 ? out_scale[m] : nullptr;
    b.k_begin = k_begin[m];
    b.k_end = k_end[m];
    b.add_bias = (m == 0);
    b.accumulate = (sum_branches && m > 0);
    // one branch running all K orders is the "all orders" cluster (entry L.M), otherwise predictor m's own
    const int set = (k_end[m] - k_begin[m] == L.K) ? L.M : m;
    b.blk = block_table(L, d_blob, set);
    b.rec = L.lay.rec_off[set] ? static_cast<const uint8_t*>(d_blob) + L.lay.rec_off[set] : nullptr;
    b.dec = L.lay.dec_off[set] ? reinterpret_cast<const int32_t*>(static_cast<const uint8_t*>(d_blob) + L.lay.dec_off[set]) : nullptr;
  }
  a.decode_split = (M == 1 && k_end[0] - k_begin[0] == L.K) ? L.lay.decode_split_all : L.lay.decode_split;
  a.sum_blk = nullptr;
  a.sum_rec = nullptr;
  if (sum_branches && M > 1 && L.lay.rec_off[L.M]) {
    a.sum_blk = block_table(L, d_blob, L.M);
    a.sum_rec = static_cast<const uint8_t*>(d_blob) + L.lay.rec_off[L.M];
  }
  a.blob_settled = expansion_marked(stream) ? 0 : 1;   // (the mark is cleared once this call has queued a kernel)
  a.O = L.O; a.I = L.I; a.bits = L.bits; a.g = L.g; a.G = L.G;
  a.T = T; a.ldxq = ldxq; a.ldy = ldy;
  a.bias = d_bias;
  a.partials = d_partials;
  a.total_rows = L.lay.total_rows;
  a.kernel_row_bytes = L.lay.kernel_row_bytes;
  a.canon_row_bytes = L.lay.canon_row_bytes;
  a.status = device_status_word();
  if (!a.status) return PIPE_ERR_CUDA;
  a.conv_on = 0;
  a.cN = a.cH = a.cW = a.cC = a.ckh = a.ckw = a.cph = a.cpw = 0;
  a.cHo = a.cWo = 0; a.csh = a.csw = 1;
  a.q8_out = q8 ? 1 : 0;
  a.relu = relu;
  a.ldyq = ldyq;

  const pipe_status st = dispatch_forward(a, L, M, T, zp, stream);
  if (st == PIPE_OK && T > 0) take_expansion_mark(stream);   // this call's kernels now stand behind the expansion
  return st;
}

static pipe_status dispatch_forward(const ForwardArgs& a, const LayerInfo& L, int M, int64_t T, const int32_t* const* zp,
                                    cudaStream_t stream) {
  const int choice = kernel_choice();
  if (zp) {   // asymmetric codes: the CUDA-core kernel folds the zero point in (the others decline)
    if (static_cast<int64_t>(255) * L.qmax * L.I >= (static_cast<int64_t>(1) << 31)) return PIPE_ERR_ACC_OVERFLOW;
    for (int m = 0; m < M; ++m)
      if (reinterpret_cast<uintptr_t>(zp[m]) & 3) return PIPE_ERR_ALIGNMENT;
    return (choice == 0 || choice == 1) ? forward_reference(a, stream) : PIPE_ERR_UNSUPPORTED;
  }
  if (choice == 1) return forward_reference(a, stream);
  if (choice == 2) return forward_tcgen05(a, stream);
  if (choice == 3) return forward_stream(a, stream);
  if (choice == 4) return forward_tcgen05_pair(a, stream);
  if (choice == 5) return forward_decode_tc(a, stream);
  // T <= 16: weight streaming; from two token tiles on the SM-pair kernel; the one-SM kernel for what lies between
  // and for layers without channel-block tables; the CUDA-core kernel for every other shape
  pipe_status st = PIPE_ERR_UNSUPPORTED;
  // (the small-token tcgen05 kernel, choice 5, is measured slower than the weight-streaming kernel -- widening the
  // codes through shared memory for the tensor core triples the shared-memory traffic per weight byte -- and is
  // therefore not on the automatic path)
  if (T <= 16) st = forward_stream(a, stream);
  if (T <= 16 && st == PIPE_ERR_UNSUPPORTED) st = forward_decode_tc(a, stream);
  if (st == PIPE_ERR_UNSUPPORTED) st = forward_tcgen05_pair(a, stream);
  if (st == PIPE_ERR_UNSUPPORTED) st = forward_tcgen05(a, stream);
  if (st == PIPE_ERR_UNSUPPORTED) st = forward_reference(a, stream);
  return st;
}

}  // namespace pipe

using namespace pipe;

extern "C" pipe_status pipe_expanded_linear(const pipe_layer_desc* desc, const void* d_blob, const int8_t* d_xq, int64_t T,
                                            int64_t ldxq, const float* d_sx, const float* d_bias, float* d_y, int64_t ldy,
                                            int32_t* d_partials, void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  const int kb = 0, ke = L.K;
  return run_forward(L, d_blob, 1, &d_xq, &d_sx, &d_y, &kb, &ke, T, ldxq, ldy, d_bias, 0, d_partials,
                     static_cast<cudaStream_t>(stream));
}

extern "C" pipe_status pipe_ensemble_forward(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                             int64_t T, int64_t ldxq, const float* const* h_sx_m, const float* d_bias,
                                             float* const* h_y_m, int64_t ldy, int32_t sum_branches, int32_t* d_partials,
                                             void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  if (!h_xq_m || !h_sx_m || !h_y_m) return PIPE_ERR_INVALID_ARG;
  int kb[PIPE_MAX_ORDERS], ke[PIPE_MAX_ORDERS];
  for (int m = 0; m < L.M; ++m) {
    kb[m] = L.branch_begin[m];
    ke[m] = L.branch_begin[m + 1];
  }
  return run_forward(L, d_blob, L.M, h_xq_m, h_sx_m, h_y_m, kb, ke, T, ldxq, ldy, d_bias, sum_branches ? 1 : 0,
                     d_partials, static_cast<cudaStream_t>(stream));
}

extern "C" pipe_status pipe_ensemble_forward_zp(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                                int64_t T, int64_t ldxq, const float* const* h_sx_m,
                                                const int32_t* const* h_zp_m, const float* d_bias, float* const* h_y_m,
                                                int64_t ldy, int32_t sum_branches, int32_t* d_partials, void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  if (!h_xq_m || !h_sx_m || !h_zp_m || !h_y_m) return PIPE_ERR_INVALID_ARG;
  int kb[PIPE_MAX_ORDERS], ke[PIPE_MAX_ORDERS];
  for (int m = 0; m < L.M; ++m) {
    kb[m] = L.branch_begin[m];
    ke[m] = L.branch_begin[m + 1];
  }
  return run_forward(L, d_blob, L.M, h_xq_m, h_sx_m, h_y_m, kb, ke, T, ldxq, ldy, d_bias, sum_branches ? 1 : 0,
                     d_partials, static_cast<cudaStream_t>(stream), nullptr, nullptr, 0, 0, h_zp_m);
}

extern "C" pipe_status pipe_ensemble_forward_q8(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                                int64_t T, int64_t ldxq, const float* const* h_sx_m, const float* d_bias,
                                                int32_t relu, const float* const* h_out_scale_m, int8_t* const* h_yq_m,
                                                int64_t ldyq, int32_t* d_partials, void* stream) {
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  if (!h_xq_m || !h_sx_m || !h_out_scale_m || !h_yq_m) return PIPE_ERR_INVALID_ARG;
  int kb[PIPE_MAX_ORDERS], ke[PIPE_MAX_ORDERS];
  for (int m = 0; m < L.M; ++m) {
    kb[m] = L.branch_begin[m];
    ke[m] = L.branch_begin[m + 1];
  }
  return run_forward(L, d_blob, L.M, h_xq_m, h_sx_m, nullptr, kb, ke, T, ldxq, 0, d_bias, 0, d_partials,
                     static_cast<cudaStream_t>(stream), h_yq_m, h_out_scale_m, ldyq, relu);
}

// All convolution entries.  M inputs with their clusters of orders [k_begin[m], k_end[m]) (one input with all K orders
// for pipe_expanded_conv2d); yq != nullptr selects the fused inner-layer epilogue (y, ldy unused then).
static pipe_status run_conv(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob, int M, bool all_orders,
                            const int8_t* const* xq, const float* const* sx, const float* d_bias, float* const* y,
                            int64_t ldy, int sum_branches, int8_t* const* yq, const float* const* out_scale, int64_t ldyq,
                            int relu, int32_t* d_partials, void* stream) {
  const bool q8 = yq != nullptr;
  if (relu < 0 || relu > 4) return PIPE_ERR_INVALID_ARG;
  LayerInfo L;
  pipe_status st = resolve_layer(desc, &L);
  if (st != PIPE_OK) return st;
  if (!all_orders) M = L.M;
  if (!geom || !d_blob || !xq || !sx || (!q8 && !y) || (q8 && (!out_scale || sum_branches))) return PIPE_ERR_INVALID_ARG;
  if (geom->batch < 1 || geom->height < 1 || geom->width < 1 || geom->channels < 1 || geom->kernel_h < 1 ||
      geom->kernel_w < 1)
    return PIPE_ERR_INVALID_ARG;
  const int sh = geom->stride_h > 0 ? geom->stride_h : 1, sw = geom->stride_w > 0 ? geom->stride_w : 1;
  if (geom->stride_h < 0 || geom->stride_w < 0 || geom->pad_h < 0 || geom->pad_w < 0) return PIPE_ERR_INVALID_ARG;
  if (geom->pad_h >= geom->kernel_h || geom->pad_w >= geom->kernel_w) return PIPE_ERR_SHAPE;
  if (geom->height + 2 * geom->pad_h < geom->kernel_h || geom->width + 2 * geom->pad_w < geom->kernel_w) return PIPE_ERR_SHAPE;
  const int Ho = (geom->height + 2 * geom->pad_h - geom->kernel_h) / sh + 1;
  const int Wo = (geom->width + 2 * geom->pad_w - geom->kernel_w) / sw + 1;
  if (static_cast<int64_t>(geom->kernel_h) * geom->kernel_w * geom->channels != L.I) return PIPE_ERR_SHAPE;
  if ((q8 ? ldyq : ldy) < L.O) return PIPE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_blob) & (PIPE_BLOB_ALIGN - 1)) || (reinterpret_cast<uintptr_t>(d_bias) & 3) ||
      (reinterpret_cast<uintptr_t>(d_partials) & 3))
    return PIPE_ERR_ALIGNMENT;
  for (int m = 0; m < M; ++m) {
    if (!xq[m] || !sx[m]) return PIPE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(xq[m]) & 15) || (reinterpret_cast<uintptr_t>(sx[m]) & 3)) return PIPE_ERR_ALIGNMENT;
    if (q8) {
      if (!yq[m] || !out_scale[m]) return PIPE_ERR_INVALID_ARG;
      if (reinterpret_cast<uintptr_t>(out_scale[m]) & 3) return PIPE_ERR_ALIGNMENT;
    } else if (m == 0 || !sum_branches) {
      if (!y[m]) return PIPE_ERR_INVALID_ARG;
      if (reinterpret_cast<uintptr_t>(y[m]) & 3) return PIPE_ERR_ALIGNMENT;
    }
  }
  if (geom->channels % 128 != 0 || sh > 8 || sw > 8) return PIPE_ERR_UNSUPPORTED;

  ForwardArgs a;
  for (int k = 0; k < L.K; ++k) a.order[k] = order_view(L, d_blob, k);
  a.num_branches = M;
  for (int m = 0; m < M; ++m) {
    BranchArgs& b = a.branch[m];
    b.xq = xq[m];
    b.sx = sx[m];
    b.zp = nullptr;
    b.y = q8 ? nullptr : (sum_branches ? y[0] : y[m]);
    b.k_begin = all_orders ? 0 : L.branch_begin[m];
    b.k_end = all_orders ? L.K : L.branch_begin[m + 1];
    b.add_bias = (m == 0);
    b.accumulate = (sum_branches && m > 0);
    // one input running all K orders is the "all orders" cluster (entry L.M), otherwise predictor m's own
    const int set = (b.k_end - b.k_begin == L.K) ? L.M : m;
    b.blk = block_table(L, d_blob, set);
    b.rec = L.lay.rec_off[set] ? static_cast<const uint8_t*>(d_blob) + L.lay.rec_off[set] : nullptr;
    b.dec = nullptr;
    b.yq = q8 ? yq[m] : nullptr;
    b.out_scale = q8 ? out_scale[m] : nullptr;
  }
  a.decode_split = 0;
  a.sum_blk = nullptr;
  a.sum_rec = nullptr;
  if (sum_branches && M > 1 && !all_orders && L.lay.rec_off[L.M]) {
    a.sum_blk = block_table(L, d_blob, L.M);
    a.sum_rec = static_cast<const uint8_t*>(d_blob) + L.lay.rec_off[L.M];
  }
  a.blob_settled = expansion_marked(static_cast<cudaStream_t>(stream)) ? 0 : 1;
  a.q8_out = q8 ? 1 : 0;
  a.relu = relu;
  a.ldyq = ldyq;
  a.O = L.O; a.I = L.I; a.bits = L.bits; a.g = L.g; a.G = L.G;
  a.T = static_cast<int64_t>(geom->batch) * Ho * Wo;
  a.ldxq = geom->channels;
  a.ldy = ldy;
  a.bias = d_bias;
  a.partials = d_partials;
  a.total_rows = L.lay.total_rows;
  a.kernel_row_bytes = L.lay.kernel_row_bytes;
  a.canon_row_bytes = L.lay.canon_row_bytes;
  a.status = device_status_word();
  if (!a.status) return PIPE_ERR_CUDA;
  a.conv_on = 1;
  a.cN = geom->batch; a.cH = geom->height; a.cW = geom->width; a.cC = geom->channels;
  a.ckh = geom->kernel_h; a.ckw = geom->kernel_w; a.cph = geom->pad_h; a.cpw = geom->pad_w;
  a.cHo = Ho; a.cWo = Wo; a.csh = sh; a.csw = sw;
  const int choice = kernel_choice();
  pipe_status cst;
  if (choice == 4) cst = forward_tcgen05_pair(a, static_cast<cudaStream_t>(stream));
  else if (choice == 2) cst = forward_tcgen05(a, static_cast<cudaStream_t>(stream));
  else {
    cst = forward_tcgen05_pair(a, static_cast<cudaStream_t>(stream));
    if (cst == PIPE_ERR_UNSUPPORTED) cst = forward_tcgen05(a, static_cast<cudaStream_t>(stream));
  }
  if (cst == PIPE_OK && a.T > 0) take_expansion_mark(static_cast<cudaStream_t>(stream));
  return cst;
}

extern "C" pipe_status pipe_expanded_conv2d(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                            const int8_t* d_xq, const float* d_sx, const float* d_bias, float* d_y,
                                            int64_t ldy, int32_t* d_partials, void* stream) {
  if (!d_xq || !d_sx || !d_y) return PIPE_ERR_INVALID_ARG;
  return run_conv(desc, geom, d_blob, 1, true, &d_xq, &d_sx, d_bias, &d_y, ldy, 0, nullptr, nullptr, 0, 0, d_partials, stream);
}

extern "C" pipe_status pipe_expanded_conv2d_q8(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                               const int8_t* d_xq, const float* d_sx, const float* d_bias, int32_t relu,
                                               const float* d_out_scale, int8_t* d_yq, int64_t ldyq, int32_t* d_partials,
                                               void* stream) {
  if (!d_xq || !d_sx || !d_yq || !d_out_scale) return PIPE_ERR_INVALID_ARG;
  return run_conv(desc, geom, d_blob, 1, true, &d_xq, &d_sx, d_bias, nullptr, 0, 0, &d_yq, &d_out_scale, ldyq, relu, d_partials, stream);
}

extern "C" pipe_status pipe_ensemble_conv2d(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                            const int8_t* const* h_xq_m, const float* const* h_sx_m, const float* d_bias,
                                            float* const* h_y_m, int64_t ldy, int32_t sum_branches, int32_t* d_partials,
                                            void* stream) {
  if (!h_xq_m || !h_sx_m || !h_y_m) return PIPE_ERR_INVALID_ARG;
  return run_conv(desc, geom, d_blob, 0, false, h_xq_m, h_sx_m, d_bias, h_y_m, ldy, sum_branches ? 1 : 0, nullptr, nullptr, 0, 0,
                  d_partials, stream);
}

extern "C" pipe_status pipe_ensemble_conv2d_q8(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                               const int8_t* const* h_xq_m, const float* const* h_sx_m, const float* d_bias,
                                               int32_t relu, const float* const* h_out_scale_m, int8_t* const* h_yq_m,
                                               int64_t ldyq, int32_t* d_partials, void* stream) {
  if (!h_xq_m || !h_sx_m || !h_out_scale_m || !h_yq_m) return PIPE_ERR_INVALID_ARG;
  return run_conv(desc, geom, d_blob, 0, false, h_xq_m, h_sx_m, d_bias, nullptr, 0, 0, h_yq_m, h_out_scale_m, ldyq, relu, d_partials,
                  stream);
}
