/*
 * pipe.h -- C ABI of libpipe: the residual-expanded quantized layer of PIPE
 * (arXiv 2311.15806) on one NVIDIA B200 (sm_100a).
 *
 * Conventions that hold for every call unless its comment says otherwise
 *   - pointers named d_* are DEVICE pointers, h_* are HOST pointers; both are owned by the
 *     caller.  The library never allocates, frees or keeps device memory; it only queues
 *     stream-ordered work on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and returns.  Buffers must stay valid until that work has run.
 *   - matrices are row-major with the last dimension contiguous; ld* are row pitches in
 *     ELEMENTS.
 *   - every function returns a pipe_status.  Problems the host can see (null pointers, bad
 *     shapes, undersized buffers, unsupported combinations) are reported immediately and no
 *     work is queued.  Problems only the device can see (a NaN/Inf among the weights or
 *     activations, a bounded wait inside a kernel running out) set a device status word that
 *     pipe_poll_status reads; the outputs of that call are then unspecified but every access
 *     stayed in bounds.  Nothing throws, aborts, traps or prints.
 *   - there is no CPU fallback: without a CUDA device every compute call returns
 *     PIPE_ERR_CUDA.
 *   - the forward kernels are launched with programmatic stream serialization: their prologue
 *     may overlap the tail of the preceding launch on `stream`, and the weight-streaming kernel
 *     (at most 16 tokens) starts copying the blob's packed codes during that overlap.  The
 *     library orders this correctly against its own calls (a forward call that directly follows
 *     pipe_expand_weights* on the same stream waits for it in full).  A caller that writes
 *     d_blob by other means must let that work complete -- an event, a synchronize, or any other
 *     library call in between -- before queueing a forward call on the same stream.  Inputs
 *     other than d_blob (activations, scales, bias, outputs) are only touched after the
 *     preceding launch has completed, whoever queued it.
 */
#ifndef PIPE_H_
#define PIPE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PIPE_MAX_ORDERS 16
#define PIPE_BLOB_ALIGN 1024 /* d_blob must be aligned to this many bytes */

typedef enum {
  PIPE_OK = 0,
  PIPE_ERR_INVALID_ARG = 1,  /* null pointer, negative size, value out of range */
  PIPE_ERR_SHAPE = 2,        /* group size does not divide out_features, K/M inconsistent, ... */
  PIPE_ERR_ALIGNMENT = 3,    /* pointer or pitch not aligned as documented */
  PIPE_ERR_UNSUPPORTED = 4,  /* valid request the library has no kernel for */
  PIPE_ERR_WORKSPACE = 5,    /* blob / workspace smaller than pipe_layout says */
  PIPE_ERR_NONFINITE = 6,    /* device saw NaN or Inf in weights or activations */
  PIPE_ERR_ACC_OVERFLOW = 7, /* in_features so large that an int32 accumulator could overflow (see pipe_expanded_linear) */
  PIPE_ERR_TIMEOUT = 8,      /* a bounded wait inside a kernel ran out */
  PIPE_ERR_CUDA = 9          /* a CUDA runtime/driver call failed (no device, launch error) */
} pipe_status;

/*
 * One expanded layer.  Sec. 3 "Methodology overview" fixes the quantizer Q (Eq. 1: scale,
 * round to nearest) and the target bit-width b; Sec. 3.1 the expansion order K (Eq. 3) and
 * the structured mask with kept fraction gamma; Sec. 3.2 the grouping [K_1..K_M] of
 * successive orders into M predictors.
 */
typedef struct pipe_layer_desc {
  int32_t out_features;  /* O: rows of W = output channels */
  int32_t in_features;   /* I: reduction length; a multiple of the codes per byte (1, 2, 4) */
  int32_t weight_bits;   /* b: 8, 6, 4, 3 or 2 (2 = ternary {-1,0,+1}; Sec. 4.2 runs int3, int4, int6 and ternary).
                            Codes lie in [-(2^(b-1) - 1), 2^(b-1) - 1]; 3-bit codes are stored in the 4-bit format and
                            6-bit codes in the 8-bit format (every layout below then reads b = 4 resp. b = 8) */
  int32_t num_orders;    /* K, 1..PIPE_MAX_ORDERS */
  int32_t group_size;    /* g: consecutive output channels per sparsity group; divides O */
  int32_t keep_groups;   /* groups kept by every order >= 2, 1..O/g (order 1 is dense) */
  int32_t num_branches;  /* M, 1..K */
  int32_t branch_orders[PIPE_MAX_ORDERS]; /* K_m, sum = K; all zero = balanced default */
  int32_t score_mode;    /* score of the structured mask (Sec. 3.1 names no criterion): PIPE_SCORE_MAXABS = largest
                            magnitude of the current residual over the group's rows; PIPE_SCORE_L2 = its squared
                            Euclidean norm, summed in binary64 in the fixed order given at pipe_expand_weights */
  int32_t keep_elems;    /* 0, or the unstructured mask of Sec. 3.1 for the orders >= 2: in every row only the
                            keep_elems entries of the current residual with the largest magnitude are quantized (ties
                            to the lower index), the others get the code 0 and keep their residual.  Needs
                            keep_groups = G: an unstructured R^k keeps every row */
  int32_t int8_copy;     /* 0 or 1.  1: the blob also holds every order's codes widened to int8 in the operand layout of
                            the tensor-core kernel (wcodes_off below; needs g % 8 == 0).  The kernels for more than 16
                            tokens then copy weight tiles straight into place instead of widening packed codes in
                            shared memory on every use -- the choice for layers evaluated on many tokens at a time, at
                            the price of I_pad more bytes per kept row in HBM.  Results are the same bits either way; the
                            small-token kernels keep streaming the packed codes */
} pipe_layer_desc;

#define PIPE_ACT_IDENTITY 0
#define PIPE_ACT_RELU 1
#define PIPE_ACT_SILU 2
#define PIPE_ACT_GELU 3
#define PIPE_ACT_SIGMOID 4
#define PIPE_SCORE_MAXABS 0
#define PIPE_SCORE_L2 1

/*
 * Byte layout of the expanded-layer blob and the workspace sizes, as computed by
 * pipe_layout.  All offsets are from the start of the blob, so the blob is relocatable:
 * saving or moving an expanded layer is a plain byte copy.
 *
 * For order k (0-based; rows[k] = kept_groups[k] * g rows, compacted in ascending channel
 * order of the kept groups):
 *   codes_off[k]  canonical packed codes, [rows[k], canon_row_bytes] bytes.  Two's complement
 *                 fields, element e of a row at bit offset e*b of the row's little-endian bit
 *                 stream: int4 -> element 2j in bits 0-3 of byte j, 2j+1 in bits 4-7;
 *                 ternary -> element 4j+e in bits 2e..2e+1 of byte j (00 = 0, 01 = +1, 11 = -1).
 *   scales_off[k] float [rows[k]]: lambda_{R^(k)} of each compacted row.
 *   kept_off[k]   int32 [kept_groups[k]]: ascending indices of the kept groups.
 *   cum_off[k]    int32 [G + 1]: cum[j] = number of kept groups with index < j (so group j is
 *                 kept iff cum[j+1] > cum[j], and its first compacted row is cum[j] * g).
 *   kcodes_off[k] the same codes in the layout the GEMM kernels stream: the reduction axis is
 *                 zero-padded to a multiple of 128 codes and cut into blocks of 128 codes; the
 *                 section is [I_pad/128][rows[k]][128*b/8 bytes], i.e. block-major, so that the
 *                 rows a tile needs for one reduction block are one contiguous run of bytes
 *                 (kernel_row_bytes is still the total per row).  Inside every aligned 32-bit
 *                 word the fields are interleaved so that masking alone yields int8 lanes in
 *                 reduction order: int4 -> code 4h+j of the word's 8 codes sits in nibble 2j+h;
 *                 ternary -> code 4h+j of the word's 16 codes sits in bits 8j+2h..8j+2h+1;
 *                 int8 -> unchanged.
 *   wcodes_off[k] (int8_copy only, else 0) the codes as int8, block-major like kcodes_off: [I_pad/128][rows[k]][128]
 *                 bytes, with the 16-byte pieces of a row permuted the way the tensor core's 128-byte swizzle expects
 *                 them in shared memory: piece c (codes 16c .. 16c+15 of the block) of compacted row r is stored as
 *                 piece c ^ (r & 7) of that row.  A run of kept rows of one block is then one contiguous run of bytes
 *                 that lands in an operand tile by a plain bulk copy (kept-row runs start at multiples of g, hence of 8).
 * Channel-block tables, one per cluster of orders that a forward call can evaluate on one input: entry m < M
 * for predictor m (Sec. 3.2), entry M for all K orders (pipe_expanded_linear, pipe_expanded_conv2d).
 *   blk_off[m]    int32 [2 + blk_cap[m]]: n, then b_0 = 0 < b_1 < ... < b_n = G.  Block i is the channel groups
 *                 b_i .. b_{i+1} - 1.  With R the rows the cluster's orders keep in the whole layer and
 *                 n0 = max(ceil(R / PIPE_BLOCK_ROWS), ceil(O / PIPE_BLOCK_CHANNELS)) the fewest blocks that could
 *                 hold them, the limit of a block is L = min(PIPE_BLOCK_ROWS, roundup(ceil(R / n0), 16) + orders * g)
 *                 -- except for a cluster of few blocks: with h = orders * g / 2 and
 *                 ne = max(ceil(R / (PIPE_BLOCK_ROWS - h)), ceil(O / PIPE_BLOCK_CHANNELS)), a cluster with
 *                 ne <= PIPE_EVEN_BLOCKS has L = min(PIPE_BLOCK_ROWS, ceil(R / ne) + h), which gives blocks of one size --:
 *                 the groups are walked from 0 and a block is closed when the next group would take the rows it
 *                 stacks over the cluster's orders (kept groups only) beyond L or its channels beyond
 *                 PIPE_BLOCK_CHANNELS.  Blocks are the unit of work of the SM-pair tensor-core kernel, whose MMAs then
 *                 run close to their widest shape, and evenly, however sparse the orders are.  A cluster of more
 *                 than 8 orders, or whose single group can exceed the row limit (orders * g > PIPE_BLOCK_ROWS), has
 *                 no table.
 *   rec_off[m]    one record of PIPE_BLOCK_RECORD_BYTES per block of table m (room for rec_cap[m] records, a bound on
 *                 the block count that follows from the cut), everything the epilogue of a tile of that block needs,
 *                 so that a kernel fetches it with one bulk copy instead of walking the prefix counts:
 *                   int32 [32]   c0, c1 (the block's channels [c0, c1)), orders of the cluster, stacked rows n, 4 x 0,
 *                                rowbase[0..7] (row of order i's first kept row in the stacked block; n beyond the
 *                                cluster's orders), start[0..7] (that row's index in order i's compacted rows), 8 x 0
 *                   int16 [512]  entry 8 c + i: the stacked row of channel c0 + 8 c in order i, or -1 when the
 *                                order has pruned that channel's group (or c, i lie beyond the block / the cluster)
 *                   float [256]  the scale of every stacked row (0 beyond n)
 *   dec_off[m]    the same structure (n, b_0 .. b_n; room for G blocks) with the row limit dec_limit[m]: the units of
 *                 the small-token (T <= 16) tensor-core kernel, which streams every weight once.  There the limit
 *                 is chosen so that the units of the clusters that run together -- the M predictors, or the one
 *                 cluster of all orders -- come to about one per SM (148 on the B200 this library is written for),
 *                 decode_split (decode_split_all) CTAs sharing a unit's reduction axis when whole units would be
 *                 too narrow for the MMA; the plan is a function of the descriptor alone.
 */
#define PIPE_BLOCK_ROWS 256
#define PIPE_BLOCK_CHANNELS 512
#define PIPE_EVEN_BLOCKS 8   /* clusters of at most this many blocks are cut into blocks of one size (see blk_off) */
#define PIPE_BLOCK_RECORD_BYTES (32 * 4 + 8 * (PIPE_BLOCK_CHANNELS / 8) * 2 + PIPE_BLOCK_ROWS * 4)
typedef struct pipe_layer_layout {
  int32_t num_groups;        /* G = O / g */
  int32_t total_rows;        /* R_total = sum_k rows[k] = O + (K-1) * keep_groups * g */
  int32_t canon_row_bytes;   /* I * b / 8 */
  int32_t kernel_row_bytes;  /* roundup(I, 128) * b / 8 */
  int32_t rows[PIPE_MAX_ORDERS];
  int32_t kept_groups[PIPE_MAX_ORDERS];
  int32_t branch_orders[PIPE_MAX_ORDERS]; /* the resolved [K_1..K_M] */
  uint64_t codes_off[PIPE_MAX_ORDERS];
  uint64_t kcodes_off[PIPE_MAX_ORDERS];
  uint64_t wcodes_off[PIPE_MAX_ORDERS];  /* int8 operand-layout copy (see above); 0 without int8_copy */
  uint64_t scales_off[PIPE_MAX_ORDERS];
  uint64_t kept_off[PIPE_MAX_ORDERS];
  uint64_t cum_off[PIPE_MAX_ORDERS];
  uint64_t blk_off[PIPE_MAX_ORDERS + 1]; /* channel-block tables (see above); 0 = the cluster has none */
  int32_t blk_cap[PIPE_MAX_ORDERS + 1];  /* blocks each table has room for */
  uint64_t rec_off[PIPE_MAX_ORDERS + 1]; /* block records of table m (see above); 0 = the cluster has no table */
  int32_t rec_cap[PIPE_MAX_ORDERS + 1];  /* records there is room for */
  int32_t decode_split;                  /* CTAs that share one decode unit's reduction axis: predictors' tables */
  uint64_t dec_off[PIPE_MAX_ORDERS + 1]; /* decode-unit tables (see above); 0 = the cluster has none */
  int32_t dec_limit[PIPE_MAX_ORDERS + 1]; /* rows a decode unit of the cluster may stack */
  int32_t decode_split_all;              /* the same for the table of all K orders */
  uint64_t blob_bytes;        /* size d_blob must have */
  uint64_t expand_ws_bytes;   /* size d_ws must have for pipe_expand_weights */
  uint64_t quantize_ws_bytes; /* size d_ws must have for pipe_quantize_act */
} pipe_layer_layout;

/* Sec. 3.1: gamma is the kept fraction of an order's channel groups ("150 %" = K 2, gamma
 * 0.5 in Sec. 4.3).  Returns clamp(ceil(gamma * G - 1e-9), 1, G), evaluated in double. */
int32_t pipe_keep_groups_from_gamma(int32_t num_groups, double gamma);

/* Sec. 3.2 / Appendix A: balanced grouping with the remainder going to the earliest
 * predictors (K_1 largest): K_m = floor(K/M) + (m <= K mod M).  Reproduces the paper's
 * [4,4], [3,3,2], [2,2,2,2] and [2,2].  h_out: M ints. */
pipe_status pipe_default_branches(int32_t num_orders, int32_t num_branches, int32_t* h_out);

/* Appendix H (operation head-count).  A d x d convolution with stride s on D x D x n_i feature maps
 * and n_o outputs; a fully connected layer is d = D = s = 1.  A b-digit multiplication is counted
 * as b*log2(b) bit operations (the appendix leaves the base of the logarithm open; every term
 * carries one, so ratios and the order bound below do not depend on it). */
typedef struct {
  int32_t kernel_size;   /* d */
  int32_t feature_size;  /* D */
  int32_t in_channels;   /* n_i */
  int32_t out_channels;  /* n_o */
  int32_t stride;        /* s */
} pipe_op_shape;

/* O_original = D^2 d^2 n_i n_o / s^2 * 32 log2(32): the fp32 layer.  Returns a negative value for
 * an invalid shape (any field < 1).  Pure host functions, no CUDA call. */
double pipe_bit_ops_original(const pipe_op_shape* shape);

/* O_R(k) = D^2 [ (n_i + n_o / s^2) * 32 log2(32) + k * d^2 n_i n_o / s^2 * b log2(b) ]: the two
 * rescalings plus k int-b products.  `orders` is the number of full orders the layer evaluates;
 * a group-sparse expansion (Sec. 3.1) counts as 1 + (K - 1) * gamma of them, so the argument is a
 * double.  bits in 2..32, orders >= 0; a negative value is returned otherwise. */
double pipe_bit_ops_expanded(const pipe_op_shape* shape, int32_t weight_bits, double orders);

/* The largest whole number of orders whose operation count does not exceed the fp32 layer's: the
 * order bound Appendix H derives from its two counts; 0 when even one order does, -1 for invalid
 * arguments. */
int32_t pipe_max_orders_within_original(const pipe_op_shape* shape, int32_t weight_bits);

/* Sec. 3.1 / 4.3, Appendix A: a budget beta ("150 %" = 1.5, "beta = 7 and order K = 8") is the
 * number of full orders a sparse expansion of K orders costs, beta = 1 + (K - 1) * gamma.  Writes
 * the kept fraction gamma of the orders >= 2.  PIPE_ERR_INVALID_ARG unless 1 <= beta <= K and
 * K >= 1 (K = 1 admits beta = 1 only, gamma = 1). */
pipe_status pipe_gamma_from_budget(double beta, int32_t num_orders, double* h_gamma);

/* Appendix C (upper bound of the error, first theorem): for an L-layer ReLU network with spectral norms s_l and
 * per-layer quantization steps u_l, U = prod_{l=1..L} ( sum_{i=1..l} s_i u_i + 1 ) - 1 bounds
 * max_{|X| = 1} |F(X) - F^(K)(X)|.  h_s, h_u: L doubles each (all >= 0).  Returns a negative value for invalid
 * arguments.  The same expression is U_sparse of the second theorem when u_l are the steps of the sparse expansion. */
double pipe_bound_network(const double* h_s, const double* h_u, int32_t L);

/* u_l^(K) of the first theorem / Lemma B.1 for a dense expansion: (1 / (2^(b-1) - 1))^(K-1) * lambda / 2, lambda the
 * largest first-order scale of the layer's rows (the reading of the lemma's lambda under which it holds).
 * Negative for invalid arguments. */
double pipe_bound_step_dense(int32_t weight_bits, int32_t num_orders, double first_scale_max);

/* u_l of a SPARSE expansion (second theorem; its printed factor refers to a quantity this paper does not define).
 * Reading: round-to-nearest leaves a row within half the step of the LAST order that quantized it, whichever orders
 * pruned it in between, so u_l = max over rows of that step / 2.  h_last_scale: float [O], the scale each output
 * channel had at the last order that kept it (the binding gathers it from a blob). */
double pipe_bound_step_rows(const float* h_last_scale, int32_t O);

/* Largest singular value of a host matrix W [O, I] (pitch ldw) by power iteration on W^T W in binary64, started
 * from the all-ones vector; stops after max_iters rounds or when the estimate changes by less than tol (relative).
 * The s_l of Appendix C.  Pure host function. */
pipe_status pipe_spectral_norm(const float* h_W, int32_t O, int32_t I, int64_t ldw, int32_t max_iters, double tol,
                               double* h_sigma);

/* Sec. 3.1 ("to match a total budget of operations"), Sec. 4.2 and Appendix A ("budget 7 and order 8") with the
 * head-count of Appendix H: picks (K, gamma, [K_m]) for a layer shape, a weight bit-width and a budget of bit
 * operations.  beta = the number of full orders the budget pays for, (budget - rescaling) / (one order's products),
 * capped at max_orders; the paper's best trade-offs use high orders with sparse residuals, so K is the largest
 * order count <= max_orders whose kept fraction gamma = (beta - 1) / (K - 1) stays >= min_gamma (K = 1, gamma = 1
 * when the budget pays for one order only); [K_m] is the balanced split of pipe_default_branches for
 * min(num_branches, K) predictors.  h_branch_orders: PIPE_MAX_ORDERS ints (unused entries zeroed).
 * PIPE_ERR_INVALID_ARG when the budget does not pay for one order or an argument is out of range. */
pipe_status pipe_choose_expansion(const pipe_op_shape* shape, int32_t weight_bits, double bit_ops_budget, int32_t max_orders,
                                  double min_gamma, int32_t num_branches, int32_t* h_num_orders, double* h_gamma,
                                  int32_t* h_num_branches, int32_t* h_branch_orders);

/* Validates `desc` and fills `h_out`.  Pure host function, no CUDA call. */
pipe_status pipe_layout(const pipe_layer_desc* desc, pipe_layer_layout* h_out);

/*
 * Sec. 3.1 "Residual Expansion" (Eq. 2, Eq. 3 and the masked form that follows them), with
 * Q of Eq. 1 per output channel (Sec. 4.1: symmetric, per-channel):
 * for k = 1..K on the running residual r (r = W for k = 1)
 *     a[o] = max_i |r[o,i]|
 *     kept_k = all groups (k = 1, or keep_groups = G), else the keep_groups groups with the
 *              largest max_{o in group} a[o], ties to the lower index, stored ascending
 *     for rows o of kept groups:  s = a[o] / qmax (qmax = 2^(b-1) - 1, IEEE division),
 *              q[o,i] = clamp(rne(r[o,i] / s), -qmax, qmax),  r[o,i] = fma(-s, q[o,i], r[o,i]);
 *              a zero scale gives zero codes and an unchanged residual
 *     rows of pruned groups keep their residual (R^k has a zero row there).
 * d_W: float [O, I], pitch ldw, 4-byte aligned (16-byte aligned rows take the fast path).
 * PIPE_SCORE_L2: the score of group j is sum over its rows o (ascending) of S[o], binary64, where
 *     S[o] = tree(P_0..P_31), P_l = sum over i = l, l+32, ... (ascending) of (double) r[o,i]^2, and the tree adds
 *     P_l += P_{l+off} for off = 16, 8, 4, 2, 1 (a sum of squares depends on the order of its additions in the last
 *     bits, and the kept lists are compared bit for bit, so the order is part of the definition).
 * keep_elems > 0: see pipe_layer_desc.
 * d_blob: blob_bytes bytes aligned to PIPE_BLOB_ALIGN; fully overwritten.
 * d_ws: expand_ws_bytes bytes, 256-byte aligned; contents undefined afterwards.
 * Non-finite weights set PIPE_ERR_NONFINITE in the device status word.
 */
pipe_status pipe_expand_weights(const pipe_layer_desc* desc, const float* d_W, int64_t ldw, void* d_blob,
                                size_t blob_bytes, void* d_ws, size_t ws_bytes, void* stream);

/*
 * pipe_expand_weights for callers that must not allocate device memory.  (The paper has no
 * counterpart to this call; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs after the host application has handed all of the GPU's memory
 * to its own pool or has frozen its memory budget -- an inference-server plug-in re-expanding
 * a layer when new weights are swapped in, say -- and code that must not stall the device:
 * cudaMalloc and cudaFree synchronise the whole GPU, so an allocation on the weight-update path
 * would stop the streams that are serving requests.  Such a caller cannot produce the d_ws
 * buffer that pipe_expand_weights asks for.
 *
 * Here the workspace is a fixed array of PIPE_STATIC_SCRATCH_BYTES inside the library itself
 * (every GPU that loads the library holds that much until the process exits).  The call computes
 * exactly what pipe_expand_weights computes, into the caller's d_blob, and neither it nor
 * anything it calls allocates or frees memory.
 *   - Limit: the layer's expand_ws_bytes (see pipe_layout; about 4*O*I bytes) must not exceed
 *     PIPE_STATIC_SCRATCH_BYTES, otherwise PIPE_ERR_WORKSPACE is returned and nothing is queued.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as for every call here); under lazy module loading the driver may also load the
 *     module that holds the array at that moment.  Make that first call before any stream capture
 *     begins and before the application freezes its memory budget; from the second call on
 *     nothing is looked up or loaded.
 *   - All calls share the one array.  It keeps whatever the previous call left in it; this call
 *     overwrites every part before reading it, so nothing needs clearing.  Two calls whose GPU
 *     work overlaps (different streams, or different host threads) race on the array: run them
 *     one after the other on the device.
 * Arguments, alignment rules and device-side errors are those of pipe_expand_weights.
 */
#define PIPE_STATIC_SCRATCH_BYTES (4u << 20)
pipe_status pipe_expand_weights_static(const pipe_layer_desc* desc, const float* d_W, int64_t ldw, void* d_blob,
                                       size_t blob_bytes, void* stream);

/*
 * Appendix B, Eq. 9: the layer consumes Q(x) and one scale lambda_x for the whole tensor.
 * d_static_scale == NULL: lambda_x = max|x| / 127 (IEEE division); otherwise the given
 * scale is used and values are clamped.  xq = clamp(rne(x / lambda_x), -127, 127);
 * lambda_x = 0 gives all-zero codes.
 * d_x: float [T, I] pitch ldx.  d_xq: int8 [T, I] pitch ldxq.  d_sx: 1 float (written).
 * d_ws: quantize_ws_bytes bytes, 256-byte aligned.  T = 0 is allowed (lambda_x = 0).
 */
pipe_status pipe_quantize_act(const float* d_x, int64_t T, int32_t I, int64_t ldx, const float* d_static_scale,
                              int8_t* d_xq, int64_t ldxq, float* d_sx, void* d_ws, size_t ws_bytes, void* stream);

/*
 * The activation quantizers of Sec. 4.3 beside the int8 symmetric one: A6 and A4 ("150 % x W4/A6", W4/A4) and
 * asymmetric quantization (the parallelized comparison).  Codes are int8 values in every case, so the GEMM calls
 * take them unchanged.
 *   symmetric (asymmetric = 0), act_bits in {8, 6, 4}: qx = 2^(b-1) - 1, lambda_x = max|x| / qx or the static
 *       scale, c = clamp(rne(x / lambda_x), -qx, qx); *d_zp = 0.
 *   asymmetric: lo = min(x, 0), hi = max(x, 0) over the tensor, or d_static_range = {lo, hi} (lo <= 0 <= hi);
 *       lambda_x = (hi - lo) / (2^b - 1); z = clamp(rne(-2^(b-1) - lo / lambda_x)), c = clamp(rne(x / lambda_x) + z),
 *       both clamped to [-2^(b-1), 2^(b-1) - 1]; x ~ lambda_x * (c - z).  *d_zp = z is what
 *       pipe_ensemble_forward_zp takes.  d_static_scale must be NULL.
 * d_zp: one int32 (written).  Everything else as in pipe_quantize_act (binary32, IEEE division, ties to even).
 */
pipe_status pipe_quantize_act_ex(const float* d_x, int64_t T, int32_t I, int64_t ldx, int32_t act_bits, int32_t asymmetric,
                                 const float* d_static_scale, const float* d_static_range, int8_t* d_xq, int64_t ldxq,
                                 float* d_sx, int32_t* d_zp, void* d_ws, size_t ws_bytes, void* stream);

/*
 * Appendix B, Eq. 9 without the activation function: all K orders on one input,
 *     acc_k[t,o] = sum_i xq[t,i] * q_k[o,i]                    (exact int32)
 *     y[t,o]     = sum_{k ascending, o kept at k} fma(float(acc_k[t,o]), s_k[o] * lambda_x, .) (+ b[o])
 * i.e. the scale product is formed first, terms are added in ascending order starting from
 * zero, the bias last.  d_blob: output of pipe_expand_weights for the same desc.
 * d_xq: int8 [T, I] pitch ldxq; d_sx: 1 float; d_bias: float [O] or NULL;
 * d_y: float [T, O] pitch ldy.  d_partials (NULL, or int32 [T, total_rows]): when given,
 * receives acc_k[t, row] at column (sum_{j<k} rows[j]) + compacted row.  T = 0 is a no-op.
 * PIPE_ERR_ACC_OVERFLOW (from every call that takes the descriptor, pipe_layout included) if
 * 127 * qmax * 2^(8-b) * I >= 2^31, i.e. beyond I = 133144 (b = 8), 150976 (b = 4), 264208 (b = 2): the
 * kernels hold sub-byte codes as code * 2^(8-b) in their int32 accumulators.
 */
pipe_status pipe_expanded_linear(const pipe_layer_desc* desc, const void* d_blob, const int8_t* d_xq, int64_t T,
                                 int64_t ldxq, const float* d_sx, const float* d_bias, float* d_y, int64_t ldy,
                                 int32_t* d_partials, void* stream);

/*
 * Sec. 3.2 "Ensembling from Expansion", Fig. 2 and Appendix B: predictor m evaluates only the
 * orders of its cluster (orders sum_{l<m} K_l + 1 .. sum_{l<=m} K_l) on its own input x_m
 * with its own lambda_{x_m}; the bias belongs to predictor 1; predictor outputs are added
 * only after the last layer.  One layer of all M predictors as ONE grouped launch.
 * h_xq_m, h_sx_m, h_y_m: HOST arrays of M device pointers (int8 [T,I] pitch ldxq; 1 float;
 * float [T,O] pitch ldy); inputs may alias (shared input, the first layer of a network).
 * sum_branches != 0: only h_y_m[0] is written, with ((y_1 + y_2) + ...) + y_M, every y_m being predictor m's own
 * chain from zero (the bias closing y_1).  Predictors that share input and step (the same pointers) run as one launch
 * when K <= 8 (for more than 16 tokens the layer must also have the channel-block table of all K orders): the sums are
 * formed in registers; with distinct inputs it is one launch per predictor, in order, each adding into h_y_m[0].
 * d_partials as in pipe_expanded_linear.
 */
pipe_status pipe_ensemble_forward(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                  int64_t T, int64_t ldxq, const float* const* h_sx_m, const float* d_bias,
                                  float* const* h_y_m, int64_t ldy, int32_t sum_branches, int32_t* d_partials,
                                  void* stream);

/*
 * pipe_ensemble_forward on asymmetric activation codes (Sec. 4.3): with x_m ~ lambda_{x_m} (c_m - z_m) the
 * contraction is acc_k[t,o] = sum_i (c_m[t,i] - z_m) * q_k[o,i], an exact integer that the kernel forms as
 * sum_i c q - z_m * sum_i q; everything after it is unchanged.  h_zp_m: HOST array of M device pointers to one int32
 * each (NULL entries mean 0).  d_partials receives acc_k with the zero point taken out.  PIPE_ERR_ACC_OVERFLOW
 * cannot be excluded by the descriptor alone here: |c - z| reaches 255, so the layer must satisfy
 * 255 * qmax * I < 2^31 (checked).  Runs on the CUDA-core kernel.
 */
pipe_status pipe_ensemble_forward_zp(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                     int64_t T, int64_t ldxq, const float* const* h_sx_m, const int32_t* const* h_zp_m,
                                     const float* d_bias, float* const* h_y_m, int64_t ldy, int32_t sum_branches,
                                     int32_t* d_partials, void* stream);

/*
 * An INNER layer of the M predictors (Sec. 3.2, Fig. 2; Appendix B, Eq. 9 with its activation
 * function): predictor m's output never leaves the integer pipeline as floats.  Per predictor
 *     y_m            as in pipe_ensemble_forward (same order of operations, bias with predictor 1),
 *     a_m[t,o]       = sigma(y_m[t,o]), sigma chosen by `relu` (the argument keeps its first name): PIPE_ACT_IDENTITY,
 *                      PIPE_ACT_RELU, PIPE_ACT_SILU v / (1 + exp(-v)), PIPE_ACT_GELU v (1 + erf(v / sqrt 2)) / 2,
 *                      PIPE_ACT_SIGMOID 1 / (1 + exp(-v)) -- the functions Sec. 3.2 names for Eq. 9.  Identity and
 *                      ReLU are exact; the other three are evaluated in binary32 with the device's exp and erf, so
 *                      a_m can differ from a correctly rounded evaluation in its last bits and a code that lies on a
 *                      rounding boundary can come out one step off
 *     yq_m[t,o]      = clamp(rne(a_m[t,o] / s_m), -127, 127)             (Eq. 1 as the next layer's Q,
 *                                                                         IEEE binary32 quotient, ties to even)
 * so that yq_m and s_m are the next layer's xq_m and lambda_{x_m}.  s_m is a static step the caller
 * calibrated: h_out_scale_m is a HOST array of M device pointers to one float each (s_m >= 0 and
 * finite, else PIPE_ERR_INVALID_ARG through the device status; s_m = 0 gives all-zero codes).
 * h_yq_m: HOST array of M device pointers, int8 [T, O] pitch ldyq (>= O); no float output is
 * written.  The other arguments are those of pipe_ensemble_forward; M = 1 is the plain expanded
 * layer with this epilogue.  
 */
pipe_status pipe_ensemble_forward_q8(const pipe_layer_desc* desc, const void* d_blob, const int8_t* const* h_xq_m,
                                     int64_t T, int64_t ldxq, const float* const* h_sx_m, const float* d_bias,
                                     int32_t relu, const float* const* h_out_scale_m, int8_t* const* h_yq_m,
                                     int64_t ldyq, int32_t* d_partials, void* stream);

/*
 * The expanded layer as a two-dimensional convolution (Appendix H counts a d x d convolution as
 * d^2 * n_i * n_o multiplications per output pixel: the same contraction with the reduction
 * index running over (tap, input channel)).  Implicit GEMM: the quantized NHWC input is read in
 * place, tap by tap, at the convolution's stride, with zero padding supplied by the copy engine;
 * no im2col matrix exists.
 * Output size Ho = (H + 2*pad_h - kernel_h) / stride_h + 1, Wo likewise.  Output row
 * t = (n*Ho + ho)*Wo + wo, input pixel (stride_h*ho + dh - pad_h, stride_w*wo + dw - pad_w),
 * reduction index (dh*kernel_w + dw)*C + c, i.e. the weight tensor [O, kernel_h, kernel_w, C]
 * flattened to [O, I] with I = kernel_h*kernel_w*C = in_features.
 * All K orders act on the one input (as in pipe_expanded_linear).
 * d_xq: int8 [N, H, W, C], dense, 16-byte aligned (quantize it with pipe_quantize_act as a
 * [N*H*W, C] matrix).  d_y: float [N*Ho*Wo, O] pitch ldy.  d_partials as in pipe_expanded_linear
 * with T = N*Ho*Wo.
 * The library takes C a multiple of 128, strides 1..8 (0 means 1), 0 <= pad < kernel; anything else
 * returns PIPE_ERR_UNSUPPORTED (PIPE_ERR_SHAPE if the geometry contradicts itself or the layer).
 */
typedef struct pipe_conv_geom {
  int32_t batch, height, width, channels; /* N, H, W, C of the input */
  int32_t kernel_h, kernel_w;
  int32_t pad_h, pad_w;                   /* zeros on each side */
  int32_t stride_h, stride_w;             /* 0 is read as 1 */
} pipe_conv_geom;

pipe_status pipe_expanded_conv2d(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                 const int8_t* d_xq, const float* d_sx, const float* d_bias, float* d_y, int64_t ldy,
                                 int32_t* d_partials, void* stream);

/*
 * The convolution as an inner layer: pipe_expanded_conv2d with the epilogue of
 * pipe_ensemble_forward_q8 (sigma of Eq. 9, then Eq. 1 as the next layer's input quantizer with
 * the static step *d_out_scale).  d_yq: int8 [N*Ho*Wo, O] pitch ldyq; with ldyq = O it is the
 * NHWC input of the next convolution as it stands.  No float output is written.
 */
pipe_status pipe_expanded_conv2d_q8(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                    const int8_t* d_xq, const float* d_sx, const float* d_bias, int32_t relu,
                                    const float* d_out_scale, int8_t* d_yq, int64_t ldyq, int32_t* d_partials,
                                    void* stream);

/*
 * Sec. 3.2 (Fig. 2) for a convolution: predictor m applies its own cluster of orders (pipe_default_branches, or
 * desc->branch_orders) to its own NHWC input h_xq_m[m] with step *h_sx_m[m]; everything else as in
 * pipe_expanded_conv2d (geometry, layouts, alignment) and pipe_ensemble_forward (bias with predictor 0 only;
 * sum_branches != 0: the predictors' outputs are added in ascending m into h_y_m[0], each by the thread that wrote it;
 * otherwise predictor m writes h_y_m[m]; d_partials covers all K orders, each from its own predictor's input).
 * h_* are host arrays of num_branches device pointers.  One grouped launch; with sum_branches one launch if the
 * predictors share input and step (see pipe_ensemble_forward), one per predictor otherwise.
 */
pipe_status pipe_ensemble_conv2d(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                 const int8_t* const* h_xq_m, const float* const* h_sx_m, const float* d_bias,
                                 float* const* h_y_m, int64_t ldy, int32_t sum_branches, int32_t* d_partials, void* stream);

/*
 * The same as an inner layer of the M predictors (pipe_ensemble_forward_q8 on convolutions): predictor m hands
 * Q(sigma(y_m)) with the static step *h_out_scale_m[m] to h_yq_m[m], int8 [N*Ho*Wo, O] pitch ldyq -- with ldyq = O the
 * NHWC input of predictor m's next convolution.  `relu` is the activation kind (PIPE_ACT_*).
 */
pipe_status pipe_ensemble_conv2d_q8(const pipe_layer_desc* desc, const pipe_conv_geom* geom, const void* d_blob,
                                    const int8_t* const* h_xq_m, const float* const* h_sx_m, const float* d_bias,
                                    int32_t relu, const float* const* h_out_scale_m, int8_t* const* h_yq_m, int64_t ldyq,
                                    int32_t* d_partials, void* stream);

/*
 * The explicit form of the same contraction (Appendix H: reduction index (tap, input channel)), for the geometries
 * pipe_expanded_conv2d does not take -- a channel count that is not a multiple of 128, as in a network's first
 * layer: lowers the quantized NHWC tensor d_xq [N, H, W, C] to the rows
 *     d_rows[t, (dh*kernel_w + dw)*C + c] = d_xq[n, stride_h*ho + dh - pad_h, stride_w*wo + dw - pad_w, c]   (0 outside the image),
 * t = (n*Ho + ho)*Wo + wo, int8 [N*Ho*Wo, kernel_h*kernel_w*C] with row pitch ld_rows, which pipe_expanded_linear /
 * pipe_ensemble_forward then take as their [T, I] input with the tensor's own step.  Bytes of a row beyond
 * kernel_h*kernel_w*C are not written.  Caller-owned buffers; any alignment (16-byte aligned pointers, pitch and C give
 * the fast path).
 */
pipe_status pipe_lower_conv_input(const pipe_conv_geom* geom, const int8_t* d_xq, int8_t* d_rows, int64_t ld_rows, void* stream);

/* Number of kernels the library has launched in this process (all calls, all streams). */
uint64_t pipe_launch_count(void);

/* Synchronises `stream`, returns the device status word of the current device in
 * *h_status (a pipe_status value; PIPE_OK if nothing went wrong) and clears it. */
pipe_status pipe_poll_status(void* stream, int32_t* h_status);

const char* pipe_status_string(pipe_status s);

#ifdef __cplusplus
}
#endif
#endif /* PIPE_H_ */
