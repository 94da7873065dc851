/*
 * ampq.h -- C ABI of the B200 loss-MSE sensitivity pass.
 *
 * The library scores every linear layer (operands X, W) and every batched GEMM
 * (operands X0, X1) of a model over R calibration samples: per-tensor amax and
 * FP8 scale, round-to-nearest-even FP8 cast, quantisation error, squared error
 * weighted by the squared loss gradient, per-sample and mean sensitivities; it
 * then sums the loss-MSE terms per sequential sub-graph and selects the
 * precision assignment of the paper's integer program under a loss-MSE budget.
 * Everything up to the per-layer values runs in CUDA kernels on one sm_100a
 * device; the sub-graph sums and the selection run on the host.
 *
 * Conventions
 *   - Every function returns an int status: AMPQ_OK (0) or a negative
 *     AMPQ_ERR_* code.  Nothing throws, aborts or prints.  ampq_strerror maps a
 *     code to text; ampq_last_error(ctx) adds detail for the last failure.
 *   - "device pointer" = memory of the context's CUDA device; "host pointer" =
 *     ordinary host memory.  The caller owns every tensor and every output
 *     array; the library owns only its workspace (tables, per-tile partial
 *     sums, results), allocated with cudaMalloc when ampq_score first needs it
 *     and released by ampq_destroy.
 *   - Kernels are launched on the stream given to ampq_create.  ampq_score is
 *     asynchronous; the getters synchronise that stream.
 *   - A context is not thread-safe; use one per thread or lock around it.
 *   - There is no CPU fallback: without a CUDA device ampq_create fails with
 *     AMPQ_ERR_CUDA.
 */
#ifndef AMPQ_H
#define AMPQ_H

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ampq_ctx ampq_ctx;

/* element type of an operand and of its gradient */
enum { AMPQ_F32 = 0, AMPQ_BF16 = 1 };
/* numerical formats.  BASE is the high-precision format (BF16 in the paper's
 * setup, Sec. 3.1); its loss-MSE contribution is 0.  E4M3: 4 exponent, 3
 * mantissa bits, bias 7, no infinity, largest finite value 448.  E5M2: 5
 * exponent, 2 mantissa bits, bias 15, largest finite value 57344. */
enum { AMPQ_FMT_BASE = 0, AMPQ_FMT_E4M3 = 1, AMPQ_FMT_E5M2 = 2 };
/* layer kinds: Y = X W^T + b (Sec. 2.2, linear layer) and Y = X0 (x) X1 (BGEMM) */
enum { AMPQ_LINEAR = 0, AMPQ_BGEMM = 1 };
/* which per-layer loss-MSE feeds the sub-graph sums:
 * MODEL    d_{l,f} = alpha_f * s_l, alpha_f = 2^(-2 m_f)/12   (Sec. 2.2)
 * MEASURED d_{l,f} = (1/R) sum_r sum_k (g_k (Q_f(z_k) - z_k))^2, the same
 *          expectation with the realised FP8 rounding error                */
enum { AMPQ_D_MODEL = 0, AMPQ_D_MEASURED = 1 };
/* where a bound tensor lives */
enum { AMPQ_MEM_DEVICE = 0, AMPQ_MEM_HOST = 1 };

enum {
    AMPQ_OK = 0,
    AMPQ_ERR_INVALID = -1,     /* null pointer, bad enum, bad id, bad size          */
    AMPQ_ERR_ALIGN = -2,       /* a tensor pointer is not aligned to its element    */
    AMPQ_ERR_STATE = -3,       /* call out of order (e.g. results before a score)   */
    AMPQ_ERR_CUDA = -4,        /* a CUDA call failed; see ampq_last_error           */
    AMPQ_ERR_NONFINITE = -5,   /* a scored operand holds Inf or NaN                 */
    AMPQ_ERR_INFEASIBLE = -6,  /* no assignment meets the budget                    */
    AMPQ_ERR_TOO_LARGE = -7,   /* too large: selection state limit, tile count, fixed scratch */
    AMPQ_ERR_NOMEM = -8,
    AMPQ_ERR_TIMEOUT = -9      /* a bounded wait inside a kernel ran out; results invalid */
};

const char *ampq_strerror(int status);
const char *ampq_last_error(const ampq_ctx *ctx);

/* Creates a context on CUDA device `device`.  `cuda_stream` is a cudaStream_t
 * (0 = the default stream), borrowed for the life of the context: every kernel
 * and copy of this context is issued on it. */
int ampq_create(ampq_ctx **out, int device, void *cuda_stream);
int ampq_destroy(ampq_ctx *ctx);

/* The F formats of the problem (Sec. 2.1: "F distinct numerical formats").
 * fmt[0] must be AMPQ_FMT_BASE; fmt[1..F-1] are distinct low-precision formats
 * (F <= 3).  Default: {BASE, E4M3}.  Must be called before layers are scored;
 * changing it invalidates earlier results. */
int ampq_set_formats(ampq_ctx *ctx, const int *fmt, int F);

/* Registers one layer with R calibration samples (Sec. 2.2: layer l, samples
 * r = 0..R-1).  `name` is copied (may be NULL).  Writes the layer id
 * (0, 1, 2, ... in registration order). */
int ampq_register_layer(ampq_ctx *ctx, int kind, const char *name, int R, int *layer_id);

/* Binds operand 0 (X or X0) or 1 (W or X1) of a layer: the two halves of the
 * layer's extended input z_l (Sec. 2.2).
 *   values  numel elements of `dtype`, contiguous.
 *           per_sample_values = 1: laid out [R, numel/R]; sample r owns slice r
 *           (activations, BGEMM operands; numel must be a multiple of R).
 *           per_sample_values = 0: one tensor shared by all samples (weights).
 *   grads   the loss gradient with respect to this operand, same dtype: sample
 *           r's gradient starts at grads + r*grad_stride elements and has the
 *           extent of the values it weights (numel/R, or numel when shared).
 *   mem     AMPQ_MEM_DEVICE: device pointers, read in place.  AMPQ_MEM_HOST:
 *           host pointers; every ampq_score copies them to library-owned device
 *           staging on the stream first (pinned memory makes that copy
 *           asynchronous).
 * The tensors are borrowed: they must stay valid and unchanged until the work
 * of the last ampq_score on the stream has finished.  Pointers must be aligned
 * to the element size (AMPQ_ERR_ALIGN otherwise); 16-byte alignment of every
 * sample slice enables the vectorised path, anything else is scored
 * correctly through a slower scalar path.  numel = 0 is allowed (scores 0).
 * Re-binding replaces the previous binding.  Several layers may bind the very
 * same values (layers that read one input); see ampq_set_sharing. */
int ampq_bind_operand(ampq_ctx *ctx, int layer_id, int operand, int dtype, int mem,
                      const void *values, long long numel, int per_sample_values,
                      const void *grads, long long grad_stride);

/* Optional static scale: use `amax` for this operand instead of measuring it
 * (the amax pass then skips the tensor).  Values above amax saturate.  A
 * negative amax removes the preset. */
int ampq_set_amax(ampq_ctx *ctx, int layer_id, int operand, float amax);

/* Declares that every sample slice of a per-sample operand is a stack of T x T
 * matrices (the last two dimensions) whose entries right of the diagonal are
 * EXACTLY zero, as in a causal softmax.  Such entries add nothing to amax, S or
 * D_f whatever their gradient holds, so the library does not read them (about
 * half the bytes of the operand and of its gradient).  Taken up when T is a
 * power of two in [64, 32768], a sample slice is a whole number of matrices and
 * the slices are 16-byte aligned; otherwise the operand is scored in full, with
 * the same result.  The declaration is a promise: if the triangle is not zero,
 * some of its entries (those sharing a 16-byte vector with the diagonal) are
 * still scored and the rest are not, so the result is neither the dense one nor
 * that of the zeroed operand.  T = 0 removes the declaration. */
int ampq_set_causal(ampq_ctx *ctx, int layer_id, int operand, long long T);

/* How the per-tensor scale is formed from amax (default AMPQ_SCALE_AMAX):
 *   AMPQ_SCALE_AMAX  scale = fl32(amax/fmax_f), inv = fl32(fmax_f/amax)
 *   AMPQ_SCALE_POW2  scale = the smallest power of two p with fmax_f*p >= amax,
 *                    inv = 1/p: nothing saturates and z*inv is exact; (1,1)
 *                    when amax = 0 or p is not a normal fp32.
 * Applies to ampq_score, ampq_stream_sample and ampq_fake_quant. */
enum { AMPQ_SCALE_AMAX = 0, AMPQ_SCALE_POW2 = 1 };
int ampq_set_scale_mode(ampq_ctx *ctx, int mode);

/* on = 0: score only the paper's own term, S = sum (z g)^2, from which
 * d_model_f = alpha_f s follows (Sec. 2.2); the amax pass, the scales and the FP8
 * cast are skipped, every measured value (D_f, d_meas) reads 0, amax reads 0
 * (or the preset) and the scales are those of that amax.  One read of operand and
 * gradient instead of two of the operand.  Inf/NaN in an operand is then not
 * detected up front: it shows as a non-finite S.  on = 1 (default): both terms.
 * Applies to ampq_score and ampq_stream_sample. */
int ampq_set_measured(ampq_ctx *ctx, int on);

/* Layers that read one input (q, k, v or gate, up of a transformer block) bind
 * the very same values pointer with gradients of their own: z is shared, the
 * per-layer sensitivity s_l^r = ||z (.) dz||^2 of Sec. 2.2 differs only in the
 * gradient.  With sharing on (the default) the library recognises such
 * bindings by pointer, size, dtype, R, gradient stride and preset: the amax of
 * the values is measured once, and up to four such per-sample operands are
 * scored in one read and one FP8 cast of the values with one gradient stream
 * per layer.  Results are those of separate scoring up to the order of the
 * fp64 additions.  on = 0 treats every binding as a tensor of its own -- for
 * callers that re-use one buffer for unrelated layers' bindings. */
int ampq_set_sharing(ampq_ctx *ctx, int on);

/* Only the first step of ampq_score: amax of every bound operand of every fully
 * bound layer (preset ones keep their preset), asynchronously on the stream.
 * ampq_get_amax (synchronises) then gives amax[2] of a layer; it also works
 * after ampq_score.  Meant for calibration split over several processes by
 * sample: each measures its own samples, the maxima are combined outside (a
 * MAX all-reduce), set with ampq_set_amax, and then every process scores. */
int ampq_measure_amax(ampq_ctx *ctx);
int ampq_get_amax(ampq_ctx *ctx, int layer_id, float *amax);

/* Scores every layer whose two operands are bound (Algorithm 1 step 2, the
 * per-element part), asynchronously on the context's stream:
 *   amax_t = max_k |z_k| per tensor; per format f: scale = fl32(amax/fmax_f),
 *   inv = fl32(fmax_f/amax) ((1,1) when amax = 0 or inv is not finite);
 *   q_k = RNE saturating FP8 cast of fl32(z_k * inv); e_k = dec(q_k)*scale - z_k;
 *   per (tensor, sample): S = sum_k (z_k g_k)^2, D_f = sum_k (g_k e_k)^2;
 *   per layer: s^r = S(op0,r) + S(op1,r), s = mean_r s^r, d_model_f = alpha_f s,
 *   d_meas_f = mean_r (D_f(op0,r) + D_f(op1,r)).
 * Sums are accumulated in fp32 over runs of at most 64 terms per lane and
 * combined in a fixed order in fp64, so results are reproducible run to run.
 * The scoring kernel's internal waits are bounded: if one ever runs out, the
 * getters return AMPQ_ERR_TIMEOUT for that score and the context stays usable. */
int ampq_score(ampq_ctx *ctx);

/* Streaming form of the same step, for calibration loops that see one sample
 * at a time (Algorithm 1 step 2: forward and backward per calibration sample)
 * and never hold all R per-sample weight gradients at once.
 *   ampq_stream_begin   clears the per-sample sums of every registered layer.
 *   ampq_stream_sample  scores ONE sample r of one operand, asynchronously on
 *                       the stream: values/grads are device pointers to numel
 *                       elements each (activations: sample r's slice; weights:
 *                       the whole weight and the gradient of sample r's loss
 *                       with respect to it), borrowed until the work has
 *                       finished.  The operand's preset amax (ampq_set_amax) is
 *                       used when there is one -- the static-scale case, and
 *                       the way to score activations with one scale for all
 *                       samples; without a preset the amax of the tensor passed
 *                       in THIS call is measured and used.  A sample streamed
 *                       twice is overwritten, not added.  Operands need not be
 *                       bound.
 *   ampq_stream_end     forms the per-layer values from whatever was streamed
 *                       (samples never streamed count as 0); afterwards
 *                       ampq_get_layer / ampq_get_operand / ampq_group_costs /
 *                       ampq_select work as after ampq_score.  The amax a
 *                       getter reports is the largest any sample used, the
 *                       scales are those of the last sample streamed.
 * Sums equal those of ampq_score over the same data and amax up to the order
 * of the fp64 additions. */
int ampq_stream_begin(ampq_ctx *ctx);
int ampq_stream_sample(ampq_ctx *ctx, int layer_id, int operand, int r, int dtype, const void *values,
                       const void *grads, long long numel);
int ampq_stream_end(ampq_ctx *ctx);

/* The quantised operand itself (z^ = z + z~ of Sec. 2.2): writes
 * dec(Q(z*inv))*scale, one fp32 product stored in the operand's own dtype
 * (bf16: round to nearest even), for numel elements; values and dev_out are
 * device pointers (dev_out may equal values).  amax >= 0: use it; < 0: measure
 * it over `values`.  fmt must be in the context's format list.  Asynchronous
 * on the stream.  Used to run a model "in format f" when checking predicted
 * against measured loss MSE (Sec. 3.2). */
int ampq_fake_quant(ampq_ctx *ctx, int dtype, int fmt, const void *values, long long numel, float amax,
                    void *dev_out);

/* Number of kernel launches issued by the last ampq_score (diagnostics). */
int ampq_last_launch_count(const ampq_ctx *ctx);

/* log2 of the scoring tile (elements) the last ampq_score used, 13..21: the
 * largest that still gives every CTA of the persistent grid 16 tiles; 0 before
 * a score (diagnostics: tests use it to check that they run the launch geometry
 * they mean to). */
int ampq_last_tile_shift(const ampq_ctx *ctx);

/* Bytes of the bound tensors that the last ampq_score (or ampq_measure_amax)
 * reads (diagnostics; host pointer, bytes[2]): bytes[0] the amax pass -- every
 * operand without a preset once, an operand several layers share once;
 * bytes[1] the scoring pass -- values and gradients as the kernels walk them:
 * shared values (weights) once per group of up to four samples, an input shared
 * by several layers once per group, triangular operands only up to the
 * diagonal. */
int ampq_get_pass_bytes(ampq_ctx *ctx, long long *bytes);

/* Optional device timing of the kernels of a score.  With timing on, ampq_score
 * records CUDA events on its stream around the amax kernel, the scoring kernel
 * and the whole call; ampq_get_timing (synchronises) writes ms[3] = {amax
 * kernel, scoring kernel, whole score including staging copies and read-back}
 * of the last score, in milliseconds.  Off by default. */
int ampq_set_timing(ampq_ctx *ctx, int on);
int ampq_get_timing(ampq_ctx *ctx, float *ms);

/* Results of one layer after ampq_score (synchronises the stream on the first
 * call after a score).  Any output pointer may be NULL.  Host pointers.
 *   amax[2]                 per operand
 *   scale[2*F], inv_scale[2*F]   index operand*F + f; entry f = 0 is 1
 *   s_per_sample[R]         s_l^r      (Sec. 2.2, per-sample sensitivity)
 *   s_mean                  s_l        (Sec. 2.2, average sensitivity)
 *   d_meas_per_sample[R*F]  index r*F + f; column 0 is 0
 *   d_model[F], d_meas[F]   entry 0 is 0
 * Returns AMPQ_ERR_NONFINITE if the layer's operands held Inf/NaN. */
int ampq_get_layer(ampq_ctx *ctx, int layer_id, float *amax, float *scale, float *inv_scale,
                   double *s_per_sample, double *s_mean, double *d_meas_per_sample,
                   double *d_model, double *d_meas);

/* The per-layer table of n layers in one call (synchronises like ampq_get_layer):
 * out is [n][1 + 2F] row-major, row i = {s_l, d_model[0..F-1], d_meas[0..F-1]} of
 * layer layer_ids[i] -- what the sub-graph sums and the selection need, and what
 * processes that share a model exchange.  Host pointers.  AMPQ_ERR_NONFINITE
 * (rows still written) if one of the layers held Inf/NaN. */
int ampq_get_layer_table(ampq_ctx *ctx, const int *layer_ids, int n, double *out);

/* Per-operand sums of a layer: out[R*F], index r*F + a, a = 0: S, a = f >= 1:
 * D_f.  Host pointer. */
int ampq_get_operand(ampq_ctx *ctx, int layer_id, int operand, double *out);

/* Test hook: writes the FP8 code of every element of a bound DEVICE operand
 * (numel bytes, device pointer), using the scales of the last ampq_score and
 * the same cast the scoring kernel applies.  Asynchronous on the stream. */
int ampq_export_codes(ampq_ctx *ctx, int layer_id, int operand, int fmt, unsigned char *dev_out);

/* Defines sequential sub-graph (group) V_j = {layer_ids[0..Lj-1]} with Pj
 * configurations (Sec. 2.1): Q[l + Lj*p] in [0,F-1] is the index into the
 * context's format list that configuration p gives layer l of the group, and
 * c[p] is its performance metric (time gain, MAC gain or memory gain).  Q and
 * c are copied.  Writes the group id (0, 1, ... in definition order, which is
 * also the order j of the selection). */
int ampq_define_group(ampq_ctx *ctx, const int *layer_ids, int Lj, const unsigned char *Q,
                      const double *c, int Pj, int *group_id);
int ampq_clear_groups(ampq_ctx *ctx);

/* d_{j,p} = sum_{l=0}^{Lj-1} d_{l_{j,l}, Q_j[l,p]} (Sec. 2.2, last equation),
 * left fold in l, from the last score.  d_out[Pj], host pointer. */
int ampq_group_costs(ampq_ctx *ctx, int group_id, int d_mode, double *d_out);

/* The same sums from a caller-supplied per-layer table (no context, no GPU;
 * used when layers were scored by several contexts or processes): d_layer is
 * [L][F] row-major, layer_ids[l] in [0, L).  d_out[Pj]. */
int ampq_group_costs_table(const int *layer_ids, int Lj, const unsigned char *Q, int Pj,
                           const double *d_layer, int L, int F, double *d_out);

/* budget = tau^2 * (1/R) sum_r losses[r]^2 (Sec. 2.1; E[g^2] is the
 * mean-square loss of Algorithm 1 step 2).  Needs no context. */
int ampq_budget_from_tau(double tau, const double *losses, int R, double *budget);

/* Loss MSE of the configuration that puts every scored layer in format index
 * f (1..F-1): the left fold over layers of d_{l,f}; used for budgets stated as
 * a fraction of the all-low-precision loss MSE. */
int ampq_all_lowp_cost(ampq_ctx *ctx, int d_mode, int f, double *d_all);

/* Solves the integer program of Sec. 2.1 exactly over the defined groups:
 * maximise sum_j c_{j,p_j} subject to sum_j d_{j,p_j} <= budget, one p_j per
 * group.  Sums are left folds over j = 0..J-1 in double.  Among optimal
 * assignments the one with the smaller d wins, then the lexicographically
 * smaller (p_0..p_{J-1}).  p_out[J] host.  AMPQ_ERR_INFEASIBLE if no
 * assignment meets the budget. */
int ampq_select(ampq_ctx *ctx, int d_mode, double budget, int *p_out, double *c_total,
                double *d_total);

/* The same solver on caller-supplied tables (no context, no GPU): group j owns
 * entries off[j] .. off[j]+P[j]-1 of c[] and d[]. */
int ampq_select_tables(int J, const int *P, const long long *off, const double *c,
                       const double *d, double budget, int *p_out, double *c_total,
                       double *d_total);

/* Calibration split over several processes by SAMPLE: every entry of a
 * per-layer table (s_l, d_model_{l,f}, d_meas_{l,f}) is a mean over calibration
 * samples (Sec. 2.2: s_l = (1/R) sum_r s_l^r), so the value over all samples is
 * the R-weighted mean of the per-process values.  tables is [nranks][L][K]
 * row-major (process i's table computed over its R_local[i] samples), out is
 * [L][K]: out = sum_i R_local[i] * tables[i] / sum_i R_local[i], the sum taken
 * in order i = 0..nranks-1.  Host pointers; no context, no GPU. */
int ampq_merge_sample_tables(const double *tables, const int *R_local, int nranks, int L, int K,
                             double *out);

/* Partition of a model's computation graph into sequential sub-graphs
 * (Appendix B, Algorithm 2).  Vertices 0..n-1, directed edges edge_src[e] ->
 * edge_dst[e]; the graph must be acyclic with exactly one sink (the end
 * vertex); a start vertex is put in front of every source.  Every vertex that
 * all start -> end paths run through closes a sub-graph; a vertex belongs to
 * the sub-graph closed by the first such vertex it reaches.  group_of[v] is the
 * index (0, 1, ... in execution order) of the sub-graph of quantisable vertex v
 * and -1 for the others; sub-graphs without a quantisable vertex get no index.
 * Residual connections drawn as edges merge everything they span into one
 * sub-graph; leave them out to split a transformer layer as the paper's figure
 * does.  Host pointers.  AMPQ_ERR_INVALID for a cycle, several sinks or a bad
 * edge. */
int ampq_partition(int n, int n_edges, const int *edge_src, const int *edge_dst,
                   const unsigned char *quantisable, int *group_of, int *n_groups);

/* Performance-metric table of one group from layer shapes: c_out[p] = sum_l
 * c_{l, Q[l + Lj*p]} with, per layer and format f,
 *   AMPQ_GAIN_MAC     N C K delta[f] (linear), N C^2 delta[f] (BGEMM): the
 *                     theoretical time gain of Sec. 2.3.2, delta[f] the time
 *                     gained per multiply-accumulate in format f;
 *   AMPQ_GAIN_MEMORY  C K delta[f] (linear), 0 (BGEMM): the memory gain of
 *                     Sec. 2.3.3, delta[f] the bytes saved per stored parameter.
 * N, C, K [Lj]; delta[F] (delta[0] = 0 for the baseline format).  Host pointers. */
enum { AMPQ_GAIN_MAC = 0, AMPQ_GAIN_MEMORY = 1 };
int ampq_gain_table(int gain_kind, int Lj, const int *layer_kind, const long long *N, const long long *C,
                    const long long *K, const unsigned char *Q, int Pj, const double *delta, int F,
                    double *c_out);

/* The baseline strategies the paper compares with (Sec. 3.1): units (layers or
 * groups) are switched to low precision one after the other in the order given
 * while the loss-MSE budget holds, stopping at the first that does not fit.
 * order = 0..L-1 is "Prefix"; a random permutation drawn by the caller is
 * "Random".  d_low[u], c_low[u]: loss MSE and gain of unit u in low precision.
 * chosen[u] = 1 for the units switched.  Host pointers. */
int ampq_select_in_order(int L, const int *order, const double *d_low, const double *c_low, double budget,
                         unsigned char *chosen, double *c_total, double *d_total);

/* The paper has no counterpart of this call; it exists for callers that are
 * not allowed to allocate device memory: code that runs while another library
 * owns the device heap through its own pool, code in a phase where a device
 * allocation would stall or fragment the heap, plug-ins that are handed fixed
 * buffers.  It runs the same pass as ampq_score (amax, scales, FP8 cast,
 * error, gradient weighting, per-tile sums, ordered fp64 combine) on ONE
 * segment -- numel elements of `values` weighted by `grads`, one low-precision
 * format `fmt` (AMPQ_FMT_E4M3 or AMPQ_FMT_E5M2) -- and calls no cudaMalloc,
 * cudaFree or other allocating routine: its tables and per-tile partial sums
 * live in a fixed array in the library's device image (about 64 KiB, held by
 * every GPU that loads the library until the process exits).
 *   device, cuda_stream   the device, and a cudaStream_t on it (0 = default)
 *   values, grads         device pointers, numel elements of `dtype` each,
 *                         aligned to the element size; borrowed until the work
 *                         on the stream has finished
 *   numel                 0 .. AMPQ_NOALLOC_MAX_NUMEL; larger sizes are refused
 *                         with AMPQ_ERR_TOO_LARGE before anything is launched
 *   amax                  >= 0: use this amax (static scale); < 0: measure it
 *   dev_out               device pointer, 3 doubles, 8-byte aligned:
 *                         {S = sum (z g)^2, D = sum (g (Q(z) - z))^2, amax};
 *                         S and D are NaN when the operand holds Inf or NaN
 * Asynchronous on the stream; nothing is copied to the host.  The first call on
 * a device looks up the array's device address (once per device); make that
 * first call before any stream capture begins.  Every call on a device uses
 * the same array and overwrites what the previous call left there, so calls
 * whose work may overlap on the GPU (different streams, different threads)
 * race: order them on one stream or with events. */
#define AMPQ_NOALLOC_MAX_NUMEL 2147483648LL
int ampq_score_segment_noalloc(int device, void *cuda_stream, int dtype, int fmt, const void *values,
                               const void *grads, long long numel, float amax, double *dev_out);

#ifdef __cplusplus
}
#endif
#endif /* AMPQ_H */
