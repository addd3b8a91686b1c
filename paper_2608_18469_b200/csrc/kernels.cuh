// Launchers of the hand-written CUDA kernels behind the ERASE step library (host-callable).
// Every launcher only enqueues on the given stream and returns the launch's cudaError_t.
// "T" below is the model's activation type: float (ERASE_F32) or __nv_bfloat16 (ERASE_BF16),
// selected at run time by `bf16`.  All reductions use a fixed partition and a fixed combine
// order, so results do not depend on which stream or in which order kernels were enqueued.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace erase {

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU = 2 };

// Values of a model's device status word (0 = fine).  1..8: a bounded device-side wait expired
// (which one); STATUS_BAD_ID: the input staging met a token or sparse id outside its table.
enum { STATUS_WAIT_SELFTEST = 8, STATUS_BAD_ID = 64 };

// Epilogue of C = A * B^T.  With v = alpha * acc (+ bias[n]):
//   pre_out != 0 : pre_out[m,n] = v                    (pre-activation kept for the backward)
//   v = act(v)
//   mul    != 0 : v *= mul[m,n]                        (DCN-v2 cross: x0 (.) (W x + b))
//   res    != 0 : v += res[m,n]                        (residual / cross skip path)
//   dact   != 0 : v *= act'(dact_src[m,n])             (dgrad through an activation; GELU reads
//                                                       the pre-activation, ReLU the output)
// mul/res/dact_src/pre_out are T matrices with the row stride ld_aux.
struct Epilogue {
  const float* bias = nullptr;
  int act = ACT_NONE;
  void* pre_out = nullptr;
  const void* mul = nullptr;
  const void* res = nullptr;
  int dact = ACT_NONE;
  const void* dact_src = nullptr;
  long long ld_aux = 0;
  float alpha = 1.f;
  // Softmax cross-entropy head, forward (tensor-core kernels only): with l = acc + bias[n] the GEMM
  // stores exp(l - ce_ref[m]) instead of l and writes the fp32 sum of the unrounded exponentials of
  // row m over each group of columns to ce_psum[m * ce_groups + group].
  const float* ce_ref = nullptr;
  float* ce_psum = nullptr;
  int ce_groups = 0;
};

// C[M,N] = epilogue( sum_k A(m,k) * B(n,k) ).  A(m,k) = A[m*sa_m + k*sa_k], B likewise, so one
// routine serves the forward (X W^T), the dgrad (dY W: B strided over k) and the wgrad
// (dY^T X: both strided over k).  c_f32: C is float whatever T is (weight gradients).
// splits > 1: deterministic split-K; partial s is written to ws + s*M*N (float, row stride N)
// and summed in order s = 0..splits-1 by splitk_reduce; the epilogue must then be empty.
struct GemmArgs {
  int M = 0, N = 0, K = 0;
  const void* A = nullptr; long long sa_m = 0, sa_k = 0;
  const void* B = nullptr; long long sb_n = 0, sb_k = 0;
  void* C = nullptr; long long ldc = 0;
  int c_f32 = 0;
  int splits = 1;
  float* ws = nullptr;
  Epilogue epi;
  // Weight-gradient layout on the CTA-pair tensor-core kernel only (A and B both strided over k, no split,
  // N a multiple of 256): B carries 16 more columns behind its N (B(n, k) is valid for n < N + 16), and
  // xcol_out[m] = sum_k A(m, k) B(N, k), the product with the first of them, fp32, M values.  With the local
  // softmax head this is its bias gradient: A = P, column N of B = the row scales.  The extra columns cost one
  // narrow tile per row tile (a 16-wide MMA on the A tiles the neighbouring column tiles are reading anyway)
  // instead of a second pass over A.  tc_gemm_plan says whether a plan takes it (TcPlan::xcol).
  float* xcol_out = nullptr;
};

cudaError_t gemm_simt(const GemmArgs& g, bool bf16, cudaStream_t s);
// writes the device's nanosecond clock to *slot when the stream reaches this point
cudaError_t stamp_time(unsigned long long* slot, cudaStream_t s);
// out: float, or bfloat16 when out_bf16 (the sum is rounded once, after the last partial)
cudaError_t splitk_reduce(const float* ws, int splits, long long mn, int N, void* out, long long ldo,
                          cudaStream_t s, bool out_bf16 = false);

// out[c] = colscale[c] * sum_r scale[r] * f(X[r, c]); X is [rows, cols] with row stride ldx,
// f = identity or the derivative of activation `dact` evaluated at X; scale and colscale may be
// null (read as 1) and so may X (read as 1).  Two-stage with a fixed row partition into `chunks`
// in ONE launch: ws holds chunks*cols floats, tickets ceil(cols/64) zero-initialised ints (left
// at zero); the CTA that finishes a column strip last adds the partials in chunk order.
int colsum_chunks(int rows, int cols);
cudaError_t colsum(const void* X, bool x_bf16, long long ldx, int rows, int cols, const float* scale,
                   float* ws, int chunks, int* tickets, float* out, cudaStream_t s, int dact = ACT_NONE,
                   const float* colscale = nullptr);

// One entry of reduce_batch's job table (device memory).  kind 0: colsum with X, ldx, a = scale,
// b = colscale, dact, out0; kind 1: layernorm_param_grad with X = dy, X2 = x, a = mean, b = rstd,
// cols = d, out0 = dgain, out1 = dshift; kind 2: splitk_reduce to a float result with X = ws,
// rows = splits, mn, cols = N, ldx = ldo (mn, N, ldo multiples of 4, 16-byte aligned), chunks = 1.
// x_f32: X (and X2) hold floats, else bfloat16.  The job's CTAs are
// cta_begin .. cta_begin + strips*chunks - 1 of the launch (strip fastest).
struct ReduceJob {
  int kind = 0, x_f32 = 0, dact = ACT_NONE;
  int rows = 0, cols = 0, chunks = 1, strips = 1, cta_begin = 0;
  long long ldx = 0, mn = 0;
  const void* X = nullptr;
  const void* X2 = nullptr;
  const float* a = nullptr;
  const float* b = nullptr;
  float* ws = nullptr;
  float* out0 = nullptr;
  float* out1 = nullptr;
  int* tickets = nullptr;
};
int reduce_job_strips(const ReduceJob& j);
// All jobs of the table in one launch of total_ctas CTAs; each job computes what colsum /
// layernorm_param_grad would with the same arguments.
cudaError_t reduce_batch(const ReduceJob* jobs_dev, int njobs, int total_ctas, cudaStream_t s);

// LayerNorm over the last dimension (eps 1e-5, biased variance); saves mean and 1/std per row.
cudaError_t layernorm_fwd(const void* x, const float* gain, const float* shift, void* y, float* mean,
                          float* rstd, int rows, int d, bool bf16, cudaStream_t s);
// dx = rstd*(g - mean(g) - xhat*mean(g*xhat)) + add, g = dy*gain  (add may be null)
cudaError_t layernorm_bwd_dx(const void* dy, const void* x, const float* gain, const float* mean,
                             const float* rstd, const void* add, void* dx, int rows, int d, bool bf16,
                             cudaStream_t s);
// dgain[c] = sum_r dy*xhat, dshift[c] = sum_r dy; ws holds 2*chunks*d floats, tickets as for colsum.
cudaError_t layernorm_param_grad(const void* dy, const void* x, const float* mean, const float* rstd,
                                 float* ws, int chunks, int* tickets, float* dgain, float* dshift, int rows, int d,
                                 bool bf16, cudaStream_t s);

// Causal self-attention over qkv [batch*T, 3*d] = [Q | K | V], heads are contiguous dh-wide
// column slices; scale 1/sqrt(dh); o [batch*T, d]; lse [batch*heads*T] (natural log).
cudaError_t attention_fwd(const void* qkv, void* o, float* lse, int batch, int T, int heads, int dh,
                          bool bf16, cudaStream_t s, int* status = nullptr);
// dqkv [batch*T, 3*d] from do, with delta [batch*heads*T] as scratch.
cudaError_t attention_bwd(const void* qkv, const void* o, const void* dout, const float* lse,
                          float* delta, void* dqkv, int batch, int T, int heads, int dh, bool bf16,
                          cudaStream_t s, int* status = nullptr);

// tcgen05 / TMEM / TMA versions for bf16 with 64-wide heads (attention_tc.cu); same contracts.  status:
// the model's device status word (bounded waits), may be null.
bool attention_tc_supported(int dh, int d, const void* qkv, const void* o);
cudaError_t attention_fwd_tc(const void* qkv, void* o, float* lse, int batch, int T, int heads, int* status, cudaStream_t s);
// dqkv from dout, o and lse; delta [batch*heads*T] is scratch (delta[b,h,t] = sum_c dout * o over the head's 64 columns)
cudaError_t attention_bwd_tc(const void* qkv, const void* o, const void* dout, const float* lse, float* delta, void* dqkv, int batch,
                             int T, int heads, int* status, cudaStream_t s);
cudaError_t attention_delta_bf16(const void* o, const void* dout, float* delta, int batch, int T, int heads, cudaStream_t s);

// Tensor-core versions (mma.sync m16n8k16) for bf16 with 64-wide heads; same contracts.
bool attention_mma_supported(int dh, int d);
cudaError_t attention_fwd_mma(const void* qkv, void* o, float* lse, int batch, int T, int heads, cudaStream_t s);
cudaError_t attention_bwd_mma(const void* qkv, const void* o, const void* dout, const float* lse, float* delta,
                              void* dqkv, int batch, int T, int heads, cudaStream_t s);

// Softmax cross-entropy over logits [rows, V] (row stride V), in place:
// logits <- (softmax - onehot(target)) * inv_rows; rowloss[r] = logsumexp - logit[target].
// target of row r = ids[(r / T) * (T + 1) + (r % T) + 1].
// The same in-place softmax-CE (bf16 logits, V % 8 == 0, V <= 32768) as a persistent kernel of
// softmax_ce_fused_ctas(rows) CTAs that also leaves per-CTA column sums of the gradient it writes
// (fp32, before the bf16 rounding) in colpart[ctas][V]: summed over the CTAs they are the gradient
// of the head's bias.
int softmax_ce_fused_ctas(int rows);
bool softmax_ce_fused_supported(int V, bool bf16, const void* logits);
cudaError_t softmax_ce_fused(void* logits, const int32_t* ids, int T, float* rowloss, float* colpart, int rows, int V,
                             float inv_rows, cudaStream_t s);
cudaError_t softmax_ce_inplace(void* logits, const int32_t* ids, int T, float* rowloss, int rows, int V,
                               float inv_rows, bool bf16, cudaStream_t s);
// Softmax cross-entropy head without a pass over the logits (bf16, d % 8 == 0): see kernels.cu.
//   ce_target_logit  tgt[n] (clamped), ref[n] = lt[n] = z_n . W[t_n] + bias[t_n]; clears bad[0]
//   (head GEMM with Epilogue::ce_ref = ref writes P = exp(l - ref) and the partial sums psum)
//   ce_finalize      rowloss, rowscale r_n = 1/(S_n rows), P[n,t_n] -= S_n, zs = r (.) z; unsafe rows -> bad[1..], bad[0] = count
//                    (zs has row stride ldzs; with ldzs >= d + 16 each row ends in [r_n, 0 x 15]: GemmArgs::xcol_out)
//   ce_fixup         recomputes the listed rows exactly (no-op when bad[0] == 0 or *status != 0); bad holds rows+1 ints
//   ce_dz_finish     dz = r_n * (sum of `splits` fp32 partials of P W), rounded once
// after which the gradient of the logits is r (.) P: dW = P^T zs, db = column sums of P weighted by r.
cudaError_t ce_target_logit(const void* z, const void* W, const float* bias, const int32_t* ids, int T, int rows, int d, int V,
                            int* tgt, float* ref, float* lt, int* bad, cudaStream_t s);
cudaError_t ce_finalize(const float* psum, int groups, const float* ref, const float* lt, const int* tgt, void* P, int V, const void* z,
                        void* zs, int ldzs, float* rowloss, float* rowscale, int* bad, int rows, int d, float inv_rows, cudaStream_t s);
cudaError_t ce_fixup(const int* bad, const int* status, const int* tgt, const void* z, const void* W, const float* bias, void* P, float* ref,
                     const float* lt, void* zs, int ldzs, float* rowloss, float* rowscale, int rows, int d, int V, float inv_rows, cudaStream_t s);
cudaError_t ce_dz_finish(const float* part, int splits, int rows, int d, const float* rowscale, void* dz, cudaStream_t s);

// out[0] = (sum of v[0..n)) * scale, fixed-order tree in one CTA.
cudaError_t reduce_sum(const float* v, int n, float scale, float* out, cudaStream_t s);

// BCE head: s = z[r,:].w + b; rowloss = softplus(s) - y*s; ds[r] = (sigmoid(s) - y) * inv_rows
cudaError_t bce_head_fwd(const void* z, long long ldz, const float* w, const float* b, const float* y,
                         float* rowloss, float* ds, int rows, int d, float inv_rows, bool bf16,
                         cudaStream_t s);
// dz[r,c] = ds[r] * w[c]  (times act'(src[r,c]) when dact != ACT_NONE)
cudaError_t bce_head_dz(const float* ds, const float* w, void* dz, int dact, const void* src, int rows,
                        int d, bool bf16, cudaStream_t s);
// Goodness head: s[r] = sum_c z[r,c]^2 + b[0]; rowloss and ds as for the BCE head; dz = 2 ds z (* act'(src)).
cudaError_t goodness_head_fwd(const void* z, long long ldz, const float* b, const float* y, float* rowloss, float* ds,
                              int rows, int d, float inv_rows, bool bf16, cudaStream_t s);
cudaError_t goodness_head_dz(const float* ds, const void* z, void* dz, int dact, const void* src, int rows,
                             int d, bool bf16, cudaStream_t s);

// out = a (.) b, all [n] of T
cudaError_t ew_mul(const void* a, const void* b, void* out, long long n, bool bf16, cudaStream_t s);
// out = act(u)
cudaError_t ew_act(const void* u, void* out, int act, long long n, bool bf16, cudaStream_t s);
// d <- d * act'(src)
cudaError_t ew_dact(void* d, const void* src, int act, long long n, bool bf16, cudaStream_t s);

// z0[b*T+t, :] = tok[ids[b*(T+1)+t], :] + pos[t, :].  Every id of the batch (inputs and the last
// target column) is checked against [0, vocab): an id outside is not dereferenced (row 0 stands in)
// and *status is set to STATUS_BAD_ID.
cudaError_t gather_tokens(const float* tok, const float* pos, const int32_t* ids, void* z0, int batch,
                          int T, int d, int vocab, int* status, bool bf16, cudaStream_t s);
// x0[n, t*e + c] = tables[t*table_stride + ids[n*ns+t]*e + c]; x0[n, ns*e + j] = dense[n, j]; pad 0.
// ids are checked against [0, table_rows) in the same way.
cudaError_t gather_ctr(const float* tables, long long table_stride, const int32_t* ids,
                       const float* dense, void* x0, int batch, int ns, int e, int nd, int width,
                       int table_rows, int* status, bool bf16, cudaStream_t s);

// Dot interaction.  vectors of sample n: v_0 = proj[n, 0:e], v_j = x0[n, (j-1)e : je], j = 1..ns.
// feats[n, i(i-1)/2 + j] = v_i . v_j (i > j), then proj[n,:], then zeros up to width fw.
cudaError_t dot_fwd(const void* proj, const void* x0, long long ldx0, void* feats, int batch, int ns,
                    int e, int fw, bool bf16, cudaStream_t s);
// dproj[n,:] = dfeat[n, npair : npair+e] + sum_{j>=1} dfeat[n, j(j-1)/2] * v_j
cudaError_t dot_bwd(const void* dfeat, const void* x0, long long ldx0, void* dproj, int batch, int ns,
                    int e, int fw, bool bf16, cudaStream_t s);

// u = [src_0 | src_1 | ...] column-wise (the input of the main network, Eq. 2): u[r, offset_i + c] = src_i[r * ld_i + c]
constexpr int CONCAT_MAX = 32;
struct ConcatArgs {
  int n = 0, total = 0;
  const void* src[CONCAT_MAX];
  int width[CONCAT_MAX], offset[CONCAT_MAX];
  long long ld[CONCAT_MAX];
};
cudaError_t concat_cols(const ConcatArgs& a, void* u, int rows, bool bf16, cudaStream_t s);

// Embedding backward (the main network's gradient into the input tables), deterministic scatter-add:
// per table the (id, sample) pairs are sorted, distinct rows numbered, and one warp per distinct row
// adds the samples' slices dz0[n, t*e:(t+1)*e] in sample order into grow[t][s][:]; uniq_id[t][s] names
// the row, n_uniq[t] counts them.  sorted_n, uniq_id: ns*batch ints; seg_start: ns*(batch+1); grow: ns*batch*e floats.
// batch <= embed_max_batch().  embed_update applies the optimizer to those rows only.
int embed_max_batch();
cudaError_t embed_backward(const void* dz0, long long ld, const int32_t* ids, int batch, int ns, int e, int table_rows, int* sorted_n,
                           int* seg_start, int* uniq_id, int* n_uniq, float* grow, bool bf16, cudaStream_t s);
cudaError_t embed_update(float* tables, long long table_stride, float* m, float* v, int batch, int ns, int e, const int* uniq_id,
                         const int* n_uniq, const float* grow, int kind, float lr, float beta1, float beta2, float eps, float wd,
                         const double* tick, cudaStream_t s);

// Optimizer over a flat range.  kind 0 SGD, 1 Adam, 2 AdamW.  tick[0] = step count t (as float
// bits of an int64 are avoided: tick is {t, 1-beta1^t, 1-beta2^t} kept on the device so that a
// replayed CUDA graph advances it).  shadow (bf16 copy of theta) may be null.
cudaError_t opt_tick(double* tick, float beta1, float beta2, cudaStream_t s);
cudaError_t opt_update(float* theta, const float* grad, float* m, float* v, void* shadow, long long n,
                       int kind, float lr, float beta1, float beta2, float eps, float wd,
                       const double* tick, cudaStream_t s);
// shadow[i] = bf16(theta[i])
cudaError_t to_bf16(const float* src, void* dst, long long n, cudaStream_t s);

}  // namespace erase
