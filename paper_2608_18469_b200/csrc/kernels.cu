// Hand-written CUDA kernels (plain SIMT) of the ERASE step library: the general GEMM used for
// fp32 models and for shapes the tensor-core path does not take, and every non-GEMM operation
// of the step (LayerNorm, causal attention, losses, gathers, dot interaction, optimizer).
// Reductions are fixed-partition / fixed-order: no floating-point atomics anywhere.
#include "kernels.cuh"
#include "ew_math.cuh"

#include <stdlib.h>

#include <algorithm>
#include <atomic>

#include <cuda_bf16.h>
#include <math.h>

namespace erase {

typedef __nv_bfloat16 bf16_t;

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<bf16_t>(const bf16_t* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<bf16_t>(bf16_t* p, float v) { *p = __float2bfloat16_rn(v); }
// four consecutive values (p 16-byte aligned for float, 8-byte for bf16)
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(bf16_t* p, float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 q;
  q.x = *reinterpret_cast<uint32_t*>(&lo);
  q.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = q;
}

__device__ __forceinline__ float act_apply(int act, float v) {
  if (act == ACT_RELU) return v > 0.f ? v : 0.f;
  if (act == ACT_GELU) return v * 0.5f * (1.f + erff(v * 0.70710678118654752f));
  return v;
}
// derivative of the activation; GELU takes the pre-activation, ReLU accepts either the
// pre-activation or the output (same sign test; 0 at exactly 0).
__device__ __forceinline__ float act_deriv(int act, float u) {
  if (act == ACT_RELU) return u > 0.f ? 1.f : 0.f;
  if (act == ACT_GELU) {
    float cdf = 0.5f * (1.f + erff(u * 0.70710678118654752f));
    float pdf = 0.39894228040143268f * expf(-0.5f * u * u);
    return cdf + u * pdf;
  }
  return 1.f;
}

template <typename T> __device__ __forceinline__ float gelu_ew(float u);
template <> __device__ __forceinline__ float gelu_ew<float>(float u) { return act_apply(ACT_GELU, u); }
template <> __device__ __forceinline__ float gelu_ew<bf16_t>(float u) { return gelu_bf16_value(u); }
template <typename T> __device__ __forceinline__ float dgelu_ew(float u);
template <> __device__ __forceinline__ float dgelu_ew<float>(float u) { return act_deriv(ACT_GELU, u); }
template <> __device__ __forceinline__ float dgelu_ew<bf16_t>(float u) { return gelu_bf16_deriv(u); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

static inline unsigned cdiv(long long a, long long b) { return (unsigned)((a + b - 1) / b); }

// ------------------------------------------------------------------------------------------
// general GEMM, 64x64x16 tiles, 256 threads, 4x4 outputs per thread, fp32 FMA
// ------------------------------------------------------------------------------------------
template <typename T, bool AK, bool BK>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs g) {
  __shared__ __align__(16) float As[16][68];
  __shared__ __align__(16) float Bs[16][68];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64, split = blockIdx.z;
  const int kchunk = (((g.K + g.splits - 1) / g.splits) + 15) / 16 * 16;
  const int kbeg = split * kchunk;
  const int kend = min(g.K, kbeg + kchunk);
  const T* A = (const T*)g.A;
  const T* B = (const T*)g.B;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) acc[i][j] = 0.f;

  for (int k0 = kbeg; k0 < kend; k0 += 16) {
#pragma unroll
    for (int it = 0; it < 4; it++) {
      int i = tid + it * 256;
      int mm, kk;
      if (AK) { kk = i & 15; mm = i >> 4; } else { mm = i & 63; kk = i >> 6; }
      int gm = m0 + mm, gk = k0 + kk;
      float v = 0.f;
      if (gm < g.M && gk < kend) v = ldf(A + (long long)gm * g.sa_m + (long long)gk * g.sa_k);
      As[kk][mm] = v;
      int nn;
      if (BK) { kk = i & 15; nn = i >> 4; } else { nn = i & 63; kk = i >> 6; }
      int gn = n0 + nn;
      gk = k0 + kk;
      v = 0.f;
      if (gn < g.N && gk < kend) v = ldf(B + (long long)gn * g.sb_n + (long long)gk * g.sb_k);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; kk++) {
      float4 a4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      float4 b4 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      float a[4] = {a4.x, a4.y, a4.z, a4.w};
      float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  const Epilogue& e = g.epi;
#pragma unroll
  for (int i = 0; i < 4; i++) {
    int m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      int n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float v = acc[i][j];
      if (g.splits > 1) {
        g.ws[(long long)split * g.M * g.N + (long long)m * g.N + n] = v;
        continue;
      }
      v *= e.alpha;
      if (e.bias) v += e.bias[n];
      long long ia = (long long)m * e.ld_aux + n;
      if (e.pre_out) stf((T*)e.pre_out + ia, v);
      v = act_apply(e.act, v);
      if (e.mul) v *= ldf((const T*)e.mul + ia);
      if (e.res) v += ldf((const T*)e.res + ia);
      if (e.dact != ACT_NONE) v *= act_deriv(e.dact, ldf((const T*)e.dact_src + ia));
      long long ic = (long long)m * g.ldc + n;
      if (g.c_f32) ((float*)g.C)[ic] = v; else stf((T*)g.C + ic, v);
    }
  }
}

template <typename T>
static cudaError_t gemm_simt_t(const GemmArgs& g, cudaStream_t s) {
  dim3 grid(cdiv(g.N, 64), cdiv(g.M, 64), g.splits);
  bool ak = g.sa_k == 1, bk = g.sb_k == 1;
  if (ak && bk) gemm_simt_kernel<T, true, true><<<grid, 256, 0, s>>>(g);
  else if (ak && !bk) gemm_simt_kernel<T, true, false><<<grid, 256, 0, s>>>(g);
  else if (!ak && bk) gemm_simt_kernel<T, false, true><<<grid, 256, 0, s>>>(g);
  else gemm_simt_kernel<T, false, false><<<grid, 256, 0, s>>>(g);
  return cudaGetLastError();
}

cudaError_t gemm_simt(const GemmArgs& g, bool bf16, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
  return bf16 ? gemm_simt_t<bf16_t>(g, s) : gemm_simt_t<float>(g, s);
}

// one thread writes the GPU's nanosecond clock: a phase boundary that can be captured into a graph
__global__ void stamp_kernel(unsigned long long* slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  *slot = t;
}
cudaError_t stamp_time(unsigned long long* slot, cudaStream_t s) {
  stamp_kernel<<<1, 1, 0, s>>>(slot);
  return cudaGetLastError();
}

template <bool BF16_OUT>
__global__ void splitk_reduce_kernel(const float* __restrict__ ws, int splits, long long mn, int N,
                                     void* __restrict__ out, long long ldo) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= mn) return;
  float a = 0.f;
  for (int s = 0; s < splits; s++) a += ws[(long long)s * mn + i];
  const long long o = (i / N) * ldo + (i % N);
  if (BF16_OUT) ((bf16_t*)out)[o] = __float2bfloat16_rn(a);
  else ((float*)out)[o] = a;
}

// four adjacent columns per thread (N, ldo multiples of 4); the partials of up to four splits are in flight at once
template <bool BF16_OUT>
__device__ __forceinline__ void splitk_reduce_v4_body(const float4* __restrict__ ws, int splits, long long mn4, int N4,
                                                      void* __restrict__ out, long long ldo, long long i) {
  if (i >= mn4) return;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < splits; s0 += 4) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; u++) v[u] = s0 + u < splits ? __ldcs(ws + (long long)(s0 + u) * mn4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < 4; u++)
      if (s0 + u < splits) { a.x += v[u].x; a.y += v[u].y; a.z += v[u].z; a.w += v[u].w; }
  }
  const long long o = (i / N4) * ldo + (i % N4) * 4;
  if (BF16_OUT) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
    uint2 q;
    q.x = *reinterpret_cast<uint32_t*>(&lo);
    q.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>((bf16_t*)out + o) = q;
  } else {
    *reinterpret_cast<float4*>((float*)out + o) = a;
  }
}
template <bool BF16_OUT>
__global__ void splitk_reduce_v4_kernel(const float4* __restrict__ ws, int splits, long long mn4, int N4,
                                        void* __restrict__ out, long long ldo) {
  splitk_reduce_v4_body<BF16_OUT>(ws, splits, mn4, N4, out, ldo, (long long)blockIdx.x * blockDim.x + threadIdx.x);
}

cudaError_t splitk_reduce(const float* ws, int splits, long long mn, int N, void* out, long long ldo,
                          cudaStream_t s, bool out_bf16) {
  if (mn <= 0) return cudaSuccess;
  const bool vec = N % 4 == 0 && ldo % 4 == 0 && (reinterpret_cast<uintptr_t>(ws) & 15) == 0 &&
                   (reinterpret_cast<uintptr_t>(out) & 15) == 0;
  if (vec) {
    const long long mn4 = mn / 4;
    if (out_bf16) splitk_reduce_v4_kernel<true><<<cdiv(mn4, 256), 256, 0, s>>>((const float4*)ws, splits, mn4, N / 4, out, ldo);
    else splitk_reduce_v4_kernel<false><<<cdiv(mn4, 256), 256, 0, s>>>((const float4*)ws, splits, mn4, N / 4, out, ldo);
  } else {
    if (out_bf16) splitk_reduce_kernel<true><<<cdiv(mn, 256), 256, 0, s>>>(ws, splits, mn, N, out, ldo);
    else splitk_reduce_kernel<false><<<cdiv(mn, 256), 256, 0, s>>>(ws, splits, mn, N, out, ldo);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// column sums (bias gradients, head weight gradient of the BCE head)
// A CTA sums a strip of 64 columns over one chunk of the rows (a thread owns two adjacent
// columns: one 4-byte load per bf16 pair, 128 bytes per warp and row); the chunk partials go to
// ws and the last CTA of a strip to finish (atomic ticket) adds them in chunk order, so the
// result does not depend on which CTA that is.  The ticket counter is left at zero again.
// ------------------------------------------------------------------------------------------
int colsum_chunks(int rows, int cols) {
  int strips = (cols + 127) / 128;   // at least as many strips as either element type uses
  int want = (592 + strips - 1) / strips;
  int maxc = rows / 64;
  if (maxc < 1) maxc = 1;
  if (want > maxc) want = maxc;
  if (want < 1) want = 1;
  return want;
}

template <typename T> __device__ __forceinline__ float2 ld2(const T* p, bool vec);
template <> __device__ __forceinline__ float2 ld2<float>(const float* p, bool vec) {
  if (vec) return *reinterpret_cast<const float2*>(p);
  return make_float2(p[0], p[1]);
}
template <> __device__ __forceinline__ float2 ld2<bf16_t>(const bf16_t* p, bool vec) {
  if (vec) return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
  return make_float2(__bfloat162float(p[0]), __bfloat162float(p[1]));
}

// sum_{k < chunks} p[k*stride] added in the order k = 0, 1, ..; eight loads are issued before the
// first add so that the final pass costs one memory latency per eight partials, not per partial.
__device__ __forceinline__ float ordered_sum(const float* p, long long stride, int chunks) {
  float t = 0.f;
  for (int k0 = 0; k0 < chunks; k0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; u++) v[u] = k0 + u < chunks ? __ldcg(p + (long long)(k0 + u) * stride) : 0.f;
#pragma unroll
    for (int u = 0; u < 8; u++) if (k0 + u < chunks) t += v[u];
  }
  return t;
}

// Shared tail of the two-stage reductions: returns true in the CTA that arrives last on `ticket`.
__device__ __forceinline__ bool last_cta(int* ticket, int expected) {
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    int t = atomicAdd(ticket, 1);
    s_last = (t == expected - 1);
    if (s_last) *ticket = 0;
  }
  __syncthreads();
  if (s_last) __threadfence();
  return s_last != 0;
}

template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int N = 4; };
template <> struct VecOf<bf16_t> { static constexpr int N = 8; };

// 16 bytes = VecOf<T>::N consecutive elements -> floats
template <typename T> __device__ __forceinline__ void ld_vec(const T* p, float* out);
template <> __device__ __forceinline__ void ld_vec<float>(const float* p, float* out) {
  const float4 q = *reinterpret_cast<const float4*>(p);
  out[0] = q.x; out[1] = q.y; out[2] = q.z; out[3] = q.w;
}
template <> __device__ __forceinline__ void ld_vec<bf16_t>(const bf16_t* p, float* out) {
  const uint4 q = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int j = 0; j < 4; j++) {
    out[2 * j] = __uint_as_float(w[j] << 16);
    out[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
  }
}

// A CTA sums a strip of 32*VEC columns over one chunk of rows: a thread owns VEC adjacent
// columns (one 16-byte load per row) and every 8th row, four rows in flight.
// bx = column strip, by = row chunk of this CTA (the grid of the plain kernel, or what the batched
// kernel derived from its job table).
template <typename T>
__device__ __forceinline__ void colsum_body(const T* __restrict__ X, long long ldx, int rows,
                                            int cols, const float* __restrict__ scale,
                                            float* __restrict__ ws, float* __restrict__ out, int chunks,
                                            int dact, const float* __restrict__ colscale, int* tickets, int bx, int by,
                                            float* smem) {   // 8 * 32*VEC floats
  constexpr int VEC = VecOf<T>::N;
  constexpr int SW = 32 * VEC;  // strip width
  float (*sm)[SW] = reinterpret_cast<float (*)[SW]>(smem);
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int c = bx * SW + cx * VEC;
  const int per = (rows + chunks - 1) / chunks;
  const int rb = by * per, re = min(rows, rb + per);
  const bool vec = X && (c + VEC <= cols) && (ldx % VEC == 0) && ((reinterpret_cast<uintptr_t>(X) & 15) == 0);
  float a[VEC];
#pragma unroll
  for (int j = 0; j < VEC; j++) a[j] = 0.f;
  if (c < cols) {
    if (vec) {
      int r = rb + ry;
      for (; r + 24 < re; r += 32) {
        float v[4][VEC];
#pragma unroll
        for (int u = 0; u < 4; u++) ld_vec<T>(X + (long long)(r + 8 * u) * ldx + c, v[u]);
#pragma unroll
        for (int u = 0; u < 4; u++) {
          const float sc = scale ? scale[r + 8 * u] : 1.f;
#pragma unroll
          for (int j = 0; j < VEC; j++) {
            float t = v[u][j];
            if (dact != ACT_NONE) t = act_deriv(dact, t);
            a[j] = fmaf(t, sc, a[j]);
          }
        }
      }
      for (; r < re; r += 8) {
        float v[VEC];
        ld_vec<T>(X + (long long)r * ldx + c, v);
        const float sc = scale ? scale[r] : 1.f;
#pragma unroll
        for (int j = 0; j < VEC; j++) {
          float t = v[j];
          if (dact != ACT_NONE) t = act_deriv(dact, t);
          a[j] = fmaf(t, sc, a[j]);
        }
      }
    } else {
      for (int r = rb + ry; r < re; r += 8) {
        const float sc = scale ? scale[r] : 1.f;
#pragma unroll
        for (int j = 0; j < VEC; j++) {
          if (c + j < cols) {
            float t = X ? ldf(X + (long long)r * ldx + c + j) : 1.f;
            if (dact != ACT_NONE) t = act_deriv(dact, t);
            a[j] = fmaf(t, sc, a[j]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < VEC; j++) sm[ry][cx * VEC + j] = a[j];
  __syncthreads();
  float* dst = chunks == 1 ? out : ws + (long long)by * cols;
  for (int i = threadIdx.x; i < SW; i += 256) {
    const int cc = bx * SW + i;
    if (cc < cols) {
      float t = 0.f;
#pragma unroll
      for (int k = 0; k < 8; k++) t += sm[k][i];
      if (chunks == 1 && colscale) t *= colscale[cc];
      dst[cc] = t;
    }
  }
  if (chunks == 1) return;
  if (!last_cta(tickets + bx, chunks)) return;
  for (int i = threadIdx.x; i < SW; i += 256) {
    const int cc = bx * SW + i;
    if (cc < cols) {
      float t = ordered_sum(ws + cc, cols, chunks);
      if (colscale) t *= colscale[cc];
      out[cc] = t;
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) colsum_kernel(const T* __restrict__ X, long long ldx, int rows,
                                                     int cols, const float* __restrict__ scale,
                                                     float* __restrict__ ws, float* __restrict__ out, int chunks,
                                                     int dact, const float* __restrict__ colscale, int* tickets) {
  __shared__ float smem[8 * 32 * VecOf<T>::N];
  colsum_body<T>(X, ldx, rows, cols, scale, ws, out, chunks, dact, colscale, tickets, blockIdx.x, blockIdx.y, smem);
}

cudaError_t colsum(const void* X, bool x_bf16, long long ldx, int rows, int cols, const float* scale,
                   float* ws, int chunks, int* tickets, float* out, cudaStream_t s, int dact, const float* colscale) {
  if (x_bf16) {
    dim3 grid(cdiv(cols, 256), chunks);
    colsum_kernel<bf16_t><<<grid, 256, 0, s>>>((const bf16_t*)X, ldx, rows, cols, scale, ws, out, chunks, dact, colscale, tickets);
  } else {
    dim3 grid(cdiv(cols, 128), chunks);
    colsum_kernel<float><<<grid, 256, 0, s>>>((const float*)X, ldx, rows, cols, scale, ws, out, chunks, dact, colscale, tickets);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// LayerNorm
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) layernorm_fwd_kernel(const T* __restrict__ x, const float* __restrict__ gain,
                                                            const float* __restrict__ shift, T* __restrict__ y,
                                                            float* __restrict__ mean, float* __restrict__ rstd,
                                                            int rows, int d) {
  int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const T* xr = x + (long long)row * d;
  float s = 0.f;
  for (int c = lane; c < d; c += 32) s += ldf(xr + c);
  float mu = warp_sum(s) / d;
  float q = 0.f;
  for (int c = lane; c < d; c += 32) { float t = ldf(xr + c) - mu; q += t * t; }
  float r = rsqrtf(warp_sum(q) / d + 1e-5f);
  for (int c = lane; c < d; c += 32)
    stf(y + (long long)row * d + c, (ldf(xr + c) - mu) * r * gain[c] + shift[c]);
  if (lane == 0) { mean[row] = mu; rstd[row] = r; }
}

// bf16 rows of d = 256*VPL columns: a lane keeps VPL 16-byte pieces of its row in registers, so the
// row is read once (the generic kernel above walks over it three times, two bytes per lane and load).
template <int VPL>
__global__ void __launch_bounds__(256) layernorm_fwd_vec_kernel(const bf16_t* __restrict__ x, const float* __restrict__ gain,
                                                                const float* __restrict__ shift, bf16_t* __restrict__ y,
                                                                float* __restrict__ mean, float* __restrict__ rstd,
                                                                int rows, int d) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const bf16_t* xr = x + (long long)row * d;
  float v[VPL][8];
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < VPL; k++) {
    ld_vec<bf16_t>(xr + (k * 32 + lane) * 8, v[k]);
#pragma unroll
    for (int j = 0; j < 8; j++) s += v[k][j];
  }
  const float mu = warp_sum(s) / d;
  float q = 0.f;
#pragma unroll
  for (int k = 0; k < VPL; k++)
#pragma unroll
    for (int j = 0; j < 8; j++) { const float t = v[k][j] - mu; q = fmaf(t, t, q); }
  const float r = rsqrtf(warp_sum(q) / d + 1e-5f);
#pragma unroll
  for (int k = 0; k < VPL; k++) {
    const int c = (k * 32 + lane) * 8;
    const float4 g0 = *reinterpret_cast<const float4*>(gain + c), g1 = *reinterpret_cast<const float4*>(gain + c + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(shift + c), b1 = *reinterpret_cast<const float4*>(shift + c + 4);
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    float o[8];
#pragma unroll
    for (int j = 0; j < 8; j++) o[j] = (v[k][j] - mu) * r * gg[j] + bb[j];
    uint4 w;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(o[0], o[1]); w.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(o[2], o[3]); w.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(o[4], o[5]); w.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(o[6], o[7]); w.w = *reinterpret_cast<uint32_t*>(&h);
    *reinterpret_cast<uint4*>(y + (long long)row * d + c) = w;
  }
  if (lane == 0) { mean[row] = mu; rstd[row] = r; }
}

cudaError_t layernorm_fwd(const void* x, const float* gain, const float* shift, void* y, float* mean,
                          float* rstd, int rows, int d, bool bf16, cudaStream_t s) {
  const bool al = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(gain) |
                    reinterpret_cast<uintptr_t>(shift)) & 15) == 0;
  if (bf16 && al && d % 256 == 0 && d <= 1024) {
    const bf16_t* xb = (const bf16_t*)x;
    bf16_t* yb = (bf16_t*)y;
    const unsigned grid = cdiv(rows, 8);
    switch (d / 256) {
      case 1: layernorm_fwd_vec_kernel<1><<<grid, 256, 0, s>>>(xb, gain, shift, yb, mean, rstd, rows, d); break;
      case 2: layernorm_fwd_vec_kernel<2><<<grid, 256, 0, s>>>(xb, gain, shift, yb, mean, rstd, rows, d); break;
      case 3: layernorm_fwd_vec_kernel<3><<<grid, 256, 0, s>>>(xb, gain, shift, yb, mean, rstd, rows, d); break;
      default: layernorm_fwd_vec_kernel<4><<<grid, 256, 0, s>>>(xb, gain, shift, yb, mean, rstd, rows, d); break;
    }
    return cudaGetLastError();
  }
  if (bf16) layernorm_fwd_kernel<bf16_t><<<cdiv(rows, 8), 256, 0, s>>>((const bf16_t*)x, gain, shift, (bf16_t*)y, mean, rstd, rows, d);
  else layernorm_fwd_kernel<float><<<cdiv(rows, 8), 256, 0, s>>>((const float*)x, gain, shift, (float*)y, mean, rstd, rows, d);
  return cudaGetLastError();
}

template <typename T>
__global__ void __launch_bounds__(256) layernorm_bwd_dx_kernel(const T* __restrict__ dy, const T* __restrict__ x,
                                                               const float* __restrict__ gain,
                                                               const float* __restrict__ mean,
                                                               const float* __restrict__ rstd, const T* add,
                                                               T* dx, int rows, int d) {
  int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  long long o = (long long)row * d;
  float mu = mean[row], r = rstd[row];
  float s1 = 0.f, s2 = 0.f;
  for (int c = lane; c < d; c += 32) {
    float g = ldf(dy + o + c) * gain[c];
    float xh = (ldf(x + o + c) - mu) * r;
    s1 += g;
    s2 += g * xh;
  }
  s1 = warp_sum(s1) / d;
  s2 = warp_sum(s2) / d;
  for (int c = lane; c < d; c += 32) {
    float g = ldf(dy + o + c) * gain[c];
    float xh = (ldf(x + o + c) - mu) * r;
    float v = r * (g - s1 - xh * s2);
    if (add) v += ldf(add + o + c);
    stf(dx + o + c, v);
  }
}

// bf16 rows of d = 256*VPL columns: dy and x are read once (16-byte pieces kept in registers)
template <int VPL>
__global__ void __launch_bounds__(256) layernorm_bwd_dx_vec_kernel(const bf16_t* __restrict__ dy, const bf16_t* __restrict__ x,
                                                                   const float* __restrict__ gain,
                                                                   const float* __restrict__ mean,
                                                                   const float* __restrict__ rstd, const bf16_t* add,
                                                                   bf16_t* dx, int rows, int d) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  const long long o = (long long)row * d;
  const float mu = mean[row], r = rstd[row];
  float g[VPL][8], xh[VPL][8];
  float s1 = 0.f, s2 = 0.f;
#pragma unroll
  for (int k = 0; k < VPL; k++) {
    const int c = (k * 32 + lane) * 8;
    ld_vec<bf16_t>(dy + o + c, g[k]);
    ld_vec<bf16_t>(x + o + c, xh[k]);
    const float4 g0 = *reinterpret_cast<const float4*>(gain + c), g1 = *reinterpret_cast<const float4*>(gain + c + 4);
    const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
    for (int j = 0; j < 8; j++) {
      g[k][j] *= gg[j];
      xh[k][j] = (xh[k][j] - mu) * r;
      s1 += g[k][j];
      s2 += g[k][j] * xh[k][j];
    }
  }
  s1 = warp_sum(s1) / d;
  s2 = warp_sum(s2) / d;
#pragma unroll
  for (int k = 0; k < VPL; k++) {
    const int c = (k * 32 + lane) * 8;
    float v[8], a[8];
    if (add) ld_vec<bf16_t>(add + o + c, a);
#pragma unroll
    for (int j = 0; j < 8; j++) {
      v[j] = r * (g[k][j] - s1 - xh[k][j] * s2);
      if (add) v[j] += a[j];
    }
    uint4 w;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(v[0], v[1]); w.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[2], v[3]); w.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[4], v[5]); w.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[6], v[7]); w.w = *reinterpret_cast<uint32_t*>(&h);
    *reinterpret_cast<uint4*>(dx + o + c) = w;
  }
}

cudaError_t layernorm_bwd_dx(const void* dy, const void* x, const float* gain, const float* mean,
                             const float* rstd, const void* add, void* dx, int rows, int d, bool bf16,
                             cudaStream_t s) {
  const bool al = ((reinterpret_cast<uintptr_t>(dy) | reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(gain) |
                    reinterpret_cast<uintptr_t>(add) | reinterpret_cast<uintptr_t>(dx)) & 15) == 0;
  if (bf16 && al && d % 256 == 0 && d <= 1024) {
    const bf16_t* a = (const bf16_t*)dy; const bf16_t* b = (const bf16_t*)x; const bf16_t* c = (const bf16_t*)add; bf16_t* o = (bf16_t*)dx;
    const unsigned grid = cdiv(rows, 8);
    switch (d / 256) {
      case 1: layernorm_bwd_dx_vec_kernel<1><<<grid, 256, 0, s>>>(a, b, gain, mean, rstd, c, o, rows, d); break;
      case 2: layernorm_bwd_dx_vec_kernel<2><<<grid, 256, 0, s>>>(a, b, gain, mean, rstd, c, o, rows, d); break;
      case 3: layernorm_bwd_dx_vec_kernel<3><<<grid, 256, 0, s>>>(a, b, gain, mean, rstd, c, o, rows, d); break;
      default: layernorm_bwd_dx_vec_kernel<4><<<grid, 256, 0, s>>>(a, b, gain, mean, rstd, c, o, rows, d); break;
    }
    return cudaGetLastError();
  }
  if (bf16) layernorm_bwd_dx_kernel<bf16_t><<<cdiv(rows, 8), 256, 0, s>>>((const bf16_t*)dy, (const bf16_t*)x, gain, mean, rstd, (const bf16_t*)add, (bf16_t*)dx, rows, d);
  else layernorm_bwd_dx_kernel<float><<<cdiv(rows, 8), 256, 0, s>>>((const float*)dy, (const float*)x, gain, mean, rstd, (const float*)add, (float*)dx, rows, d);
  return cudaGetLastError();
}

// dgain / dshift partial sums: a CTA takes a strip of 32*VEC columns and one chunk of rows, a thread
// VEC adjacent columns (16-byte loads of dy and x) and every 8th row, four rows in flight.
template <typename T>
__device__ __forceinline__ void layernorm_param_grad_body(const T* __restrict__ dy, const T* __restrict__ x,
                                                          const float* __restrict__ mean,
                                                          const float* __restrict__ rstd,
                                                          float* __restrict__ ws, float* __restrict__ dgain,
                                                          float* __restrict__ dshift, int rows, int d, int chunks,
                                                          int* tickets, int bx, int by, float* smem) {   // 16 * 32*VEC floats
  constexpr int VEC = VecOf<T>::N;
  constexpr int SW = 32 * VEC;
  float (*sg)[SW] = reinterpret_cast<float (*)[SW]>(smem);
  float (*sb)[SW] = reinterpret_cast<float (*)[SW]>(smem + 8 * SW);
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int c = bx * SW + cx * VEC;
  const int per = (rows + chunks - 1) / chunks;
  const int rb = by * per, re = min(rows, rb + per);
  const bool vec = (c + VEC <= d) && (d % VEC == 0);
  float ag[VEC], ab[VEC];
#pragma unroll
  for (int j = 0; j < VEC; j++) ag[j] = ab[j] = 0.f;
  if (c < d) {
    if (vec) {
      int r = rb + ry;
      for (; r + 24 < re; r += 32) {
        float gy[4][VEC], xv[4][VEC], mu[4], rs[4];
#pragma unroll
        for (int u = 0; u < 4; u++) {
          ld_vec<T>(dy + (long long)(r + 8 * u) * d + c, gy[u]);
          ld_vec<T>(x + (long long)(r + 8 * u) * d + c, xv[u]);
          mu[u] = mean[r + 8 * u];
          rs[u] = rstd[r + 8 * u];
        }
#pragma unroll
        for (int u = 0; u < 4; u++)
#pragma unroll
          for (int j = 0; j < VEC; j++) {
            ag[j] = fmaf(gy[u][j], (xv[u][j] - mu[u]) * rs[u], ag[j]);
            ab[j] += gy[u][j];
          }
      }
      for (; r < re; r += 8) {
        float gy[VEC], xv[VEC];
        ld_vec<T>(dy + (long long)r * d + c, gy);
        ld_vec<T>(x + (long long)r * d + c, xv);
        const float mu = mean[r], rs = rstd[r];
#pragma unroll
        for (int j = 0; j < VEC; j++) {
          ag[j] = fmaf(gy[j], (xv[j] - mu) * rs, ag[j]);
          ab[j] += gy[j];
        }
      }
    } else {
      for (int r = rb + ry; r < re; r += 8) {
        const float mu = mean[r], rs = rstd[r];
#pragma unroll
        for (int j = 0; j < VEC; j++)
          if (c + j < d) {
            const float g = ldf(dy + (long long)r * d + c + j);
            ag[j] = fmaf(g, (ldf(x + (long long)r * d + c + j) - mu) * rs, ag[j]);
            ab[j] += g;
          }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < VEC; j++) { sg[ry][cx * VEC + j] = ag[j]; sb[ry][cx * VEC + j] = ab[j]; }
  __syncthreads();
  float* pg = chunks == 1 ? dgain : ws + (long long)by * d;
  float* pb = chunks == 1 ? dshift : ws + (long long)(chunks + by) * d;
  for (int i = threadIdx.x; i < SW; i += 256) {
    const int cc = bx * SW + i;
    if (cc < d) {
      float tg = 0.f, tb = 0.f;
#pragma unroll
      for (int k = 0; k < 8; k++) { tg += sg[k][i]; tb += sb[k][i]; }
      pg[cc] = tg;
      pb[cc] = tb;
    }
  }
  if (chunks == 1) return;
  if (!last_cta(tickets + bx, chunks)) return;
  for (int i = threadIdx.x; i < SW; i += 256) {
    const int cc = bx * SW + i;
    if (cc < d) {
      dgain[cc] = ordered_sum(ws + cc, d, chunks);
      dshift[cc] = ordered_sum(ws + (long long)chunks * d + cc, d, chunks);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256) layernorm_param_grad_kernel(const T* __restrict__ dy, const T* __restrict__ x,
                                                                   const float* __restrict__ mean,
                                                                   const float* __restrict__ rstd,
                                                                   float* __restrict__ ws, float* __restrict__ dgain,
                                                                   float* __restrict__ dshift, int rows, int d, int chunks,
                                                                   int* tickets) {
  __shared__ float smem[16 * 32 * VecOf<T>::N];
  layernorm_param_grad_body<T>(dy, x, mean, rstd, ws, dgain, dshift, rows, d, chunks, tickets, blockIdx.x, blockIdx.y, smem);
}

// Several column reductions in ONE launch: the bias gradients and LayerNorm gain/shift gradients of
// a block are each a few MB of input, so separate launches spend most of their time ramping up and
// waiting for their last CTA.  A CTA looks its job up in a table (at most a few entries) and then
// runs exactly the code of the single-job kernels on the same partition: same bits.
__global__ void __launch_bounds__(256, 4) reduce_batch_kernel(const ReduceJob* __restrict__ jobs, int njobs) {
  __shared__ float smem[16 * 256];   // the largest need: gain and shift partials of a 256-column bf16 strip
  int j = 0;
  while (j + 1 < njobs && (int)blockIdx.x >= jobs[j + 1].cta_begin) j++;
  const ReduceJob job = jobs[j];
  const int local = (int)blockIdx.x - job.cta_begin;
  const int bx = local % job.strips, by = local / job.strips;
  if (job.kind == 2) {   // split-K partials -> fp32 result, 1024 outputs per CTA
    splitk_reduce_v4_body<false>((const float4*)job.X, job.rows, job.mn / 4, job.cols / 4, job.out0, job.ldx,
                                 (long long)local * 256 + threadIdx.x);
    return;
  }
  if (job.kind == 0) {
    if (job.x_f32)
      colsum_body<float>((const float*)job.X, job.ldx, job.rows, job.cols, job.a, job.ws, job.out0, job.chunks, job.dact, job.b, job.tickets, bx, by, smem);
    else
      colsum_body<bf16_t>((const bf16_t*)job.X, job.ldx, job.rows, job.cols, job.a, job.ws, job.out0, job.chunks, job.dact, job.b, job.tickets, bx, by, smem);
  } else {
    if (job.x_f32)
      layernorm_param_grad_body<float>((const float*)job.X, (const float*)job.X2, job.a, job.b, job.ws, job.out0, job.out1, job.rows, job.cols, job.chunks, job.tickets, bx, by, smem);
    else
      layernorm_param_grad_body<bf16_t>((const bf16_t*)job.X, (const bf16_t*)job.X2, job.a, job.b, job.ws, job.out0, job.out1, job.rows, job.cols, job.chunks, job.tickets, bx, by, smem);
  }
}

int reduce_job_strips(const ReduceJob& j) {
  if (j.kind == 2) return (int)cdiv(j.mn / 4, 256);
  return (int)cdiv(j.cols, j.x_f32 ? 128 : 256);
}

cudaError_t reduce_batch(const ReduceJob* jobs_dev, int njobs, int total_ctas, cudaStream_t s) {
  if (njobs <= 0 || total_ctas <= 0) return cudaSuccess;
  reduce_batch_kernel<<<total_ctas, 256, 0, s>>>(jobs_dev, njobs);
  return cudaGetLastError();
}

cudaError_t layernorm_param_grad(const void* dy, const void* x, const float* mean, const float* rstd,
                                 float* ws, int chunks, int* tickets, float* dgain, float* dshift, int rows, int d,
                                 bool bf16, cudaStream_t s) {
  dim3 grid(cdiv(d, bf16 ? 256 : 128), chunks);
  if (bf16) layernorm_param_grad_kernel<bf16_t><<<grid, 256, 0, s>>>((const bf16_t*)dy, (const bf16_t*)x, mean, rstd, ws, dgain, dshift, rows, d, chunks, tickets);
  else layernorm_param_grad_kernel<float><<<grid, 256, 0, s>>>((const float*)dy, (const float*)x, mean, rstd, ws, dgain, dshift, rows, d, chunks, tickets);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// causal attention, flash-style (no T x T matrix in memory), fp32 SIMT
// tiles of 32 queries x 32 keys; a warp owns 4 rows; lanes run over the 32 keys of a tile for
// the scores and over head columns (lane, lane+32, ..) for the accumulators.
// ------------------------------------------------------------------------------------------
#define ATT_MAXC 4  // head width <= 128

template <typename T>
__device__ __forceinline__ void att_load_tile(float* dst, int ldk, const T* src, long long ld, int r0,
                                              int T_, int dh) {
  for (int i = threadIdx.x; i < 32 * dh; i += 256) {
    int r = i / dh, c = i - r * dh;
    int t = r0 + r;
    dst[r * ldk + c] = t < T_ ? ldf(src + (long long)t * ld + c) : 0.f;
  }
}

template <typename T>
__global__ void __launch_bounds__(256) attn_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ o,
                                                       float* __restrict__ lse, int T_, int H, int dh,
                                                       float scale) {
  extern __shared__ float sm[];
  const int ldk = dh + 1;
  float* Qs = sm;
  float* Ks = Qs + 32 * ldk;
  float* Vs = Ks + 32 * ldk;
  const int q0 = blockIdx.x * 32, h = blockIdx.y, b = blockIdx.z;
  const int d = H * dh;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* base = qkv + (long long)b * T_ * ld + h * dh;
  att_load_tile(Qs, ldk, base, ld, q0, T_, dh);
  float mrow[4], lrow[4], acc[4][ATT_MAXC];
#pragma unroll
  for (int r = 0; r < 4; r++) {
    mrow[r] = -INFINITY;
    lrow[r] = 0.f;
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) acc[r][cc] = 0.f;
  }
  for (int j0 = 0; j0 <= q0; j0 += 32) {
    __syncthreads();
    att_load_tile(Ks, ldk, base + d, ld, j0, T_, dh);
    att_load_tile(Vs, ldk, base + 2 * d, ld, j0, T_, dh);
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; r++) {
      const int il = warp * 4 + r, i = q0 + il;
      if (i >= T_) continue;
      const int j = j0 + lane;
      float sc = 0.f;
      for (int c = 0; c < dh; c++) sc = fmaf(Qs[il * ldk + c], Ks[lane * ldk + c], sc);
      sc *= scale;
      const bool valid = j <= i;
      if (!valid) sc = -INFINITY;
      float mnew = fmaxf(mrow[r], warp_max(sc));
      float p = valid ? expf(sc - mnew) : 0.f;
      float corr = expf(mrow[r] - mnew);
      lrow[r] = lrow[r] * corr + warp_sum(p);
      mrow[r] = mnew;
#pragma unroll
      for (int cc = 0; cc < ATT_MAXC; cc++) acc[r][cc] *= corr;
      for (int jj = 0; jj < 32; jj++) {
        float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
        for (int cc = 0; cc < ATT_MAXC; cc++) {
          int c = lane + 32 * cc;
          if (c < dh) acc[r][cc] = fmaf(pj, Vs[jj * ldk + c], acc[r][cc]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int i = q0 + warp * 4 + r;
    if (i >= T_) continue;
    float inv = 1.f / lrow[r];
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) {
      int c = lane + 32 * cc;
      if (c < dh) stf(o + ((long long)b * T_ + i) * d + h * dh + c, acc[r][cc] * inv);
    }
    if (lane == 0) lse[((long long)b * H + h) * T_ + i] = mrow[r] + logf(lrow[r]);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) attn_delta_kernel(const T* __restrict__ o, const T* __restrict__ dout,
                                                         float* __restrict__ delta, int rows, int T_, int H,
                                                         int dh) {
  // one warp per (row, head)
  long long w = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  int lane = threadIdx.x & 31;
  if (w >= (long long)rows * H) return;
  int n = (int)(w / H), h = (int)(w % H);
  long long off = (long long)n * H * dh + h * dh;
  float s = 0.f;
  for (int c = lane; c < dh; c += 32) s += ldf(o + off + c) * ldf(dout + off + c);
  s = warp_sum(s);
  if (lane == 0) {
    int b = n / T_, t = n % T_;
    delta[((long long)b * H + h) * T_ + t] = s;
  }
}

// dK, dV for a tile of 32 keys: loop over the query tiles at or after it.
template <typename T>
__global__ void __launch_bounds__(256) attn_bwd_kv_kernel(const T* __restrict__ qkv, const T* __restrict__ dout,
                                                          const float* __restrict__ lse,
                                                          const float* __restrict__ delta, T* __restrict__ dqkv,
                                                          int T_, int H, int dh, float scale) {
  extern __shared__ float sm[];
  const int ldk = dh + 1;
  float* Ks = sm;
  float* Vs = Ks + 32 * ldk;
  float* Qs = Vs + 32 * ldk;
  float* Ds = Qs + 32 * ldk;
  float* Ls = Ds + 32 * ldk;  // [32] lse
  float* Es = Ls + 32;        // [32] delta
  const int k0 = blockIdx.x * 32, h = blockIdx.y, b = blockIdx.z;
  const int d = H * dh;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* base = qkv + (long long)b * T_ * ld + h * dh;
  const T* dob = dout + (long long)b * T_ * d + h * dh;
  att_load_tile(Ks, ldk, base + d, ld, k0, T_, dh);
  att_load_tile(Vs, ldk, base + 2 * d, ld, k0, T_, dh);
  float dk[4][ATT_MAXC], dv[4][ATT_MAXC];
#pragma unroll
  for (int r = 0; r < 4; r++)
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) dk[r][cc] = dv[r][cc] = 0.f;
  for (int i0 = k0; i0 < T_; i0 += 32) {
    __syncthreads();
    att_load_tile(Qs, ldk, base, ld, i0, T_, dh);
    att_load_tile(Ds, ldk, dob, (long long)d, i0, T_, dh);
    if (threadIdx.x < 32) {
      int i = i0 + threadIdx.x;
      Ls[threadIdx.x] = i < T_ ? lse[((long long)b * H + h) * T_ + i] : 0.f;
      Es[threadIdx.x] = i < T_ ? delta[((long long)b * H + h) * T_ + i] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; r++) {
      const int jl = warp * 4 + r, j = k0 + jl;
      if (j >= T_) continue;
      const int i = i0 + lane;
      float sc = 0.f, dp = 0.f;
      for (int c = 0; c < dh; c++) {
        sc = fmaf(Qs[lane * ldk + c], Ks[jl * ldk + c], sc);
        dp = fmaf(Ds[lane * ldk + c], Vs[jl * ldk + c], dp);
      }
      const bool valid = i < T_ && j <= i;
      float p = valid ? expf(sc * scale - Ls[lane]) : 0.f;
      float ds = p * (dp - Es[lane]);
      for (int ii = 0; ii < 32; ii++) {
        float pi = __shfl_sync(0xffffffffu, p, ii);
        float di = __shfl_sync(0xffffffffu, ds, ii);
#pragma unroll
        for (int cc = 0; cc < ATT_MAXC; cc++) {
          int c = lane + 32 * cc;
          if (c < dh) {
            dv[r][cc] = fmaf(pi, Ds[ii * ldk + c], dv[r][cc]);
            dk[r][cc] = fmaf(di, Qs[ii * ldk + c], dk[r][cc]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int j = k0 + warp * 4 + r;
    if (j >= T_) continue;
    T* row = dqkv + ((long long)b * T_ + j) * ld + h * dh;
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) {
      int c = lane + 32 * cc;
      if (c < dh) {
        stf(row + d + c, dk[r][cc] * scale);
        stf(row + 2 * d + c, dv[r][cc]);
      }
    }
  }
}

// dQ for a tile of 32 queries: loop over the key tiles at or before it.
template <typename T>
__global__ void __launch_bounds__(256) attn_bwd_q_kernel(const T* __restrict__ qkv, const T* __restrict__ dout,
                                                         const float* __restrict__ lse,
                                                         const float* __restrict__ delta, T* __restrict__ dqkv,
                                                         int T_, int H, int dh, float scale) {
  extern __shared__ float sm[];
  const int ldk = dh + 1;
  float* Qs = sm;
  float* Ds = Qs + 32 * ldk;
  float* Ks = Ds + 32 * ldk;
  float* Vs = Ks + 32 * ldk;
  const int q0 = blockIdx.x * 32, h = blockIdx.y, b = blockIdx.z;
  const int d = H * dh;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const T* base = qkv + (long long)b * T_ * ld + h * dh;
  const T* dob = dout + (long long)b * T_ * d + h * dh;
  att_load_tile(Qs, ldk, base, ld, q0, T_, dh);
  att_load_tile(Ds, ldk, dob, (long long)d, q0, T_, dh);
  float dq[4][ATT_MAXC], lrow[4], erow[4];
#pragma unroll
  for (int r = 0; r < 4; r++) {
    int i = q0 + warp * 4 + r;
    lrow[r] = i < T_ ? lse[((long long)b * H + h) * T_ + i] : 0.f;
    erow[r] = i < T_ ? delta[((long long)b * H + h) * T_ + i] : 0.f;
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) dq[r][cc] = 0.f;
  }
  for (int j0 = 0; j0 <= q0; j0 += 32) {
    __syncthreads();
    att_load_tile(Ks, ldk, base + d, ld, j0, T_, dh);
    att_load_tile(Vs, ldk, base + 2 * d, ld, j0, T_, dh);
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; r++) {
      const int il = warp * 4 + r, i = q0 + il;
      if (i >= T_) continue;
      const int j = j0 + lane;
      float sc = 0.f, dp = 0.f;
      for (int c = 0; c < dh; c++) {
        sc = fmaf(Qs[il * ldk + c], Ks[lane * ldk + c], sc);
        dp = fmaf(Ds[il * ldk + c], Vs[lane * ldk + c], dp);
      }
      float p = j <= i ? expf(sc * scale - lrow[r]) : 0.f;
      float ds = p * (dp - erow[r]);
      for (int jj = 0; jj < 32; jj++) {
        float dj = __shfl_sync(0xffffffffu, ds, jj);
#pragma unroll
        for (int cc = 0; cc < ATT_MAXC; cc++) {
          int c = lane + 32 * cc;
          if (c < dh) dq[r][cc] = fmaf(dj, Ks[jj * ldk + c], dq[r][cc]);
        }
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 4; r++) {
    const int i = q0 + warp * 4 + r;
    if (i >= T_) continue;
    T* row = dqkv + ((long long)b * T_ + i) * ld + h * dh;
#pragma unroll
    for (int cc = 0; cc < ATT_MAXC; cc++) {
      int c = lane + 32 * cc;
      if (c < dh) stf(row + c, dq[r][cc] * scale);
    }
  }
}

template <typename K>
static cudaError_t set_smem(K kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

template <typename T>
static cudaError_t attention_fwd_t(const T* qkv, T* o, float* lse, int batch, int T_, int heads, int dh,
                                   cudaStream_t s) {
  size_t smem = (size_t)3 * 32 * (dh + 1) * sizeof(float);
  cudaError_t e = set_smem(attn_fwd_kernel<T>, smem);
  if (e != cudaSuccess) return e;
  dim3 grid(cdiv(T_, 32), heads, batch);
  attn_fwd_kernel<T><<<grid, 256, smem, s>>>(qkv, o, lse, T_, heads, dh, 1.f / sqrtf((float)dh));
  return cudaGetLastError();
}

// 0: fp32 SIMT / mma.sync kernels only; 1 (default): tcgen05 kernels where they apply
static int attention_tc_mode() { return getenv("ERASE_ATTN_TC") ? atoi(getenv("ERASE_ATTN_TC")) : 1; }

cudaError_t attention_fwd(const void* qkv, void* o, float* lse, int batch, int T_, int heads, int dh,
                          bool bf16, cudaStream_t s, int* status) {
  if (dh > 32 * ATT_MAXC) return cudaErrorInvalidValue;
  if (bf16 && attention_tc_mode() && attention_tc_supported(dh, heads * dh, qkv, o))
    return attention_fwd_tc(qkv, o, lse, batch, T_, heads, status, s);
  if (bf16 && attention_mma_supported(dh, heads * dh)) return attention_fwd_mma(qkv, o, lse, batch, T_, heads, s);
  return bf16 ? attention_fwd_t<bf16_t>((const bf16_t*)qkv, (bf16_t*)o, lse, batch, T_, heads, dh, s)
              : attention_fwd_t<float>((const float*)qkv, (float*)o, lse, batch, T_, heads, dh, s);
}

template <typename T>
static cudaError_t attention_bwd_t(const T* qkv, const T* o, const T* dout, const float* lse, float* delta,
                                   T* dqkv, int batch, int T_, int heads, int dh, cudaStream_t s) {
  int rows = batch * T_;
  attn_delta_kernel<T><<<cdiv((long long)rows * heads, 8), 256, 0, s>>>(o, dout, delta, rows, T_, heads, dh);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  size_t smem = ((size_t)4 * 32 * (dh + 1) + 64) * sizeof(float);
  if ((e = set_smem(attn_bwd_kv_kernel<T>, smem)) != cudaSuccess) return e;
  if ((e = set_smem(attn_bwd_q_kernel<T>, smem)) != cudaSuccess) return e;
  dim3 grid(cdiv(T_, 32), heads, batch);
  float scale = 1.f / sqrtf((float)dh);
  attn_bwd_kv_kernel<T><<<grid, 256, smem, s>>>(qkv, dout, lse, delta, dqkv, T_, heads, dh, scale);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  attn_bwd_q_kernel<T><<<grid, 256, smem, s>>>(qkv, dout, lse, delta, dqkv, T_, heads, dh, scale);
  return cudaGetLastError();
}

cudaError_t attention_bwd(const void* qkv, const void* o, const void* dout, const float* lse, float* delta,
                          void* dqkv, int batch, int T_, int heads, int dh, bool bf16, cudaStream_t s, int* status) {
  if (dh > 32 * ATT_MAXC) return cudaErrorInvalidValue;
  if (bf16 && attention_tc_mode() && attention_tc_supported(dh, heads * dh, qkv, dout) && ((reinterpret_cast<uintptr_t>(dqkv) | reinterpret_cast<uintptr_t>(o)) & 15) == 0) {
    return attention_bwd_tc(qkv, o, dout, lse, delta, dqkv, batch, T_, heads, status, s);
  }
  if (bf16 && attention_mma_supported(dh, heads * dh)) return attention_bwd_mma(qkv, o, dout, lse, delta, dqkv, batch, T_, heads, s);
  return bf16 ? attention_bwd_t<bf16_t>((const bf16_t*)qkv, (const bf16_t*)o, (const bf16_t*)dout, lse, delta, (bf16_t*)dqkv, batch, T_, heads, dh, s)
              : attention_bwd_t<float>((const float*)qkv, (const float*)o, (const float*)dout, lse, delta, (float*)dqkv, batch, T_, heads, dh, s);
}

// ------------------------------------------------------------------------------------------
// losses
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float block_reduce_256(float v, float* sm, bool is_max) {
  int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = is_max ? warp_max(v) : warp_sum(v);
  __syncthreads();
  if (lane == 0) sm[warp] = v;
  __syncthreads();
  float r = sm[0];
#pragma unroll
  for (int i = 1; i < 8; i++) r = is_max ? fmaxf(r, sm[i]) : r + sm[i];
  return r;
}

template <typename T>
__global__ void __launch_bounds__(256) softmax_ce_kernel(T* __restrict__ logits, const int32_t* __restrict__ ids,
                                                         int T_, float* __restrict__ rowloss, int V,
                                                         float inv_rows) {
  __shared__ float sm[8];
  const int row = blockIdx.x;
  T* p = logits + (long long)row * V;
  // an id out of range was reported by the input staging; here it must only not be used as an index
  const int tgt = min(max(ids[(long long)(row / T_) * (T_ + 1) + (row % T_) + 1], 0), V - 1);
  const float lt = ldf(p + tgt);
  float mx = -INFINITY;
  for (int v = threadIdx.x; v < V; v += 256) mx = fmaxf(mx, ldf(p + v));
  mx = block_reduce_256(mx, sm, true);
  float se = 0.f;
  for (int v = threadIdx.x; v < V; v += 256) se += expf(ldf(p + v) - mx);
  se = block_reduce_256(se, sm, false);
  const float lse = mx + logf(se);
  __syncthreads();  // lt was read by every thread before any store below
  for (int v = threadIdx.x; v < V; v += 256) {
    float g = expf(ldf(p + v) - lse) - (v == tgt ? 1.f : 0.f);
    stf(p + v, g * inv_rows);
  }
  if (threadIdx.x == 0) rowloss[row] = lse - lt;
}

// bf16 rows kept in registers: one 16-byte load and one 16-byte store per 8 logits, nothing re-read.
// A thread owns vectors tid, tid+THREADS, ...; VPT of them (V <= THREADS*8*VPT, V % 8 == 0).
template <int THREADS, int VPT>
__global__ void __launch_bounds__(THREADS) softmax_ce_reg_kernel(bf16_t* __restrict__ logits,
                                                                  const int32_t* __restrict__ ids, int T_,
                                                                  float* __restrict__ rowloss, int V, float inv_rows) {
  __shared__ float sm[THREADS / 32];
  const int row = blockIdx.x, nvec = V >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint4* p = reinterpret_cast<uint4*>(logits + (long long)row * V);
  const int tgt = ids[(long long)(row / T_) * (T_ + 1) + (row % T_) + 1];
  const float L2E = 1.4426950408889634f;
  float x[VPT][8];
  float mx = -INFINITY, lt = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; k++) {
    const int i = threadIdx.x + k * THREADS;
    if (i < nvec) {
      const uint4 q = p[i];
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; j++) {
        x[k][2 * j] = __uint_as_float(w[j] << 16);
        x[k][2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
      }
#pragma unroll
      for (int j = 0; j < 8; j++) {
        mx = fmaxf(mx, x[k][j]);
        if (i * 8 + j == tgt) lt = x[k][j];
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; j++) x[k][j] = -INFINITY;
    }
  }
  auto block_reduce = [&](float v, bool is_max) {
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    float r = sm[0];
    for (int i = 1; i < THREADS / 32; i++) r = is_max ? fmaxf(r, sm[i]) : r + sm[i];
    return r;
  };
  mx = block_reduce(mx, true);
  float se = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; k++)
#pragma unroll
    for (int j = 0; j < 8; j++) {
      x[k][j] = exp2f((x[k][j] - mx) * L2E);     // keep exp(x - max): the probabilities are this over the sum
      se += x[k][j];
    }
  se = block_reduce(se, false);
  const float lse = mx + logf(se);
  const float inv_se = 1.f / se;
#pragma unroll
  for (int k = 0; k < VPT; k++) {
    const int i = threadIdx.x + k * THREADS;
    if (i < nvec) {
      float g[8];
#pragma unroll
      for (int j = 0; j < 8; j++) g[j] = (x[k][j] * inv_se - (i * 8 + j == tgt ? 1.f : 0.f)) * inv_rows;
      uint4 q;
      __nv_bfloat162 h;
      h = __floats2bfloat162_rn(g[0], g[1]); q.x = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(g[2], g[3]); q.y = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(g[4], g[5]); q.z = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(g[6], g[7]); q.w = *reinterpret_cast<uint32_t*>(&h);
      p[i] = q;
    }
  }
  if ((tgt >> 3) % THREADS == threadIdx.x) rowloss[row] = lse - lt;   // the thread that holds the target logit
}

// Long rows (vocabularies beyond 16 Ki): the row is kept PACKED (bf16 pairs) in registers so
// that two 512-thread CTAs fit on an SM and their load / reduce / store phases overlap; the
// exponentials of the first pass overwrite the logits in place (as bf16) and the second pass only
// scales them, so each element costs one exp.
template <int THREADS, int VPT>
__global__ void __launch_bounds__(THREADS, 2) softmax_ce_packed_kernel(bf16_t* __restrict__ logits,
                                                                       const int32_t* __restrict__ ids, int T_,
                                                                       float* __restrict__ rowloss, int V,
                                                                       float inv_rows) {
  __shared__ float sm[THREADS / 32];
  const int row = blockIdx.x, nvec = V >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint4* p = reinterpret_cast<uint4*>(logits + (long long)row * V);
  const int tgt = ids[(long long)(row / T_) * (T_ + 1) + (row % T_) + 1];
  const float L2E = 1.4426950408889634f;
  uint32_t w[VPT][4];
  float mx = -INFINITY, lt = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; k++) {
    const int i = threadIdx.x + k * THREADS;
    if (i < nvec) {
      const uint4 q = p[i];
      w[k][0] = q.x; w[k][1] = q.y; w[k][2] = q.z; w[k][3] = q.w;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const float lo = __uint_as_float(w[k][j] << 16), hi = __uint_as_float(w[k][j] & 0xffff0000u);
        mx = fmaxf(mx, fmaxf(lo, hi));
        if (i * 8 + 2 * j == tgt) lt = lo;
        if (i * 8 + 2 * j + 1 == tgt) lt = hi;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; j++) w[k][j] = 0xff80ff80u;   // two bf16 -inf
    }
  }
  auto block_reduce = [&](float v, bool is_max) {
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    float r = sm[0];
    for (int i = 1; i < THREADS / 32; i++) r = is_max ? fmaxf(r, sm[i]) : r + sm[i];
    return r;
  };
  mx = block_reduce(mx, true);
  float se = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; k++)
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const float lo = exp2f((__uint_as_float(w[k][j] << 16) - mx) * L2E);
      const float hi = exp2f((__uint_as_float(w[k][j] & 0xffff0000u) - mx) * L2E);
      se += lo + hi;                                       // the sum uses the unrounded exponentials
      __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
      w[k][j] = *reinterpret_cast<uint32_t*>(&h);
    }
  se = block_reduce(se, false);
  const float lse = mx + logf(se);
  const float scale = inv_rows / se;
#pragma unroll
  for (int k = 0; k < VPT; k++) {
    const int i = threadIdx.x + k * THREADS;
    if (i < nvec) {
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; j++) {
        float lo = __uint_as_float(w[k][j] << 16) * scale, hi = __uint_as_float(w[k][j] & 0xffff0000u) * scale;
        if (i * 8 + 2 * j == tgt) lo -= inv_rows;
        if (i * 8 + 2 * j + 1 == tgt) hi -= inv_rows;
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        o[j] = *reinterpret_cast<uint32_t*>(&h);
      }
      p[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  if ((tgt >> 3) % THREADS == threadIdx.x) rowloss[row] = lse - lt;
}

// Persistent variant that also produces the head's bias gradient.  A CTA walks over rows
// blockIdx.x, blockIdx.x + gridDim.x, ...; the next row streams into a shared-memory buffer
// (cp.async) while the current one, held packed in registers, goes through max / exp-sum / scale,
// so the memory system stays busy through the reductions; every thread adds the gradients it
// writes (unrounded, fp32) to column sums it alone owns in shared memory, and the CTA leaves one
// row of partial sums per CTA: colpart[gridDim.x][V].  Their ordered sum over the CTAs is the bias
// gradient -- without reading the rows x V gradient matrix a second time.
// Dynamic shared memory: V*2 bytes (row buffer) + V*4 bytes (column sums).
template <int THREADS, int VPT>
__global__ void __launch_bounds__(THREADS) softmax_ce_fused_kernel(bf16_t* __restrict__ logits,
                                                                    const int32_t* __restrict__ ids, int T_,
                                                                    float* __restrict__ rowloss, float* __restrict__ colpart,
                                                                    int rows, int V, float inv_rows) {
  extern __shared__ __align__(16) uint8_t dyn[];
  __shared__ float sm[THREADS / 32];
  uint4* buf = reinterpret_cast<uint4*>(dyn);
  float* acc = reinterpret_cast<float*>(dyn + (size_t)V * 2);
  const int nvec = V >> 3;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float L2E = 1.4426950408889634f;
  for (int i = threadIdx.x; i < V; i += THREADS) acc[i] = 0.f;
  auto fetch = [&](int row) {
    const uint4* src = reinterpret_cast<const uint4*>(logits + (long long)row * V);
#pragma unroll
    for (int k = 0; k < VPT; k++) {
      const int i = threadIdx.x + k * THREADS;
      if (i < nvec)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(buf + i)), "l"(src + i) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  auto block_reduce = [&](float v, bool is_max) {
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    float r = sm[0];
    for (int i = 1; i < THREADS / 32; i++) r = is_max ? fmaxf(r, sm[i]) : r + sm[i];
    return r;
  };
  int row = blockIdx.x;
  if (row < rows) fetch(row);
  for (; row < rows; row += gridDim.x) {
    uint4* p = reinterpret_cast<uint4*>(logits + (long long)row * V);
    const int tgt = ids[(long long)(row / T_) * (T_ + 1) + (row % T_) + 1];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    uint32_t w[VPT][4];
    float mx = -INFINITY, lt = 0.f;
#pragma unroll
    for (int k = 0; k < VPT; k++) {
      const int i = threadIdx.x + k * THREADS;
      if (i < nvec) {
        const uint4 q = buf[i];
        w[k][0] = q.x; w[k][1] = q.y; w[k][2] = q.z; w[k][3] = q.w;
#pragma unroll
        for (int j = 0; j < 4; j++) {
          const float lo = __uint_as_float(w[k][j] << 16), hi = __uint_as_float(w[k][j] & 0xffff0000u);
          mx = fmaxf(mx, fmaxf(lo, hi));
          if (i * 8 + 2 * j == tgt) lt = lo;
          if (i * 8 + 2 * j + 1 == tgt) lt = hi;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; j++) w[k][j] = 0xff80ff80u;   // two bf16 -inf
      }
    }
    mx = block_reduce(mx, true);                 // its first barrier also says: every thread has read buf
    if (row + (int)gridDim.x < rows) fetch(row + gridDim.x);
    float se = 0.f;
#pragma unroll
    for (int k = 0; k < VPT; k++)
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const float lo = exp2f((__uint_as_float(w[k][j] << 16) - mx) * L2E);
        const float hi = exp2f((__uint_as_float(w[k][j] & 0xffff0000u) - mx) * L2E);
        se += lo + hi;                                       // the sum uses the unrounded exponentials
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
        w[k][j] = *reinterpret_cast<uint32_t*>(&h);
      }
    se = block_reduce(se, false);
    const float lse = mx + logf(se);
    const float scale = inv_rows / se;
#pragma unroll
    for (int k = 0; k < VPT; k++) {
      const int i = threadIdx.x + k * THREADS;
      if (i < nvec) {
        uint32_t o[4];
        float g[8];
#pragma unroll
        for (int j = 0; j < 4; j++) {
          float lo = __uint_as_float(w[k][j] << 16) * scale, hi = __uint_as_float(w[k][j] & 0xffff0000u) * scale;
          if (i * 8 + 2 * j == tgt) lo -= inv_rows;
          if (i * 8 + 2 * j + 1 == tgt) hi -= inv_rows;
          g[2 * j] = lo; g[2 * j + 1] = hi;
          __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
          o[j] = *reinterpret_cast<uint32_t*>(&h);
        }
        p[i] = make_uint4(o[0], o[1], o[2], o[3]);
        float4* a4 = reinterpret_cast<float4*>(acc + i * 8);   // columns i*8 .. i*8+7 belong to this thread alone
        float4 a0 = a4[0], a1 = a4[1];
        a0.x += g[0]; a0.y += g[1]; a0.z += g[2]; a0.w += g[3];
        a1.x += g[4]; a1.y += g[5]; a1.z += g[6]; a1.w += g[7];
        a4[0] = a0; a4[1] = a1;
      }
    }
    if ((tgt >> 3) % THREADS == threadIdx.x) rowloss[row] = lse - lt;
  }
  // this CTA's column sums (zeros if it had no row)
  float4* dst = reinterpret_cast<float4*>(colpart + (long long)blockIdx.x * V);
#pragma unroll
  for (int k = 0; k < VPT; k++) {
    const int i = threadIdx.x + k * THREADS;
    if (i < nvec) {
      const float4* a4 = reinterpret_cast<const float4*>(acc + i * 8);
      dst[2 * i] = a4[0];
      dst[2 * i + 1] = a4[1];
    }
  }
}

int softmax_ce_fused_ctas(int rows) { return rows < 296 ? rows : 296; }

bool softmax_ce_fused_supported(int V, bool bf16, const void* logits) {
  return bf16 && V % 8 == 0 && V / 8 <= 512 * 16 && (size_t)V * 6 <= 200 * 1024 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0;
}

template <int THREADS, int VPT>
static cudaError_t softmax_ce_fused_launch(bf16_t* lg, const int32_t* ids, int T_, float* rowloss, float* colpart, int rows, int V,
                                           float inv_rows, cudaStream_t s) {
  const size_t smem = (size_t)V * 6;
  static size_t attr = 0;
  if (smem > 40 * 1024 && smem > attr) {   // dynamic + static shared memory beyond the 48 KB default
    cudaError_t e = cudaFuncSetAttribute(softmax_ce_fused_kernel<THREADS, VPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr = smem;
  }
  softmax_ce_fused_kernel<THREADS, VPT><<<softmax_ce_fused_ctas(rows), THREADS, smem, s>>>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows);
  return cudaGetLastError();
}

cudaError_t softmax_ce_fused(void* logits, const int32_t* ids, int T_, float* rowloss, float* colpart, int rows, int V,
                             float inv_rows, cudaStream_t s) {
  const int nvec = V / 8;
  bf16_t* lg = (bf16_t*)logits;
  if (nvec <= 256 * 2) return softmax_ce_fused_launch<256, 2>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows, s);
  if (nvec <= 256 * 4) return softmax_ce_fused_launch<256, 4>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows, s);
  if (nvec <= 512 * 4) return softmax_ce_fused_launch<512, 4>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows, s);
  if (nvec <= 512 * 8) return softmax_ce_fused_launch<512, 8>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows, s);
  return softmax_ce_fused_launch<512, 16>(lg, ids, T_, rowloss, colpart, rows, V, inv_rows, s);
}

cudaError_t softmax_ce_inplace(void* logits, const int32_t* ids, int T_, float* rowloss, int rows, int V,
                               float inv_rows, bool bf16, cudaStream_t s) {
  if (bf16 && V % 8 == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0) {
    const int nvec = V / 8;
    bf16_t* lg = (bf16_t*)logits;
    if (nvec <= 256 * 2) { softmax_ce_reg_kernel<256, 2><<<rows, 256, 0, s>>>(lg, ids, T_, rowloss, V, inv_rows); return cudaGetLastError(); }
    if (nvec <= 256 * 4) { softmax_ce_reg_kernel<256, 4><<<rows, 256, 0, s>>>(lg, ids, T_, rowloss, V, inv_rows); return cudaGetLastError(); }
    if (nvec <= 512 * 4) { softmax_ce_packed_kernel<512, 4><<<rows, 512, 0, s>>>(lg, ids, T_, rowloss, V, inv_rows); return cudaGetLastError(); }
    if (nvec <= 512 * 8) { softmax_ce_packed_kernel<512, 8><<<rows, 512, 0, s>>>(lg, ids, T_, rowloss, V, inv_rows); return cudaGetLastError(); }
    if (nvec <= 512 * 16) { softmax_ce_packed_kernel<512, 16><<<rows, 512, 0, s>>>(lg, ids, T_, rowloss, V, inv_rows); return cudaGetLastError(); }
  }
  if (bf16) softmax_ce_kernel<bf16_t><<<rows, 256, 0, s>>>((bf16_t*)logits, ids, T_, rowloss, V, inv_rows);
  else softmax_ce_kernel<float><<<rows, 256, 0, s>>>((float*)logits, ids, T_, rowloss, V, inv_rows);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Softmax cross-entropy head without a pass over the logits (bf16 models, tensor-core head GEMM).
//
// With a per-row reference c_n known BEFORE the head GEMM, the GEMM's epilogue stores
// P[n,v] = exp(l[n,v] - c_n) (bf16) instead of the logit and leaves fp32 partial sums of the
// unrounded exponentials.  Then, with S_n = sum_v exp(l[n,v] - c_n):
//     lse_n = c_n + log S_n,      loss_n = lse_n - l[n,t_n],
//     dl[n,v] = (softmax - onehot)/N = r_n * (P[n,v] - S_n [v = t_n]),     r_n = 1 / (S_n N).
// The finalize kernel therefore patches ONE element per row, P[n,t_n] <- P[n,t_n] - S_n, and from
// then on the gradient of the logits is r (.) P: the backward GEMMs consume P directly,
//     dW_h = P^T (r (.) z),     dz_n = r_n (P W_h)_n,     db_h = sum_n r_n P[n,:].
// c_n is the target's own logit (z_n . W_h[t_n] + b_h[t_n], a gather and a dot product): it is at
// most the row maximum, and it is far enough below it to endanger the exponent range only when the
// token's loss exceeds ~69 nats.  Such rows (S_n >= 1e30 or not finite) are listed by the finalize
// kernel and recomputed exactly, with c_n = the true row maximum, by ce_fixup_kernel, which does
// nothing when the list is empty.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float dot8_bf16(uint4 a, uint4 b) {
  const uint32_t x[4] = {a.x, a.y, a.z, a.w}, y[4] = {b.x, b.y, b.z, b.w};
  float acc = 0.f;
#pragma unroll
  for (int j = 0; j < 4; j++) {
    acc = fmaf(__uint_as_float(x[j] << 16), __uint_as_float(y[j] << 16), acc);
    acc = fmaf(__uint_as_float(x[j] & 0xffff0000u), __uint_as_float(y[j] & 0xffff0000u), acc);
  }
  return acc;
}

// One warp per row: tgt[n] (clamped into the vocabulary; a bad id was already reported by the
// input staging), ref[n] = lt[n] = z_n . W[t_n] + b[t_n].  Thread 0 of the launch clears the
// list of rows to recompute.  d % 8 == 0.
__global__ void __launch_bounds__(256) ce_target_logit_kernel(const bf16_t* __restrict__ z, const bf16_t* __restrict__ W,
                                                              const float* __restrict__ bias, const int32_t* __restrict__ ids,
                                                              int T_, int rows, int d, int V, int* __restrict__ tgt,
                                                              float* __restrict__ ref, float* __restrict__ lt, int* __restrict__ bad) {
  if (blockIdx.x == 0 && threadIdx.x == 0) bad[0] = 0;
  const int lane = threadIdx.x & 31;
  for (int n = blockIdx.x * 8 + (threadIdx.x >> 5); n < rows; n += gridDim.x * 8) {
    const int t = min(max(ids[(long long)(n / T_) * (T_ + 1) + (n % T_) + 1], 0), V - 1);
    const uint4* zr = reinterpret_cast<const uint4*>(z + (long long)n * d);
    const uint4* wr = reinterpret_cast<const uint4*>(W + (long long)t * d);
    float acc = 0.f;
    for (int i = lane; i < (d >> 3); i += 32) acc += dot8_bf16(__ldg(zr + i), __ldg(wr + i));
    acc = warp_sum(acc);
    if (lane == 0) {
      const float l = acc + bias[t];
      tgt[n] = t;
      ref[n] = l;
      lt[n] = l;
    }
  }
}

__device__ __forceinline__ void scale_row_bf16(const bf16_t* __restrict__ z, bf16_t* __restrict__ zs, int d, float r, int lane) {
  const uint4* src = reinterpret_cast<const uint4*>(z);
  uint4* dst = reinterpret_cast<uint4*>(zs);
  for (int i = lane; i < (d >> 3); i += 32) {
    const uint4 q = src[i];
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
      __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(w[j] << 16) * r, __uint_as_float(w[j] & 0xffff0000u) * r);
      o[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    dst[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// The 16 columns behind a scaled row (row stride d + 16): the row scale itself, then zeros.  The weight-gradient
// GEMM multiplies P^T with them too, which makes the head's bias gradient sum_n r_n P[n,:] its 769th column.
__device__ __forceinline__ void scale_row_tail(bf16_t* __restrict__ zs_row, int d, int ldzs, float r, int lane) {
  if (ldzs >= d + 16 && lane < 2) {
    const __nv_bfloat16 rb = __float2bfloat16_rn(r);
    const uint32_t first = lane == 0 ? (uint32_t)(*reinterpret_cast<const unsigned short*>(&rb)) : 0u;
    reinterpret_cast<uint4*>(zs_row + d)[lane] = make_uint4(first, 0u, 0u, 0u);
  }
}

// One warp per row: S_n from the GEMM's partial sums (lanes stride over the groups, then a fixed
// shuffle tree), loss_n, r_n, the patch P[n,t_n] -= S_n, the scaled copy r_n z_n for the
// weight-gradient GEMM; rows whose sum left the safe range are appended to the list bad[1..]
// (count in bad[0]).
__global__ void __launch_bounds__(256) ce_finalize_kernel(const float* __restrict__ psum, int groups, const float* __restrict__ ref,
                                                          const float* __restrict__ lt, const int* __restrict__ tgt,
                                                          bf16_t* __restrict__ P, int V, const bf16_t* __restrict__ z,
                                                          bf16_t* __restrict__ zs, float* __restrict__ rowloss,
                                                          float* __restrict__ rowscale, int* __restrict__ bad, int rows, int d,
                                                          int ldzs, float inv_rows) {
  const int lane = threadIdx.x & 31;
  for (int n = blockIdx.x * 8 + (threadIdx.x >> 5); n < rows; n += gridDim.x * 8) {
    const float* ps = psum + (long long)n * groups;
    float S = 0.f;
    for (int g = lane; g < groups; g += 32) S += ps[g];
    S = warp_sum(S);
    const bool ok = S < 1e30f && S > 0.f;      // false for inf and NaN too
    const float r = ok ? inv_rows / S : 0.f;
    if (lane == 0) {
      rowloss[n] = ok ? ref[n] + logf(S) - lt[n] : 0.f;
      rowscale[n] = r;
      if (ok) P[(long long)n * V + tgt[n]] = __float2bfloat16_rn(expf(lt[n] - ref[n]) - S);   // the one-hot part of the gradient
      else bad[1 + atomicAdd(bad, 1)] = n;
    }
    scale_row_bf16(z + (long long)n * d, zs + (long long)n * ldzs, d, r, lane);
    scale_row_tail(zs + (long long)n * ldzs, d, ldzs, r, lane);
  }
}

// Rows listed by the finalize kernel, one CTA per row at a time: the logits of the row are
// recomputed from z_n and the head's operands (twice: maximum, then exponentials), P[n,:] is
// rewritten relative to the true maximum, and loss_n, r_n and the scaled copy of z_n follow.
// Every quantity of a row depends on that row alone, so the order of the list does not matter.
__global__ void __launch_bounds__(256) ce_fixup_kernel(const int* __restrict__ bad, const int* __restrict__ status, const int* __restrict__ tgt,
                                                       const bf16_t* __restrict__ z, const bf16_t* __restrict__ W, const float* __restrict__ bias,
                                                       bf16_t* __restrict__ P, float* __restrict__ ref, const float* __restrict__ lt,
                                                       bf16_t* __restrict__ zs, float* __restrict__ rowloss,
                                                       float* __restrict__ rowscale, int d, int ldzs, int V, float inv_rows) {
  __shared__ float red[8];
  if (status && *status != 0) return;      // the step is already void (an expired wait, a bad id): its sums mean nothing
  const int nbad = bad[0];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int i = blockIdx.x; i < nbad; i += gridDim.x) {
    const int n = bad[1 + i];
    const uint4* zr = reinterpret_cast<const uint4*>(z + (long long)n * d);
    auto logit = [&](int v) {
      const uint4* wr = reinterpret_cast<const uint4*>(W + (long long)v * d);
      float acc = 0.f;
      for (int k = lane; k < (d >> 3); k += 32) acc += dot8_bf16(__ldg(zr + k), __ldg(wr + k));
      return warp_sum(acc) + bias[v];
    };
    float mx = -INFINITY;
    for (int v = warp; v < V; v += 8) mx = fmaxf(mx, logit(v));
    __syncthreads();
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int w = 1; w < 8; w++) mx = fmaxf(mx, red[w]);
    float S = 0.f;
    for (int v = warp; v < V; v += 8) {
      const float e = expf(logit(v) - mx);
      S += e;
      if (lane == 0) P[(long long)n * V + v] = __float2bfloat16_rn(e);
    }
    __syncthreads();
    if (lane == 0) red[warp] = S;
    __syncthreads();
    S = red[0];
#pragma unroll
    for (int w = 1; w < 8; w++) S += red[w];
    const float r = inv_rows / S;
    if (threadIdx.x == 0) {      // (the barrier above ordered every warp's writes of P before this patch)
      ref[n] = mx;
      rowloss[n] = mx + logf(S) - lt[n];
      rowscale[n] = r;
      P[(long long)n * V + tgt[n]] = __float2bfloat16_rn(expf(lt[n] - mx) - S);
    }
    if (warp == 0) {
      scale_row_bf16(z + (long long)n * d, zs + (long long)n * ldzs, d, r, lane);
      scale_row_tail(zs + (long long)n * ldzs, d, ldzs, r, lane);
    }
    __syncthreads();
  }
}

// dz[n,c] = r_n * sum_s part[s][n,c]   (partials of P W_h in split order; rounded to bf16 once)
__global__ void __launch_bounds__(256) ce_dz_finish_kernel(const float4* __restrict__ part, int splits, long long mn4, int d4,
                                                           const float* __restrict__ rowscale, bf16_t* __restrict__ dz) {
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= mn4) return;
  const int n = (int)(i / d4);
  float4 a = part[i];
  for (int s = 1; s < splits; s++) {
    const float4 b = part[(long long)s * mn4 + i];
    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
  }
  const float r = rowscale[n];
  store4(dz + i * 4, make_float4(a.x * r, a.y * r, a.z * r, a.w * r));
}

cudaError_t ce_target_logit(const void* z, const void* W, const float* bias, const int32_t* ids, int T_, int rows, int d, int V,
                            int* tgt, float* ref, float* lt, int* bad, cudaStream_t s) {
  const int grid = (int)std::min<long long>(cdiv(rows, 8), 148 * 8);
  ce_target_logit_kernel<<<grid, 256, 0, s>>>((const bf16_t*)z, (const bf16_t*)W, bias, ids, T_, rows, d, V, tgt, ref, lt, bad);
  return cudaGetLastError();
}
cudaError_t ce_finalize(const float* psum, int groups, const float* ref, const float* lt, const int* tgt, void* P, int V, const void* z,
                        void* zs, int ldzs, float* rowloss, float* rowscale, int* bad, int rows, int d, float inv_rows, cudaStream_t s) {
  const int grid = (int)std::min<long long>(cdiv(rows, 8), 148 * 8);
  ce_finalize_kernel<<<grid, 256, 0, s>>>(psum, groups, ref, lt, tgt, (bf16_t*)P, V, (const bf16_t*)z, (bf16_t*)zs, rowloss, rowscale, bad,
                                          rows, d, ldzs, inv_rows);
  return cudaGetLastError();
}
cudaError_t ce_fixup(const int* bad, const int* status, const int* tgt, const void* z, const void* W, const float* bias, void* P, float* ref,
                     const float* lt, void* zs, int ldzs, float* rowloss, float* rowscale, int rows, int d, int V, float inv_rows, cudaStream_t s) {
  const int grid = rows < 32 ? rows : 32;
  ce_fixup_kernel<<<grid, 256, 0, s>>>(bad, status, tgt, (const bf16_t*)z, (const bf16_t*)W, bias, (bf16_t*)P, ref, lt, (bf16_t*)zs, rowloss,
                                       rowscale, d, ldzs, V, inv_rows);
  return cudaGetLastError();
}
cudaError_t ce_dz_finish(const float* part, int splits, int rows, int d, const float* rowscale, void* dz, cudaStream_t s) {
  const long long mn4 = (long long)rows * d / 4;
  ce_dz_finish_kernel<<<cdiv(mn4, 256), 256, 0, s>>>((const float4*)part, splits, mn4, d / 4, rowscale, (bf16_t*)dz);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(1024) reduce_sum_kernel(const float* __restrict__ v, int n, float scale,
                                                          float* __restrict__ out) {
  __shared__ float sm[1024];
  float a = 0.f;
  for (int i = threadIdx.x; i < n; i += 1024) a += v[i];
  sm[threadIdx.x] = a;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[0] = sm[0] * scale;
}

cudaError_t reduce_sum(const float* v, int n, float scale, float* out, cudaStream_t s) {
  reduce_sum_kernel<<<1, 1024, 0, s>>>(v, n, scale, out);
  return cudaGetLastError();
}

template <typename T>
__global__ void __launch_bounds__(256) bce_head_fwd_kernel(const T* __restrict__ z, long long ldz,
                                                           const float* __restrict__ w, const float* __restrict__ b,
                                                           const float* __restrict__ y, float* __restrict__ rowloss,
                                                           float* __restrict__ ds, int rows, int d, float inv_rows) {
  int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float s = 0.f;
  for (int c = lane; c < d; c += 32) s = fmaf(ldf(z + (long long)row * ldz + c), w[c], s);
  s = warp_sum(s) + b[0];
  if (lane == 0) {
    float yy = y[row];
    float e = expf(-fabsf(s));
    rowloss[row] = fmaxf(s, 0.f) - s * yy + log1pf(e);
    float sig = s >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
    ds[row] = (sig - yy) * inv_rows;
  }
}

cudaError_t bce_head_fwd(const void* z, long long ldz, const float* w, const float* b, const float* y,
                         float* rowloss, float* ds, int rows, int d, float inv_rows, bool bf16,
                         cudaStream_t s) {
  if (bf16) bce_head_fwd_kernel<bf16_t><<<cdiv(rows, 8), 256, 0, s>>>((const bf16_t*)z, ldz, w, b, y, rowloss, ds, rows, d, inv_rows);
  else bce_head_fwd_kernel<float><<<cdiv(rows, 8), 256, 0, s>>>((const float*)z, ldz, w, b, y, rowloss, ds, rows, d, inv_rows);
  return cudaGetLastError();
}

template <typename T>
__global__ void __launch_bounds__(256) bce_head_dz_kernel(const float* __restrict__ ds, const float* __restrict__ w,
                                                          T* __restrict__ dz, int dact, const T* __restrict__ src,
                                                          long long n, int d) {
  long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float v = ds[i / d] * w[i % d];
  if (dact != ACT_NONE) v *= act_deriv(dact, ldf(src + i));
  stf(dz + i, v);
}

// one 16-byte piece (8 bf16 / 4 floats of one row) per thread; d a multiple of the piece
template <typename T>
__global__ void __launch_bounds__(256) bce_head_dz_vec_kernel(const float* __restrict__ ds, const float* __restrict__ w,
                                                              T* __restrict__ dz, int dact, const T* __restrict__ src,
                                                              long long nvec, int dvec) {
  constexpr int VEC = VecOf<T>::N;
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= nvec) return;
  const long long row = i / dvec;
  const int c = (int)(i - row * dvec) * VEC;
  const float dsr = ds[row];
  float v[VEC], u[VEC];
  if (dact != ACT_NONE) ld_vec<T>(src + i * VEC, u);
#pragma unroll
  for (int j = 0; j < VEC; j++) {
    v[j] = dsr * w[c + j];
    if (dact != ACT_NONE) v[j] *= act_deriv(dact, u[j]);
  }
  if (VEC == 8) {
    uint4 q;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(v[0], v[1]); q.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[2], v[3]); q.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[4 % VEC], v[5 % VEC]); q.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(v[6 % VEC], v[7 % VEC]); q.w = *reinterpret_cast<uint32_t*>(&h);
    *reinterpret_cast<uint4*>(dz + i * VEC) = q;
  } else {
    *reinterpret_cast<float4*>(dz + i * VEC) = make_float4(v[0], v[1], v[2], v[3]);
  }
}

cudaError_t bce_head_dz(const float* ds, const float* w, void* dz, int dact, const void* src, int rows,
                        int d, bool bf16, cudaStream_t s) {
  long long n = (long long)rows * d;
  const int vec = bf16 ? 8 : 4;
  const bool al = ((reinterpret_cast<uintptr_t>(dz) | reinterpret_cast<uintptr_t>(src)) & 15) == 0;
  if (al && d % vec == 0) {
    const long long nvec = n / vec;
    if (bf16) bce_head_dz_vec_kernel<bf16_t><<<cdiv(nvec, 256), 256, 0, s>>>(ds, w, (bf16_t*)dz, dact, (const bf16_t*)src, nvec, d / vec);
    else bce_head_dz_vec_kernel<float><<<cdiv(nvec, 256), 256, 0, s>>>(ds, w, (float*)dz, dact, (const float*)src, nvec, d / vec);
    return cudaGetLastError();
  }
  if (bf16) bce_head_dz_kernel<bf16_t><<<cdiv(n, 256), 256, 0, s>>>(ds, w, (bf16_t*)dz, dact, (const bf16_t*)src, n, d);
  else bce_head_dz_kernel<float><<<cdiv(n, 256), 256, 0, s>>>(ds, w, (float*)dz, dact, (const float*)src, n, d);
  return cudaGetLastError();
}

// Goodness head (binary cross-entropy on G = sum_j z_j^2 with the logit G + b): one warp per row,
// the same outputs as the BCE head (row losses, ds = (sigmoid(s) - y)/rows).
template <typename T>
__global__ void __launch_bounds__(256) goodness_head_fwd_kernel(const T* __restrict__ z, long long ldz,
                                                                const float* __restrict__ b, const float* __restrict__ y,
                                                                float* __restrict__ rowloss, float* __restrict__ ds,
                                                                int rows, int d, float inv_rows) {
  int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float s = 0.f;
  for (int c = lane; c < d; c += 32) {
    const float v = ldf(z + (long long)row * ldz + c);
    s = fmaf(v, v, s);
  }
  s = warp_sum(s) + b[0];
  if (lane == 0) {
    float yy = y[row];
    float e = expf(-fabsf(s));
    rowloss[row] = fmaxf(s, 0.f) - s * yy + log1pf(e);
    float sig = s >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
    ds[row] = (sig - yy) * inv_rows;
  }
}
cudaError_t goodness_head_fwd(const void* z, long long ldz, const float* b, const float* y, float* rowloss, float* ds,
                              int rows, int d, float inv_rows, bool bf16, cudaStream_t s) {
  if (bf16) goodness_head_fwd_kernel<bf16_t><<<cdiv(rows, 8), 256, 0, s>>>((const bf16_t*)z, ldz, b, y, rowloss, ds, rows, d, inv_rows);
  else goodness_head_fwd_kernel<float><<<cdiv(rows, 8), 256, 0, s>>>((const float*)z, ldz, b, y, rowloss, ds, rows, d, inv_rows);
  return cudaGetLastError();
}

// dz = 2 ds z (times act'(src) when z = act(src) closes the block)
template <typename T>
__global__ void __launch_bounds__(256) goodness_head_dz_kernel(const float* __restrict__ ds, const T* __restrict__ z,
                                                               T* __restrict__ dz, int dact, const T* __restrict__ src,
                                                               long long n, int d) {
  long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float v = 2.f * ds[i / d] * ldf(z + i);
  if (dact != ACT_NONE) v *= act_deriv(dact, ldf(src + i));
  stf(dz + i, v);
}
cudaError_t goodness_head_dz(const float* ds, const void* z, void* dz, int dact, const void* src, int rows,
                             int d, bool bf16, cudaStream_t s) {
  long long n = (long long)rows * d;
  if (bf16) goodness_head_dz_kernel<bf16_t><<<cdiv(n, 256), 256, 0, s>>>(ds, (const bf16_t*)z, (bf16_t*)dz, dact, (const bf16_t*)src, n, d);
  else goodness_head_dz_kernel<float><<<cdiv(n, 256), 256, 0, s>>>(ds, (const float*)z, (float*)dz, dact, (const float*)src, n, d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// elementwise
// ------------------------------------------------------------------------------------------
// One 16-byte vector per thread and step (8 bf16 or 4 floats); the element tail is scalar.
// mode 0: out = a * b      mode 1: out = act(a)      mode 2: out = a * act'(b)
template <typename T>
__global__ void __launch_bounds__(256) ew_kernel(const T* a, const T* __restrict__ b, T* out,   // a may alias out
                                                 long long n, int mode, int act) {
  constexpr int VEC = VecOf<T>::N;
  const long long nvec = n / VEC;
  const long long stride = (long long)gridDim.x * 256;
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < nvec; i += stride) {
    float x[VEC], y[VEC];
    ld_vec<T>(a + i * VEC, x);
    if (mode != 1) ld_vec<T>(b + i * VEC, y);
    if (act == ACT_GELU && mode != 0) {     // the common case, with the cheaper normal CDF for bf16 data
#pragma unroll
      for (int j = 0; j < VEC; j++) x[j] = mode == 1 ? gelu_ew<T>(x[j]) : x[j] * dgelu_ew<T>(y[j]);
    } else {
#pragma unroll
      for (int j = 0; j < VEC; j++)
        x[j] = mode == 0 ? x[j] * y[j] : (mode == 1 ? act_apply(act, x[j]) : x[j] * act_deriv(act, y[j]));
    }
    if (VEC == 8) {
      uint4 q;
      __nv_bfloat162 h;
      h = __floats2bfloat162_rn(x[0], x[1]); q.x = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(x[2], x[3]); q.y = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(x[4 % VEC], x[5 % VEC]); q.z = *reinterpret_cast<uint32_t*>(&h);
      h = __floats2bfloat162_rn(x[6 % VEC], x[7 % VEC]); q.w = *reinterpret_cast<uint32_t*>(&h);
      *reinterpret_cast<uint4*>(out + i * VEC) = q;
    } else {
      *reinterpret_cast<float4*>(out + i * VEC) = make_float4(x[0], x[1], x[2], x[3]);
    }
  }
  if (blockIdx.x == 0)
    for (long long i = nvec * VEC + threadIdx.x; i < n; i += 256) {
      const float xa = ldf(a + i);
      stf(out + i, mode == 0 ? xa * ldf(b + i) : (mode == 1 ? act_apply(act, xa) : xa * act_deriv(act, ldf(b + i))));
    }
}

static cudaError_t ew_launch(const void* a, const void* b, void* out, long long n, int mode, int act, bool bf16, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  const bool aligned = ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(out)) & 15) == 0;
  if (!aligned) return cudaErrorMisalignedAddress;   // every buffer of the library is 256-byte aligned
  const long long nvec = n / (bf16 ? 8 : 4);
  long long blocks = (nvec + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  if (bf16) ew_kernel<bf16_t><<<(unsigned)blocks, 256, 0, s>>>((const bf16_t*)a, (const bf16_t*)b, (bf16_t*)out, n, mode, act);
  else ew_kernel<float><<<(unsigned)blocks, 256, 0, s>>>((const float*)a, (const float*)b, (float*)out, n, mode, act);
  return cudaGetLastError();
}
cudaError_t ew_mul(const void* a, const void* b, void* out, long long n, bool bf16, cudaStream_t s) {
  return ew_launch(a, b, out, n, 0, ACT_NONE, bf16, s);
}
cudaError_t ew_act(const void* u, void* out, int act, long long n, bool bf16, cudaStream_t s) {
  return ew_launch(u, nullptr, out, n, 1, act, bf16, s);
}
cudaError_t ew_dact(void* d, const void* src, int act, long long n, bool bf16, cudaStream_t s) {
  return ew_launch(d, src, d, n, 2, act, bf16, s);
}

// ------------------------------------------------------------------------------------------
// input staging (z_0)
// ------------------------------------------------------------------------------------------
// An id outside its table is never used as an index: the row is filled from row 0 instead and the
// model's status word is set to STATUS_BAD_ID, which the next synchronisation reports as an
// invalid argument (the step's results are void).
__device__ __forceinline__ int checked_id(int id, int rows, int* status) {
  if ((unsigned)id >= (unsigned)rows) {
    if (status) atomicExch(status, STATUS_BAD_ID);
    return 0;
  }
  return id;
}


// Token + position gather, one warp per output row: the id is read once per row, a lane moves four
// consecutive columns per step (two 16-byte loads, one 8- or 16-byte store), so a warp reads 512
// contiguous bytes of the embedding row at a time.  VEC = false is the scalar form for widths that
// are not multiples of four.
template <typename T, bool VEC>
__global__ void __launch_bounds__(256) gather_tokens_kernel(const float* __restrict__ tok, const float* __restrict__ pos,
                                                            const int32_t* __restrict__ ids, T* __restrict__ z0, int T_, int d,
                                                            int rows, int vocab, int* status) {
  const int lane = threadIdx.x & 31;
  for (int row = blockIdx.x * 8 + (threadIdx.x >> 5); row < rows; row += gridDim.x * 8) {
    const int t = row % T_, b = row / T_;
    const int id = checked_id(ids[(long long)b * (T_ + 1) + t], vocab, status);
    if (t == T_ - 1 && lane == 0) checked_id(ids[(long long)b * (T_ + 1) + T_], vocab, status);   // the last target is no input
    const float* te = tok + (long long)id * d;
    const float* pe = pos + (long long)t * d;
    T* out = z0 + (long long)row * d;
    if (VEC) {
      for (int c = lane * 4; c < d; c += 128) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(te + c));
        const float4 q = __ldg(reinterpret_cast<const float4*>(pe + c));
        store4(out + c, make_float4(a.x + q.x, a.y + q.y, a.z + q.z, a.w + q.w));
      }
    } else {
      for (int c = lane; c < d; c += 32) stf(out + c, te[c] + pe[c]);
    }
  }
}
cudaError_t gather_tokens(const float* tok, const float* pos, const int32_t* ids, void* z0, int batch,
                          int T_, int d, int vocab, int* status, bool bf16, cudaStream_t s) {
  const int rows = batch * T_;
  const bool vec = d % 4 == 0 && ((reinterpret_cast<uintptr_t>(tok) | reinterpret_cast<uintptr_t>(pos) | reinterpret_cast<uintptr_t>(z0)) & 15) == 0;
  const int grid = (int)std::min<long long>(cdiv(rows, 8), 148 * 8);
  if (bf16) {
    if (vec) gather_tokens_kernel<bf16_t, true><<<grid, 256, 0, s>>>(tok, pos, ids, (bf16_t*)z0, T_, d, rows, vocab, status);
    else gather_tokens_kernel<bf16_t, false><<<grid, 256, 0, s>>>(tok, pos, ids, (bf16_t*)z0, T_, d, rows, vocab, status);
  } else {
    if (vec) gather_tokens_kernel<float, true><<<grid, 256, 0, s>>>(tok, pos, ids, (float*)z0, T_, d, rows, vocab, status);
    else gather_tokens_kernel<float, false><<<grid, 256, 0, s>>>(tok, pos, ids, (float*)z0, T_, d, rows, vocab, status);
  }
  return cudaGetLastError();
}

// CTR gather and pack, one warp per sample: x0[n] = [table_t[ids[n,t]] for t | dense | zero pad].
// The lanes run over (table, four columns) pairs, so a table row leaves as 16-byte loads and lands
// as 8-byte (bf16) or 16-byte stores; the dense columns and the padding follow in a scalar tail.
template <typename T, bool VEC>
__global__ void __launch_bounds__(256) gather_ctr_kernel(const float* __restrict__ tables, long long table_stride,
                                                         const int32_t* __restrict__ ids, const float* __restrict__ dense,
                                                         T* __restrict__ x0, int batch, int ns, int e, int nd, int width,
                                                         int table_rows, int* status) {
  const int lane = threadIdx.x & 31;
  for (int n = blockIdx.x * 8 + (threadIdx.x >> 5); n < batch; n += gridDim.x * 8) {
    T* out = x0 + (long long)n * width;
    const int32_t* idn = ids + (long long)n * ns;
    if (VEC) {
      const int vpr = e >> 2;                                  // 16-byte vectors per table row
      for (int i = lane; i < ns * vpr; i += 32) {
        const int t = i / vpr, c = (i - t * vpr) * 4;
        const int id = checked_id(idn[t], table_rows, status);
        const float4 v = __ldg(reinterpret_cast<const float4*>(tables + (long long)t * table_stride + (long long)id * e + c));
        store4(out + t * e + c, v);
      }
    } else {
      for (int i = lane; i < ns * e; i += 32) {
        const int t = i / e, c = i - t * e;
        const int id = checked_id(idn[t], table_rows, status);
        stf(out + i, tables[(long long)t * table_stride + (long long)id * e + c]);
      }
    }
    for (int c = ns * e + lane; c < width; c += 32) stf(out + c, c < ns * e + nd ? dense[(long long)n * nd + (c - ns * e)] : 0.f);
  }
}
cudaError_t gather_ctr(const float* tables, long long table_stride, const int32_t* ids, const float* dense,
                       void* x0, int batch, int ns, int e, int nd, int width, int table_rows, int* status, bool bf16,
                       cudaStream_t s) {
  const bool vec = e % 4 == 0 && width % 4 == 0 && table_stride % 4 == 0 &&
                   ((reinterpret_cast<uintptr_t>(tables) | reinterpret_cast<uintptr_t>(x0)) & 15) == 0;
  const int grid = (int)std::min<long long>(cdiv(batch, 8), 148 * 8);
  if (bf16) {
    if (vec) gather_ctr_kernel<bf16_t, true><<<grid, 256, 0, s>>>(tables, table_stride, ids, dense, (bf16_t*)x0, batch, ns, e, nd, width, table_rows, status);
    else gather_ctr_kernel<bf16_t, false><<<grid, 256, 0, s>>>(tables, table_stride, ids, dense, (bf16_t*)x0, batch, ns, e, nd, width, table_rows, status);
  } else {
    if (vec) gather_ctr_kernel<float, true><<<grid, 256, 0, s>>>(tables, table_stride, ids, dense, (float*)x0, batch, ns, e, nd, width, table_rows, status);
    else gather_ctr_kernel<float, false><<<grid, 256, 0, s>>>(tables, table_stride, ids, dense, (float*)x0, batch, ns, e, nd, width, table_rows, status);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// dot interaction: one CTA of 128 threads per sample
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) dot_fwd_kernel(const T* __restrict__ proj, const T* __restrict__ x0,
                                                      long long ldx0, T* __restrict__ feats, int ns, int e, int fw) {
  extern __shared__ float sm[];  // [(ns+1)][e+1]
  const int n = blockIdx.x, nv = ns + 1, lde = e + 1;
  for (int i = threadIdx.x; i < nv * e; i += 128) {
    int j = i / e, c = i - j * e;
    sm[j * lde + c] = j == 0 ? ldf(proj + (long long)n * e + c) : ldf(x0 + (long long)n * ldx0 + (j - 1) * e + c);
  }
  __syncthreads();
  const int npair = nv * (nv - 1) / 2;
  T* f = feats + (long long)n * fw;
  for (int p = threadIdx.x; p < fw; p += 128) {
    float v = 0.f;
    if (p < npair) {
      // invert p = i(i-1)/2 + j, 0 <= j < i
      int i = (int)((1.f + sqrtf(1.f + 8.f * p)) * 0.5f);
      while (i * (i - 1) / 2 > p) i--;
      while ((i + 1) * i / 2 <= p) i++;
      int j = p - i * (i - 1) / 2;
      for (int c = 0; c < e; c++) v = fmaf(sm[i * lde + c], sm[j * lde + c], v);
    } else if (p < npair + e) {
      v = sm[p - npair];
    }
    stf(f + p, v);
  }
}
cudaError_t dot_fwd(const void* proj, const void* x0, long long ldx0, void* feats, int batch, int ns, int e,
                    int fw, bool bf16, cudaStream_t s) {
  size_t smem = (size_t)(ns + 1) * (e + 1) * sizeof(float);
  if (bf16) dot_fwd_kernel<bf16_t><<<batch, 128, smem, s>>>((const bf16_t*)proj, (const bf16_t*)x0, ldx0, (bf16_t*)feats, ns, e, fw);
  else dot_fwd_kernel<float><<<batch, 128, smem, s>>>((const float*)proj, (const float*)x0, ldx0, (float*)feats, ns, e, fw);
  return cudaGetLastError();
}

template <typename T>
__global__ void __launch_bounds__(128) dot_bwd_kernel(const T* __restrict__ dfeat, const T* __restrict__ x0,
                                                      long long ldx0, T* __restrict__ dproj, int ns, int e, int fw) {
  const int n = blockIdx.x, nv = ns + 1;
  const int npair = nv * (nv - 1) / 2;
  const T* df = dfeat + (long long)n * fw;
  for (int c = threadIdx.x; c < e; c += 128) {
    float v = ldf(df + npair + c);
    for (int j = 1; j < nv; j++)
      v = fmaf(ldf(df + j * (j - 1) / 2), ldf(x0 + (long long)n * ldx0 + (j - 1) * e + c), v);
    stf(dproj + (long long)n * e + c, v);
  }
}
cudaError_t dot_bwd(const void* dfeat, const void* x0, long long ldx0, void* dproj, int batch, int ns, int e,
                    int fw, bool bf16, cudaStream_t s) {
  if (bf16) dot_bwd_kernel<bf16_t><<<batch, 128, 0, s>>>((const bf16_t*)dfeat, (const bf16_t*)x0, ldx0, (bf16_t*)dproj, ns, e, fw);
  else dot_bwd_kernel<float><<<batch, 128, 0, s>>>((const float*)dfeat, (const float*)x0, ldx0, (float*)dproj, ns, e, fw);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// optimizer
// ------------------------------------------------------------------------------------------
__global__ void opt_tick_kernel(double* tick, double b1, double b2) {
  double t = tick[0] + 1.0;
  tick[0] = t;
  tick[1] = 1.0 - pow(b1, t);
  tick[2] = 1.0 - pow(b2, t);
}
cudaError_t opt_tick(double* tick, float beta1, float beta2, cudaStream_t s) {
  opt_tick_kernel<<<1, 1, 0, s>>>(tick, (double)beta1, (double)beta2);
  return cudaGetLastError();
}

// One element of SGD / Adam / AdamW; every path below applies exactly this arithmetic.
__device__ __forceinline__ void opt_element(float& th, float g, float& mm, float& vv, int kind, float lr, float b1, float b2,
                                            float eps, float wd, float bc1, float bc2) {
  if (kind == 0) {
    th -= lr * g;
  } else {
    if (kind == 2) th *= (1.f - lr * wd);
    mm = b1 * mm + (1.f - b1) * g;
    vv = b2 * vv + (1.f - b2) * g * g;
    th -= lr * (mm / bc1) / (sqrtf(vv / bc2) + eps);
  }
}

// Four consecutive parameters per thread (16-byte accesses; the arenas are 256-byte aligned and a
// block's slice starts on a multiple of 64 elements); the last, partial quad is done element-wise.
__global__ void __launch_bounds__(256) opt_update_kernel(float* __restrict__ theta, const float* __restrict__ grad,
                                                         float* __restrict__ m, float* __restrict__ v,
                                                         bf16_t* __restrict__ shadow, long long n, int kind, float lr,
                                                         float b1, float b2, float eps, float wd,
                                                         const double* __restrict__ tick, int vec) {
  const long long q = (long long)blockIdx.x * 256 + threadIdx.x;
  const long long i = q * 4;
  if (i >= n) return;
  float bc1 = 1.f, bc2 = 1.f;
  if (kind != 0) { bc1 = (float)tick[1]; bc2 = (float)tick[2]; }
  if (vec && i + 4 <= n) {
    float4 th = reinterpret_cast<float4*>(theta)[q];
    const float4 g = reinterpret_cast<const float4*>(grad)[q];
    float4 mm = make_float4(0.f, 0.f, 0.f, 0.f), vv = mm;
    if (kind != 0) { mm = reinterpret_cast<float4*>(m)[q]; vv = reinterpret_cast<float4*>(v)[q]; }
    opt_element(th.x, g.x, mm.x, vv.x, kind, lr, b1, b2, eps, wd, bc1, bc2);
    opt_element(th.y, g.y, mm.y, vv.y, kind, lr, b1, b2, eps, wd, bc1, bc2);
    opt_element(th.z, g.z, mm.z, vv.z, kind, lr, b1, b2, eps, wd, bc1, bc2);
    opt_element(th.w, g.w, mm.w, vv.w, kind, lr, b1, b2, eps, wd, bc1, bc2);
    if (kind != 0) { reinterpret_cast<float4*>(m)[q] = mm; reinterpret_cast<float4*>(v)[q] = vv; }
    reinterpret_cast<float4*>(theta)[q] = th;
    if (shadow) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
      uint2 w;
      w.x = *reinterpret_cast<uint32_t*>(&lo);
      w.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(shadow)[q] = w;
    }
    return;
  }
  for (long long k = i; k < n && k < i + 4; k++) {
    float th = theta[k], mm = 0.f, vv = 0.f;
    if (kind != 0) { mm = m[k]; vv = v[k]; }
    opt_element(th, grad[k], mm, vv, kind, lr, b1, b2, eps, wd, bc1, bc2);
    if (kind != 0) { m[k] = mm; v[k] = vv; }
    theta[k] = th;
    if (shadow) shadow[k] = __float2bfloat16_rn(th);
  }
}
cudaError_t opt_update(float* theta, const float* grad, float* m, float* v, void* shadow, long long n, int kind,
                       float lr, float beta1, float beta2, float eps, float wd, const double* tick,
                       cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  auto al = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
  const int vec = al(theta, 16) && al(grad, 16) && (!m || al(m, 16)) && (!v || al(v, 16)) && (!shadow || al(shadow, 8));
  opt_update_kernel<<<cdiv((n + 3) / 4, 256), 256, 0, s>>>(theta, grad, m, v, (bf16_t*)shadow, n, kind, lr, beta1, beta2, eps, wd, tick, vec);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// The undetached remainder (Section 2.2, Eq. 2): input of the main network and the embedding backward
// ------------------------------------------------------------------------------------------
// u[n, off_s .. off_s + w_s) = src_s[n, 0 .. w_s) for up to CONCAT_MAX sources: u = [z_0 | z_1 | ... | z_B]
template <typename T>
__global__ void __launch_bounds__(256) concat_kernel(ConcatArgs a, T* __restrict__ u, int rows) {
  const int src = blockIdx.y;
  const T* p = (const T*)a.src[src];
  const int w = a.width[src], off = a.offset[src];
  const long long n = (long long)rows * w;
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
    const long long r = i / w;
    const int c = (int)(i - r * w);
    u[r * a.total + off + c] = p[r * a.ld[src] + c];
  }
}
cudaError_t concat_cols(const ConcatArgs& a, void* u, int rows, bool bf16, cudaStream_t s) {
  int wmax = 1;
  for (int i = 0; i < a.n; i++) wmax = std::max(wmax, a.width[i]);
  dim3 grid((unsigned)std::min<long long>(cdiv((long long)rows * wmax, 256), 148 * 4), a.n);
  if (bf16) concat_kernel<bf16_t><<<grid, 256, 0, s>>>(a, (bf16_t*)u, rows);
  else concat_kernel<float><<<grid, 256, 0, s>>>(a, (float*)u, rows);
  return cudaGetLastError();
}

// Embedding backward, step 1: one CTA per table sorts (id, sample) pairs (bitonic, in shared memory),
// so that the samples that read one table row are contiguous and in sample order, and numbers the
// distinct rows: sorted_n[t][pos] = sample at sorted position pos, seg_start[t][s] = first position of
// the s-th distinct row (seg_start[t][n_uniq] = batch), uniq_id[t][s] = that row, n_uniq[t].
__global__ void __launch_bounds__(1024) embed_sort_kernel(const int32_t* __restrict__ ids, int batch, int ns, int table_rows, int npow2,
                                                          int* __restrict__ sorted_n, int* __restrict__ seg_start,
                                                          int* __restrict__ uniq_id, int* __restrict__ n_uniq) {
  extern __shared__ unsigned long long keys[];
  __shared__ int scan[1024];
  const int t = blockIdx.x;
  for (int i = threadIdx.x; i < npow2; i += 1024) {
    unsigned long long k = ~0ull;                            // padding sorts to the end
    if (i < batch) {
      int id = ids[(long long)i * ns + t];
      id = min(max(id, 0), table_rows - 1);                  // a bad id was reported by the input staging
      k = ((unsigned long long)(unsigned)id << 32) | (unsigned)i;
    }
    keys[i] = k;
  }
  __syncthreads();
  for (int size = 2; size <= npow2; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = threadIdx.x; i < npow2 / 2; i += 1024) {
        const int lo = (i / stride) * stride * 2 + (i % stride), hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long a = keys[lo], b = keys[hi];
        if ((a > b) == up) { keys[lo] = b; keys[hi] = a; }
      }
      __syncthreads();
    }
  // segment starts and their numbering: every thread owns a contiguous run of positions
  const int per = (batch + 1023) / 1024, lo = threadIdx.x * per, hi = min(batch, lo + per);
  int cnt = 0;
  for (int i = lo; i < hi; i++) cnt += (i == 0 || (keys[i] >> 32) != (keys[i - 1] >> 32));
  scan[threadIdx.x] = cnt;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {                       // inclusive scan over the 1024 counts
    const int v = threadIdx.x >= o ? scan[threadIdx.x - o] : 0;
    __syncthreads();
    scan[threadIdx.x] += v;
    __syncthreads();
  }
  int seg = scan[threadIdx.x] - cnt;
  int* sn = sorted_n + (long long)t * batch;
  int* ss = seg_start + (long long)t * (batch + 1);
  int* ui = uniq_id + (long long)t * batch;
  for (int i = lo; i < hi; i++) {
    sn[i] = (int)(keys[i] & 0xffffffffu);
    if (i == 0 || (keys[i] >> 32) != (keys[i - 1] >> 32)) {
      ss[seg] = i;
      ui[seg] = (int)(keys[i] >> 32);
      seg++;
    }
  }
  if (threadIdx.x == 1023) {
    n_uniq[t] = scan[1023];
    ss[scan[1023]] = batch;
  }
}

// Step 2: one warp per distinct row: grow[t][s][:] = sum over the samples of segment s, in sample order,
// of dz0[n, t*e : (t+1)*e] -- the scatter-add without atomics (one writer, fixed order).
template <typename T>
__global__ void __launch_bounds__(256) embed_rows_kernel(const T* __restrict__ dz0, long long ld, int batch, int e,
                                                         const int* __restrict__ sorted_n, const int* __restrict__ seg_start,
                                                         const int* __restrict__ n_uniq, float* __restrict__ grow) {
  const int t = blockIdx.y, seg = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (seg >= n_uniq[t]) return;
  const int* sn = sorted_n + (long long)t * batch;
  const int* ss = seg_start + (long long)t * (batch + 1);
  const int beg = ss[seg], end = ss[seg + 1];
  for (int c = lane; c < e; c += 32) {
    float acc = 0.f;
    for (int pos = beg; pos < end; pos++) acc += ldf(dz0 + (long long)sn[pos] * ld + t * e + c);
    grow[((long long)t * batch + seg) * e + c] = acc;
  }
}

// Step 3: the optimizer on the touched rows only (untouched rows keep values and moments; the bias
// correction is the global one in tick[]); the same element update as the dense optimizer.
__global__ void __launch_bounds__(256) embed_update_kernel(float* __restrict__ tables, long long table_stride, float* __restrict__ m,
                                                           float* __restrict__ v, int batch, int e, const int* __restrict__ uniq_id,
                                                           const int* __restrict__ n_uniq, const float* __restrict__ grow, int kind,
                                                           float lr, float b1, float b2, float eps, float wd,
                                                           const double* __restrict__ tick) {
  const int t = blockIdx.y, seg = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (seg >= n_uniq[t]) return;
  float bc1 = 1.f, bc2 = 1.f;
  if (kind != 0) { bc1 = (float)tick[1]; bc2 = (float)tick[2]; }
  const long long base = (long long)t * table_stride + (long long)uniq_id[(long long)t * batch + seg] * e;
  for (int c = lane; c < e; c += 32) {
    float th = tables[base + c], mm = 0.f, vv = 0.f;
    if (kind != 0) { mm = m[base + c]; vv = v[base + c]; }
    opt_element(th, grow[((long long)t * batch + seg) * e + c], mm, vv, kind, lr, b1, b2, eps, wd, bc1, bc2);
    if (kind != 0) { m[base + c] = mm; v[base + c] = vv; }
    tables[base + c] = th;
  }
}

int embed_max_batch() { return 16384; }

cudaError_t embed_backward(const void* dz0, long long ld, const int32_t* ids, int batch, int ns, int e, int table_rows, int* sorted_n,
                           int* seg_start, int* uniq_id, int* n_uniq, float* grow, bool bf16, cudaStream_t s) {
  int npow2 = 1;
  while (npow2 < batch) npow2 <<= 1;
  const size_t smem = (size_t)npow2 * sizeof(unsigned long long);
  static std::atomic<size_t> attr[64];
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) dev = 0;
  if (smem > 48 * 1024 && smem > attr[dev].load()) {
    cudaError_t e2 = cudaFuncSetAttribute(embed_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e2 != cudaSuccess) return e2;
    attr[dev].store(smem);
  }
  embed_sort_kernel<<<ns, 1024, smem, s>>>(ids, batch, ns, table_rows, npow2, sorted_n, seg_start, uniq_id, n_uniq);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  dim3 grid(cdiv(batch, 8), ns);
  if (bf16) embed_rows_kernel<bf16_t><<<grid, 256, 0, s>>>((const bf16_t*)dz0, ld, batch, e, sorted_n, seg_start, n_uniq, grow);
  else embed_rows_kernel<float><<<grid, 256, 0, s>>>((const float*)dz0, ld, batch, e, sorted_n, seg_start, n_uniq, grow);
  return cudaGetLastError();
}

cudaError_t embed_update(float* tables, long long table_stride, float* m, float* v, int batch, int ns, int e, const int* uniq_id,
                         const int* n_uniq, const float* grow, int kind, float lr, float beta1, float beta2, float eps, float wd,
                         const double* tick, cudaStream_t s) {
  dim3 grid(cdiv(batch, 8), ns);
  embed_update_kernel<<<grid, 256, 0, s>>>(tables, table_stride, m, v, batch, e, uniq_id, n_uniq, grow, kind, lr, beta1, beta2, eps, wd, tick);
  return cudaGetLastError();
}

__global__ void to_bf16_kernel(const float* __restrict__ src, bf16_t* __restrict__ dst, long long n) {
  long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i < n) dst[i] = __float2bfloat16_rn(src[i]);
}
cudaError_t to_bf16(const float* src, void* dst, long long n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  to_bf16_kernel<<<cdiv(n, 256), 256, 0, s>>>(src, (bf16_t*)dst, n);
  return cudaGetLastError();
}

}  // namespace erase
