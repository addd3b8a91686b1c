// Causal flash attention on the tensor cores for bf16 models with 64-wide heads: forward,
// dK/dV and dQ kernels built from mma.sync m16n8k16 (bf16 x bf16 -> fp32) and ldmatrix.
// No T x T matrix is ever written to memory; the backward recomputes the probabilities from
// the saved log-sum-exp.  dK/dV and dQ are separate kernels (one loops over query tiles, the
// other over key tiles), so every output element has exactly one writer and a fixed summation
// order: no atomics, bit-reproducible.
//
// Tile = 64 queries x 64 keys, CTA = 4 warps, a warp owns 16 rows of the tile.
#include <cuda_bf16.h>
#include <stdint.h>

#include "kernels.cuh"

namespace erase {

namespace {

typedef __nv_bfloat16 bf16_t;
constexpr int TS = 64;      // tile size (queries and keys)
constexpr int DH = 64;      // head width
constexpr int LDS = 72;     // shared-memory row stride in elements (144 B: conflict-free ldmatrix)

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// 64 x 64 bf16 tile from global (row stride ld elements) into shared [64][LDS]; rows >= rows_valid are zero.
__device__ __forceinline__ void load_tile(bf16_t* dst, const bf16_t* src, long long ld, int rows_valid) {
  for (int i = threadIdx.x; i < TS * (DH / 8); i += 128) {
    int r = i >> 3, c = (i & 7) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < rows_valid) v = *reinterpret_cast<const uint4*>(src + (long long)r * ld + c);
    *reinterpret_cast<uint4*>(dst + r * LDS + c) = v;
  }
}

// The same tile, fetched with cp.async (16 bytes per request, zero-filled past rows_valid) so that
// the next tile streams in while the current one is being multiplied.  rows_valid >= 1.
__device__ __forceinline__ void load_tile_async(bf16_t* dst, const bf16_t* src, long long ld, int rows_valid) {
  for (int i = threadIdx.x; i < TS * (DH / 8); i += 128) {
    const int r = i >> 3, c = (i & 7) * 8;
    const int rs = r < rows_valid ? r : rows_valid - 1;
    const uint32_t bytes = r < rows_valid ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s_u32(dst + r * LDS + c)),
                 "l"(src + (long long)rs * ld + c), "r"(bytes) : "memory");
  }
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// A fragments (16 rows x 64 k) of a row-major tile, rows row0..row0+15: a[kk][0..3]
__device__ __forceinline__ void load_a_frags(const bf16_t* tile, int row0, uint32_t a[4][4]) {
  const int lane = threadIdx.x & 31;
  const int r = row0 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
  for (int kk = 0; kk < 4; kk++) {
    const int c = kk * 16 + (lane >> 4) * 8;
    ldsm_x4(s_u32(tile + r * LDS + c), a[kk][0], a[kk][1], a[kk][2], a[kk][3]);
  }
}

// acc[nt] (16 x 8 each, nt = 0..7) += A(16 x 64) * X^T where X is a row-major [64 n][64 k] tile
__device__ __forceinline__ void mma_a_xt(float acc[8][4], const uint32_t a[4][4], const bf16_t* x) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int kk = 0; kk < 4; kk++) {
#pragma unroll
    for (int np = 0; np < 4; np++) {
      const int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
      const int c = kk * 16 + ((lane >> 3) & 1) * 8;
      uint32_t b0, b1, b2, b3;
      ldsm_x4(s_u32(x + r * LDS + c), b0, b1, b2, b3);
      mma16816(acc[2 * np], a[kk], b0, b1);
      mma16816(acc[2 * np + 1], a[kk], b2, b3);
    }
  }
}

// out[nt] (16 x 64) += P(16 x 64, from accumulators p) * X where X is a row-major [64 k][64 n] tile
__device__ __forceinline__ void mma_p_x(float out[8][4], const float p[8][4], const bf16_t* x) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int kk = 0; kk < 4; kk++) {
    uint32_t a[4];
    a[0] = pack_bf16(p[2 * kk][0], p[2 * kk][1]);
    a[1] = pack_bf16(p[2 * kk][2], p[2 * kk][3]);
    a[2] = pack_bf16(p[2 * kk + 1][0], p[2 * kk + 1][1]);
    a[3] = pack_bf16(p[2 * kk + 1][2], p[2 * kk + 1][3]);
#pragma unroll
    for (int np = 0; np < 4; np++) {
      const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      const int c = np * 16 + (lane >> 4) * 8;
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(s_u32(x + r * LDS + c), b0, b1, b2, b3);
      mma16816(out[2 * np], a, b0, b1);
      mma16816(out[2 * np + 1], a, b2, b3);
    }
  }
}

// Half-tile versions for the dK/dV kernel, which works on 32 of the 64 query columns at a time so
// that its score and dP accumulators take 32 registers instead of 64 (three CTAs per SM, not two).
// acc[nt] (nt = 0..3: columns 32*half + 8*nt ..) += A(16 x 64) * X^T, X rows 32*half .. 32*half+31
__device__ __forceinline__ void mma_a_xt_half(float acc[4][4], const uint32_t a[4][4], const bf16_t* x, int half) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int kk = 0; kk < 4; kk++) {
#pragma unroll
    for (int np = 0; np < 2; np++) {
      const int r = (2 * half + np) * 16 + (lane & 7) + (lane >> 4) * 8;
      const int c = kk * 16 + ((lane >> 3) & 1) * 8;
      uint32_t b0, b1, b2, b3;
      ldsm_x4(s_u32(x + r * LDS + c), b0, b1, b2, b3);
      mma16816(acc[2 * np], a[kk], b0, b1);
      mma16816(acc[2 * np + 1], a[kk], b2, b3);
    }
  }
}
// out (16 x 64) += P(16 x 32: contraction rows 32*half .. 32*half+31 of X, from accumulators p) * X
__device__ __forceinline__ void mma_p_x_half(float out[8][4], const float p[4][4], const bf16_t* x, int half) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int kk = 0; kk < 2; kk++) {
    uint32_t a[4];
    a[0] = pack_bf16(p[2 * kk][0], p[2 * kk][1]);
    a[1] = pack_bf16(p[2 * kk][2], p[2 * kk][3]);
    a[2] = pack_bf16(p[2 * kk + 1][0], p[2 * kk + 1][1]);
    a[3] = pack_bf16(p[2 * kk + 1][2], p[2 * kk + 1][3]);
#pragma unroll
    for (int np = 0; np < 4; np++) {
      const int r = (2 * half + kk) * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
      const int c = np * 16 + (lane >> 4) * 8;
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(s_u32(x + r * LDS + c), b0, b1, b2, b3);
      mma16816(out[2 * np], a, b0, b1);
      mma16816(out[2 * np + 1], a, b2, b3);
    }
  }
}

__device__ __forceinline__ void zero_acc(float a[8][4]) {
#pragma unroll
  for (int i = 0; i < 8; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) a[i][j] = 0.f;
}

// ---------------------------------------------------------------------------------------------
// forward: grid (q tiles, heads, batch)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) attn_fwd_mma(const bf16_t* __restrict__ qkv, bf16_t* __restrict__ o,
                                                    float* __restrict__ lse, int T, int H, float scale) {
  __shared__ __align__(16) bf16_t Qs[TS * LDS];
  __shared__ __align__(16) bf16_t KVs[2][2][TS * LDS];   // [buffer][K|V]: the next key tile loads while this one is used
  const int qt = gridDim.x - 1 - blockIdx.x;             // heaviest (longest key loop) query tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int d = H * DH;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  const int q0 = qt * TS;
  const bf16_t* base = qkv + (long long)b * T * ld + h * DH;
  load_tile_async(Qs, base + (long long)q0 * ld, ld, T - q0);
  load_tile_async(KVs[0][0], base + d, ld, T);
  load_tile_async(KVs[0][1], base + 2 * d, ld, T);
  async_commit();
  uint32_t qa[4][4];
  float oacc[8][4];
  zero_acc(oacc);
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const float sc2 = scale * 1.4426950408889634f;  // scores are kept in log2 units
  const int row_a = q0 + warp * 16 + g, row_b = row_a + 8;
  for (int jt = 0; jt <= qt; jt++) {
    const int j0 = jt * TS;
    if (jt < qt) {
      load_tile_async(KVs[(jt + 1) & 1][0], base + d + (long long)(j0 + TS) * ld, ld, T - j0 - TS);
      load_tile_async(KVs[(jt + 1) & 1][1], base + 2 * d + (long long)(j0 + TS) * ld, ld, T - j0 - TS);
      async_commit();
      async_wait<1>();
    } else {
      async_wait<0>();
    }
    __syncthreads();
    if (jt == 0) load_a_frags(Qs, warp * 16, qa);
    const bf16_t* Ks = KVs[jt & 1][0];
    const bf16_t* Vs = KVs[jt & 1][1];
    float s[8][4];
    zero_acc(s);
    mma_a_xt(s, qa, Ks);
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 8; nt++) {
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const int col = j0 + nt * 8 + t4 * 2 + (e & 1);
        const int row = (e < 2) ? row_a : row_b;
        float v = s[nt][e] * sc2;
        if (jt == qt && col > row) v = -INFINITY;
        s[nt][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float corr[2];
#pragma unroll
    for (int r = 0; r < 2; r++) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mnew = fmaxf(mrow[r], mx[r]);   // finite: key j0 <= row is always unmasked
      corr[r] = exp2f(mrow[r] - mnew);
      mrow[r] = mnew;
      lrow[r] *= corr[r];
    }
#pragma unroll
    for (int nt = 0; nt < 8; nt++) {
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const float p = exp2f(s[nt][e] - mrow[e >> 1]);
        s[nt][e] = p;
        lrow[e >> 1] += p;
        oacc[nt][e] *= corr[e >> 1];
      }
    }
    mma_p_x(oacc, s, Vs);
    __syncthreads();   // every warp is done with this buffer before the load two tiles ahead reuses it
  }
#pragma unroll
  for (int r = 0; r < 2; r++) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  const float inv[2] = {1.f / lrow[0], 1.f / lrow[1]};
#pragma unroll
  for (int r = 0; r < 2; r++) {
    const int row = r == 0 ? row_a : row_b;
    if (row >= T) continue;
    bf16_t* orow = o + ((long long)b * T + row) * d + h * DH;
#pragma unroll
    for (int nt = 0; nt < 8; nt++)
      *reinterpret_cast<uint32_t*>(orow + nt * 8 + t4 * 2) = pack_bf16(oacc[nt][2 * r] * inv[r], oacc[nt][2 * r + 1] * inv[r]);
    if (t4 == 0) lse[((long long)b * H + h) * T + row] = (mrow[r] + log2f(lrow[r])) * 0.6931471805599453f;
  }
}

// ---------------------------------------------------------------------------------------------
// backward, dK and dV: grid (key tiles, heads, batch); loops over the query tiles at or after it.
// Works on the transposed tile: rows = keys (a warp owns 16), columns = queries.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) attn_bwd_kv_mma(const bf16_t* __restrict__ qkv, const bf16_t* __restrict__ dout,
                                                       const float* __restrict__ lse, const float* __restrict__ delta,
                                                       bf16_t* __restrict__ dqkv, int T, int H, float scale) {
  __shared__ __align__(16) bf16_t Xs[TS * LDS];   // K then V of this key tile (to build fragments), later unused
  __shared__ __align__(16) bf16_t QDs[2][2][TS * LDS];   // [buffer][Q|dO]: the next query tile loads while this one is used
  __shared__ float LEs[2][2][TS];                        // [buffer][lse*log2e | delta]
  const int kt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int d = H * DH;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  const int k0 = kt * TS;
  const bf16_t* base = qkv + (long long)b * T * ld + h * DH;
  const bf16_t* dob = dout + (long long)b * T * d + h * DH;
  uint32_t ka[4][4], va[4][4];
  float dk[8][4], dv[8][4];
  zero_acc(dk);
  zero_acc(dv);
  const float sc2 = scale * 1.4426950408889634f;
  const int key_a = k0 + warp * 16 + g, key_b = key_a + 8;
  const int n_qt = (T + TS - 1) / TS;
  auto fetch = [&](int it, int buf) {   // query tile `it` -> buffer `buf` (asynchronous)
    const int i0 = it * TS;
    load_tile_async(QDs[buf][0], base + (long long)i0 * ld, ld, T - i0);
    load_tile_async(QDs[buf][1], dob + (long long)i0 * d, d, T - i0);
    async_commit();
    if (threadIdx.x < TS) {
      const int i = i0 + threadIdx.x;
      LEs[buf][0][threadIdx.x] = i < T ? lse[((long long)b * H + h) * T + i] * 1.4426950408889634f : 0.f;
      LEs[buf][1][threadIdx.x] = i < T ? delta[((long long)b * H + h) * T + i] : 0.f;
    }
  };
  // One memory round trip for the whole prologue: this key tile's K and V (K into Xs, V into the
  // second query buffer, which the loop only refills after the fragments have been read) and the
  // first query tile are all requested before anything is waited for.
  load_tile_async(Xs, base + d + (long long)k0 * ld, ld, T - k0);
  load_tile_async(QDs[1][0], base + 2 * d + (long long)k0 * ld, ld, T - k0);
  fetch(kt, 0);
  async_wait<0>();
  __syncthreads();
  load_a_frags(Xs, warp * 16, ka);
  load_a_frags(QDs[1][0], warp * 16, va);
  __syncthreads();
  for (int it = kt; it < n_qt; it++) {
    const int i0 = it * TS;
    const int buf = (it - kt) & 1;
    if (it + 1 < n_qt) {
      fetch(it + 1, buf ^ 1);
      async_wait<1>();
    } else {
      async_wait<0>();
    }
    __syncthreads();
    const bf16_t* Qs = QDs[buf][0];
    const bf16_t* Ds = QDs[buf][1];
    const float* Ls = LEs[buf][0];
    const float* Es = LEs[buf][1];
#pragma unroll 1
    for (int half = 0; half < 2; half++) {   // 32 query columns at a time
      float st[4][4], dp[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; nt++)
#pragma unroll
        for (int e = 0; e < 4; e++) st[nt][e] = dp[nt][e] = 0.f;
      mma_a_xt_half(st, ka, Qs, half);   // S^T = K Q^T
      mma_a_xt_half(dp, va, Ds, half);   // dP^T = V dO^T
#pragma unroll
      for (int nt = 0; nt < 4; nt++) {
#pragma unroll
        for (int e = 0; e < 4; e++) {
          const int cl = half * 32 + nt * 8 + t4 * 2 + (e & 1);
          const int qi = i0 + cl;
          const int key = (e < 2) ? key_a : key_b;
          const bool valid = qi < T && key <= qi;
          const float p = valid ? exp2f(st[nt][e] * sc2 - Ls[cl]) : 0.f;
          st[nt][e] = p;
          dp[nt][e] = p * (dp[nt][e] - Es[cl]);
        }
      }
      mma_p_x_half(dv, st, Ds, half);    // dV += P^T dO
      mma_p_x_half(dk, dp, Qs, half);    // dK += dS^T Q
    }
    __syncthreads();        // this buffer is refilled two tiles ahead
  }
#pragma unroll
  for (int r = 0; r < 2; r++) {
    const int key = r == 0 ? key_a : key_b;
    if (key >= T) continue;
    bf16_t* row = dqkv + ((long long)b * T + key) * ld + h * DH;
#pragma unroll
    for (int nt = 0; nt < 8; nt++) {
      *reinterpret_cast<uint32_t*>(row + d + nt * 8 + t4 * 2) = pack_bf16(dk[nt][2 * r] * scale, dk[nt][2 * r + 1] * scale);
      *reinterpret_cast<uint32_t*>(row + 2 * d + nt * 8 + t4 * 2) = pack_bf16(dv[nt][2 * r], dv[nt][2 * r + 1]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// backward, dQ: grid (query tiles, heads, batch); loops over the key tiles at or before it.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) attn_bwd_q_mma(const bf16_t* __restrict__ qkv, const bf16_t* __restrict__ dout,
                                                      const float* __restrict__ lse, const float* __restrict__ delta,
                                                      bf16_t* __restrict__ dqkv, int T, int H, float scale) {
  __shared__ __align__(16) bf16_t Xs[TS * LDS];   // Q then dO of this query tile (fragments only)
  __shared__ __align__(16) bf16_t KVs[2][2][TS * LDS];   // [buffer][K|V]
  const int qt = gridDim.x - 1 - blockIdx.x;             // heaviest query tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int d = H * DH;
  const long long ld = 3LL * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  const int q0 = qt * TS;
  const bf16_t* base = qkv + (long long)b * T * ld + h * DH;
  const bf16_t* dob = dout + (long long)b * T * d + h * DH;
  uint32_t qa[4][4], da[4][4];
  // One memory round trip for the prologue: Q into Xs, dO into the second key buffer (refilled by
  // the loop only after the fragments have been read), the first key tile into the first buffer.
  load_tile_async(Xs, base + (long long)q0 * ld, ld, T - q0);
  load_tile_async(KVs[1][0], dob + (long long)q0 * d, d, T - q0);
  load_tile_async(KVs[0][0], base + d, ld, T);
  load_tile_async(KVs[0][1], base + 2 * d, ld, T);
  async_commit();
  async_wait<0>();
  __syncthreads();
  load_a_frags(Xs, warp * 16, qa);
  load_a_frags(KVs[1][0], warp * 16, da);
  __syncthreads();
  const int row_a = q0 + warp * 16 + g, row_b = row_a + 8;
  float lrow[2], erow[2];
#pragma unroll
  for (int r = 0; r < 2; r++) {
    const int row = r == 0 ? row_a : row_b;
    lrow[r] = row < T ? lse[((long long)b * H + h) * T + row] * 1.4426950408889634f : 0.f;
    erow[r] = row < T ? delta[((long long)b * H + h) * T + row] : 0.f;
  }
  float dq[8][4];
  zero_acc(dq);
  const float sc2 = scale * 1.4426950408889634f;
  for (int jt = 0; jt <= qt; jt++) {
    const int j0 = jt * TS;
    if (jt < qt) {
      load_tile_async(KVs[(jt + 1) & 1][0], base + d + (long long)(j0 + TS) * ld, ld, T - j0 - TS);
      load_tile_async(KVs[(jt + 1) & 1][1], base + 2 * d + (long long)(j0 + TS) * ld, ld, T - j0 - TS);
      async_commit();
      async_wait<1>();
    } else {
      async_wait<0>();
    }
    __syncthreads();
    const bf16_t* Ks = KVs[jt & 1][0];
    const bf16_t* Vs = KVs[jt & 1][1];
#pragma unroll 1
    for (int half = 0; half < 2; half++) {   // 32 key columns at a time: half the score / dP registers
      float s[4][4], dp[4][4];
#pragma unroll
      for (int nt = 0; nt < 4; nt++)
#pragma unroll
        for (int e = 0; e < 4; e++) s[nt][e] = dp[nt][e] = 0.f;
      mma_a_xt_half(s, qa, Ks, half);    // S = Q K^T
      mma_a_xt_half(dp, da, Vs, half);   // dP = dO V^T
#pragma unroll
      for (int nt = 0; nt < 4; nt++) {
#pragma unroll
        for (int e = 0; e < 4; e++) {
          const int col = j0 + half * 32 + nt * 8 + t4 * 2 + (e & 1);
          const int row = (e < 2) ? row_a : row_b;
          const float p = col <= row ? exp2f(s[nt][e] * sc2 - lrow[e >> 1]) : 0.f;
          dp[nt][e] = p * (dp[nt][e] - erow[e >> 1]);
        }
      }
      mma_p_x_half(dq, dp, Ks, half);    // dQ += dS K
    }
    __syncthreads();        // this buffer is refilled two tiles ahead
  }
#pragma unroll
  for (int r = 0; r < 2; r++) {
    const int row = r == 0 ? row_a : row_b;
    if (row >= T) continue;
    bf16_t* out = dqkv + ((long long)b * T + row) * ld + h * DH;
#pragma unroll
    for (int nt = 0; nt < 8; nt++)
      *reinterpret_cast<uint32_t*>(out + nt * 8 + t4 * 2) = pack_bf16(dq[nt][2 * r] * scale, dq[nt][2 * r + 1] * scale);
  }
}

// delta[b,h,t] = sum_c dO[row, h*64+c] * O[row, h*64+c]; one warp per (row, head)
__global__ void __launch_bounds__(256) attn_delta_mma(const bf16_t* __restrict__ o, const bf16_t* __restrict__ dout,
                                                      float* __restrict__ delta, long long rows, int T, int H) {
  const long long w = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= rows * H) return;
  const long long n = w / H;
  const int h = (int)(w % H);
  const long long off = n * H * DH + h * DH + lane * 2;
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(o + off);
  const __nv_bfloat162 c = *reinterpret_cast<const __nv_bfloat162*>(dout + off);
  float s = __bfloat162float(a.x) * __bfloat162float(c.x) + __bfloat162float(a.y) * __bfloat162float(c.y);
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) s += __shfl_xor_sync(0xffffffffu, s, k);
  if (lane == 0) delta[((n / T) * H + h) * T + (n % T)] = s;
}

}  // namespace

bool attention_mma_supported(int dh, int d) { return dh == DH && d % 8 == 0; }

cudaError_t attention_delta_bf16(const void* o, const void* dout, float* delta, int batch, int T, int heads, cudaStream_t s) {
  const long long rows = (long long)batch * T;
  attn_delta_mma<<<(unsigned)((rows * heads + 7) / 8), 256, 0, s>>>((const bf16_t*)o, (const bf16_t*)dout, delta, rows, T, heads);
  return cudaGetLastError();
}

cudaError_t attention_fwd_mma(const void* qkv, void* o, float* lse, int batch, int T, int heads, cudaStream_t s) {
  dim3 grid((T + TS - 1) / TS, heads, batch);
  attn_fwd_mma<<<grid, 128, 0, s>>>((const bf16_t*)qkv, (bf16_t*)o, lse, T, heads, 0.125f);
  return cudaGetLastError();
}

cudaError_t attention_bwd_mma(const void* qkv, const void* o, const void* dout, const float* lse, float* delta,
                              void* dqkv, int batch, int T, int heads, cudaStream_t s) {
  const long long rows = (long long)batch * T;
  attn_delta_mma<<<(unsigned)((rows * heads + 7) / 8), 256, 0, s>>>((const bf16_t*)o, (const bf16_t*)dout, delta, rows, T, heads);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 grid((T + TS - 1) / TS, heads, batch);
  attn_bwd_kv_mma<<<grid, 128, 0, s>>>((const bf16_t*)qkv, (const bf16_t*)dout, lse, delta, (bf16_t*)dqkv, T, heads, 0.125f);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  attn_bwd_q_mma<<<grid, 128, 0, s>>>((const bf16_t*)qkv, (const bf16_t*)dout, lse, delta, (bf16_t*)dqkv, T, heads, 0.125f);
  return cudaGetLastError();
}

}  // namespace erase
