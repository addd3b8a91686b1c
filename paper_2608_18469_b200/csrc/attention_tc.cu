// Causal flash attention on the 5th-generation tensor cores (tcgen05 / TMEM / TMA) for bf16 models
// with 64-wide heads: forward, dK/dV and dQ kernels.  No T x T matrix is ever written to memory;
// the backward recomputes the probabilities from the saved log-sum-exp.  dK/dV and dQ are separate
// kernels (one walks over query tiles, the other over key tiles), so every output element has one
// writer and a fixed summation order: no atomics, bit-reproducible.
//
// Tiles are 128 x 128 (queries x keys).  Q, K, V (and dO) tiles are fetched by TMA straight out of
// the [rows, 3 d] qkv matrix (128-byte swizzle: a head's 64 columns are one swizzle row).  Every
// product is one tcgen05.mma chain issued by a single thread with its accumulator in tensor memory:
//     S = Q K^T        A = Q  [q, dh]   K-major      B = K [key, dh]  K-major     (M 128, N 128, K 64)
//     O = P V          A = P  [q, key]  K-major      B = V [key, dh]  MN-major    (M 128, N  64, K 128)
// and in the backward the same tiles read through the other descriptor kind (a [row, dh] tile is a
// K-major operand when the contraction runs over dh and an MN-major one when it runs over rows), so
// nothing is ever transposed in memory.  Four softmax warps own one accumulator row (TMEM lane) per
// thread: they read S with tcgen05.ld, exponentiate, and write P (bf16) into shared memory in the
// swizzled K-major layout the next MMA reads.  All waits are clock-bounded; on expiry the model's
// status word is set, the kernel still frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <atomic>

#include "gemm_tc.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace erase {

namespace {

typedef __nv_bfloat16 bf16_t;
constexpr int TQ = 128;              // queries per tile
constexpr int TK = 128;              // keys per tile
constexpr int DH = 64;               // head width
constexpr uint32_t TILE_BYTES = 128 * DH * 2;     // a [128, 64] bf16 tile: 128 swizzle rows of 128 bytes
constexpr uint32_t P_BYTES = 2 * TILE_BYTES;      // a [128, 128] bf16 tile: two 64-column halves
constexpr int AT_THREADS = 160;      // warps 0..3 softmax (TMEM lane quarters 0..3), warp 4 issues TMA and MMA
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void set_status(int* st, int code) { if (st) atomicExch(st, code); }
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// instruction descriptor: bf16 x bf16 -> fp32, M = 128, given N and operand majors
__device__ __forceinline__ uint32_t idesc_of(int n, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// K-major [128 rows, 64 k] tile: k step of 16 elements = 32 bytes inside the swizzled row
__device__ __forceinline__ uint64_t desc_k(uint32_t tile, int k16) { return smem_desc(tile + k16 * 32, 16, 1024); }
// MN-major [64 k rows][64 m/n] block (128-byte runs along M/N, one per k): k step of 16 = 16 rows = 2048 bytes;
// the next 64 M/N elements, if any, sit `lbo` bytes further
__device__ __forceinline__ uint64_t desc_mn(uint32_t block, int k16, uint32_t lbo) { return smem_desc(block + k16 * 2048, lbo, 1024); }

// Writes 32 consecutive values of this thread's row (bf16) into a K-major [128, 128] operand tile:
// column c lives in half c / 64; inside a half a row is 128 bytes whose 16-byte pieces are XOR-ed
// with the row (the 128-byte swizzle the descriptors and TMA assume).
__device__ __forceinline__ void store_p32(uint32_t tile, int row, int col0, const float* v) {
  const uint32_t base = tile + (uint32_t)(col0 >> 6) * TILE_BYTES + (uint32_t)row * 128u;
  const int piece0 = (col0 & 63) >> 3;
#pragma unroll
  for (int g = 0; g < 4; g++)
    sts_v4(base + (uint32_t)(((piece0 + g) ^ (row & 7)) << 4), pack_bf(v[8 * g], v[8 * g + 1]), pack_bf(v[8 * g + 2], v[8 * g + 3]),
           pack_bf(v[8 * g + 4], v[8 * g + 5]), pack_bf(v[8 * g + 6], v[8 * g + 7]));
}

struct AttnArgs {
  int T, H, batch;
  float scale;           // 1 / sqrt(dh)
  float scale_log2;      // scale * log2(e)
  bf16_t* o;             // forward output [rows, d]
  float* lse;            // [batch, H, T], natural log (written by the forward, read by the backward)
  float* delta;          // backward: [batch, H, T], sum_c dO * O (written by the dQ kernel, read by the dK/dV kernel)
  bf16_t* dqkv;          // backward output [rows, 3 d]
  int* status;
};

// ------------------------------------------------------------------------------------------------
// forward: one CTA per (query tile, head, sequence); key tiles 0 .. query tile
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(AT_THREADS, 2)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ AttnArgs p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);       // the swizzled tiles need 1024-byte alignment: checked below
  const uint32_t q_s = base, k_s = base + TILE_BYTES, v_s = k_s + 2 * TILE_BYTES, p_s = v_s + 2 * TILE_BYTES;
  const uint32_t bar = p_s + P_BYTES;
  const uint32_t q_full = bar, kv_full0 = bar + 8, kv_empty0 = bar + 24, s_full = bar + 40, p_full = bar + 48, o_full = bar + 56,
                 o_free = bar + 64, tmem_slot = bar + 72;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;        // heaviest (longest key range) tiles first
  const int h = blockIdx.y, b = blockIdx.z;
  const int d = p.H * DH;
  const int q0 = qt * TQ;
  const int nt = qt + 1;                                       // key tiles 0..qt (TQ == TK)
  int st0 = status_peek(p.status);
  if (threadIdx.x == 0 && (base & 1023u)) { set_status(p.status, 10); st0 = 10; }   // never expected: do nothing rather than misread tiles

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; s++) { mbar_init(kv_full0 + 8 * s, 1); mbar_init(kv_empty0 + 8 * s, 1); }
    mbar_init(s_full, 1);
    mbar_init(p_full, 4);
    mbar_init(o_full, 1);
    mbar_init(o_free, 4);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 4) {
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_qkv) : "memory");
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t tm_s = tmem, tm_o = tmem + 128;

  if (dead) {
    // the step is already void
  } else if (warp == 4) {
    if (lane == 0) {
      const int row0 = b * p.T;
      auto load_kv = [&](int j) {
        const int s = j & 1;
        mbar_expect_tx(kv_full0 + 8 * s, 2 * TILE_BYTES);
        tma_load_2d(k_s + s * TILE_BYTES, &map_qkv, d + h * DH, row0 + j * TK, kv_full0 + 8 * s);
        tma_load_2d(v_s + s * TILE_BYTES, &map_qkv, 2 * d + h * DH, row0 + j * TK, kv_full0 + 8 * s);
      };
      mbar_expect_tx(q_full, TILE_BYTES);
      tma_load_2d(q_s, &map_qkv, h * DH, row0 + q0, q_full);
      load_kv(0);
      if (nt > 1) load_kv(1);
      const uint32_t id_s = idesc_of(TK, false, false), id_o = idesc_of(DH, false, true);
      bool ok = mbar_wait(q_full, 0);
      if (!ok) set_status(p.status, 11);
      auto issue_pv = [&](int j) {          // O_j = P_j V_j (fresh accumulator), then release the K/V stage
        const int s = j & 1;
#pragma unroll
        for (int kk = 0; kk < TK / 16; kk++)
          tc_mma(tm_o, desc_k(p_s + (kk >> 2) * TILE_BYTES, kk & 3), desc_mn(v_s + s * TILE_BYTES + (kk >> 2) * (TILE_BYTES / 2), kk & 3, TILE_BYTES / 2),
                 id_o, kk > 0 ? 1u : 0u);
        tc_commit(o_full);
        tc_commit(kv_empty0 + 8 * s);
      };
      for (int j = 0; j < nt && ok; j++) {
        const int s = j & 1;
        if (!mbar_wait(kv_full0 + 8 * s, (j >> 1) & 1)) { set_status(p.status, 12); ok = false; break; }
        if (j > 0 && !mbar_wait(p_full, (j - 1) & 1)) { set_status(p.status, 13); ok = false; break; }   // S read, P_{j-1} written
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < DH / 16; kk++) tc_mma(tm_s, desc_k(q_s, kk), desc_k(k_s + s * TILE_BYTES, kk), id_s, kk > 0 ? 1u : 0u);
        tc_commit(s_full);
        if (j > 0) {
          if (j > 1 && !mbar_wait(o_free, (j - 2) & 1)) { set_status(p.status, 14); ok = false; break; }  // O_{j-2} read
          tc_fence_after();
          issue_pv(j - 1);
          if (j + 1 < nt) {                   // tile j+1 goes where tile j-1 was, once its MMAs have read it
            if (!mbar_wait(kv_empty0 + 8 * ((j - 1) & 1), ((j - 1) >> 1) & 1)) { set_status(p.status, 15); ok = false; break; }
            load_kv(j + 1);
          }
        }
      }
      if (ok) {
        if (!mbar_wait(p_full, (nt - 1) & 1)) { set_status(p.status, 13); ok = false; }
        if (ok && nt > 1 && !mbar_wait(o_free, (nt - 2) & 1)) { set_status(p.status, 14); ok = false; }
        if (ok) {
          tc_fence_after();
          issue_pv(nt - 1);
        }
      }
      if (!ok) {   // give copies in flight time to land before shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else {
    // ------------------------------ softmax warps: one accumulator row per thread ------------------------------
    const int row = warp * 32 + lane;                 // row of the tile = TMEM lane
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    float acc[DH];
#pragma unroll
    for (int c = 0; c < DH; c++) acc[c] = 0.f;
    float m = -INFINITY, l = 0.f, alpha_prev = 1.f;
    bool ok = true;
    auto take_o = [&](int j) -> bool {                // acc <- acc * alpha + O_j
      bool w = mbar_wait(o_full, j & 1);
      if (!w) set_status(p.status, 16);
      w = __all_sync(0xffffffffu, w);
      if (!w) return false;
      tc_fence_after();
      uint32_t r[32];
#pragma unroll
      for (int c = 0; c < 2; c++) {
        tc_ld32(tm_o + lane_off + c * 32, r);
#pragma unroll
        for (int e = 0; e < 32; e++) acc[c * 32 + e] = fmaf(acc[c * 32 + e], alpha_prev, __uint_as_float(r[e]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(o_free);
      return true;
    };
    for (int j = 0; j < nt; j++) {
      bool w = mbar_wait(s_full, j & 1);
      if (!w) set_status(p.status, 17);
      w = __all_sync(0xffffffffu, w);
      if (!w) { ok = false; break; }
      tc_fence_after();
      const bool diag = j == nt - 1;                  // the only tile with keys beyond some of its queries
      uint32_t r[32];
      // pass 1: row maximum (four independent chains; only the diagonal tile masks keys beyond the query)
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < TK / 32; c++) {
        tc_ld32(tm_s + lane_off + c * 32, r);
        if (diag) {
#pragma unroll
          for (int e = 0; e < 32; e++)
            if (c * 32 + e > row) r[e] = 0xff800000u;      // -inf
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          mx0 = fmaxf(mx0, __uint_as_float(r[e]));
          mx1 = fmaxf(mx1, __uint_as_float(r[e + 1]));
          mx2 = fmaxf(mx2, __uint_as_float(r[e + 2]));
          mx3 = fmaxf(mx3, __uint_as_float(r[e + 3]));
        }
      }
      const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      const float m_new = fmaxf(m, mx * p.scale_log2);
      const float alpha = ex2f(m - m_new);            // 0 for the first tile (m = -inf)
      if (j > 0 && !take_o(j - 1)) { ok = false; break; }
      // pass 2: exponentials, row sum (four chains), P to shared memory
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 1
      for (int c = 0; c < TK / 32; c++) {
        tc_ld32(tm_s + lane_off + c * 32, r);
        float pv[32];
#pragma unroll
        for (int e = 0; e < 32; e++) pv[e] = ex2f(fmaf(__uint_as_float(r[e]), p.scale_log2, -m_new));
        if (diag) {
#pragma unroll
          for (int e = 0; e < 32; e++)
            if (c * 32 + e > row) pv[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < 32; e += 4) { s0 += pv[e]; s1 += pv[e + 1]; s2 += pv[e + 2]; s3 += pv[e + 3]; }
        store_p32(p_s, row, c * 32, pv);
      }
      const float rowsum = (s0 + s1) + (s2 + s3);
      l = fmaf(l, alpha, rowsum);
      m = m_new;
      alpha_prev = alpha;
      tc_fence_before();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full);
    }
    if (ok && take_o(nt - 1)) {
      const int t = q0 + row;
      if (t < p.T) {
        const float inv = 1.f / l;
        bf16_t* out = p.o + ((long long)b * p.T + t) * d + h * DH;
#pragma unroll
        for (int g = 0; g < DH / 8; g++) {
          uint4 q;
          q.x = pack_bf(acc[8 * g] * inv, acc[8 * g + 1] * inv);
          q.y = pack_bf(acc[8 * g + 2] * inv, acc[8 * g + 3] * inv);
          q.z = pack_bf(acc[8 * g + 4] * inv, acc[8 * g + 5] * inv);
          q.w = pack_bf(acc[8 * g + 6] * inv, acc[8 * g + 7] * inv);
          *reinterpret_cast<uint4*>(out + 8 * g) = q;
        }
        p.lse[((long long)b * p.H + h) * p.T + t] = (m + log2f(l)) * 0.6931471805599453f;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}


// ------------------------------------------------------------------------------------------------
// backward.  Both kernels: 8 softmax warps (two per TMEM lane quarter, each takes 32 of the 64
// columns of a sub-tile) and one warp that issues TMA and MMA.  The walk goes over sub-tiles of 64
// keys (dQ kernel) or 64 queries (dK/dV kernel), so that the score, dP and gradient accumulators
// take 256 TMEM columns and two CTAs share an SM: one CTA's softmax work hides the other's MMA and
// barrier latencies.  The gradient accumulators stay in tensor memory over the whole walk (no
// rescaling is needed: the probabilities are recomputed from the final log-sum-exp).
// ------------------------------------------------------------------------------------------------
constexpr int BW_THREADS = 288;
constexpr int TW = 64;                                   // sub-tile width
constexpr uint32_t SUB_BYTES = TW * DH * 2;              // a [64, 64] bf16 sub-tile: 8 KB
constexpr int NST_Q = 3;                                 // K/V sub-tile stages of the dQ kernel
constexpr int NST_KV = 2;                                // Q/dO sub-tile stages of the dK/dV kernel

__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// dot product of one swizzled 128-byte row (64 bf16) of two K-major tiles
__device__ __forceinline__ float row_dot64(const uint8_t* ta, const uint8_t* tb, int row) {
  float d0 = 0.f, d1 = 0.f;
#pragma unroll
  for (int c = 0; c < 8; c++) {
    const int off = row * 128 + ((c ^ (row & 7)) << 4);
    const uint4 qa = *reinterpret_cast<const uint4*>(ta + off), qb = *reinterpret_cast<const uint4*>(tb + off);
    const uint32_t x[4] = {qa.x, qa.y, qa.z, qa.w}, y[4] = {qb.x, qb.y, qb.z, qb.w};
#pragma unroll
    for (int j = 0; j < 4; j++) {
      d0 = fmaf(__uint_as_float(x[j] << 16), __uint_as_float(y[j] << 16), d0);
      d1 = fmaf(__uint_as_float(x[j] & 0xffff0000u), __uint_as_float(y[j] & 0xffff0000u), d1);
    }
  }
  return d0 + d1;
}

// dQ (and delta): one CTA per (query tile of 128, head, sequence), key sub-tiles of 64 from 0 up to the tile's last query.
//   delta[q] = sum_c dO[q,c] O[q,c]  (from the dO and O tiles in shared memory; also written out for the dK/dV kernel)
//   S = Q K^T, dP = dO V^T (both operands K-major);  dS = P (.) (dP - delta), P = exp(S scale - lse)
//   dQ += dS K   (A = dS [q, key] K-major from shared memory, B = K [key, dh] MN-major), times scale at the end
__global__ void __launch_bounds__(BW_THREADS, 2)
attn_bwd_q_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                     const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_o,
                     const __grid_constant__ AttnArgs p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t q_s = base, do_s = q_s + TILE_BYTES, kv_s = do_s + TILE_BYTES, ds_s = kv_s + NST_Q * 2 * SUB_BYTES;
  const uint32_t bar = ds_s + TILE_BYTES;
  const uint32_t q_full = bar, kv_full0 = bar + 8, kv_empty0 = kv_full0 + 8 * NST_Q, sdp_full = kv_empty0 + 8 * NST_Q, ds_full = sdp_full + 8,
                 ds_free = ds_full + 8, acc_full = ds_free + 8, tmem_slot = acc_full + 8;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;
  const int h = blockIdx.y, b = blockIdx.z;
  const int d = p.H * DH;
  const int q0 = qt * TQ;
  const int nsub = min(2 * (qt + 1), (p.T + TW - 1) / TW);    // key sub-tiles that hold a key <= the tile's last query
  int st0 = status_peek(p.status);
  if (threadIdx.x == 0 && (base & 1023u)) { set_status(p.status, 10); st0 = 10; }

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < NST_Q; s++) { mbar_init(kv_full0 + 8 * s, 1); mbar_init(kv_empty0 + 8 * s, 1); }
    mbar_init(sdp_full, 1);
    mbar_init(ds_full, 8);
    mbar_init(ds_free, 1);
    mbar_init(acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_kv) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_do) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_o) : "memory");
    }
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t tm_s = tmem, tm_dp = tmem + 64, tm_dq = tmem + 128;

  if (dead) {
  } else if (warp == 8) {
    if (lane == 0) {
      const int row0 = b * p.T;
      auto load_kv = [&](int j) {
        const int s = j % NST_Q;
        const uint32_t full = kv_full0 + 8 * s, dst = kv_s + s * 2 * SUB_BYTES;
        mbar_expect_tx(full, 2 * SUB_BYTES);
        tma_load_2d(dst, &map_kv, d + h * DH, row0 + j * TW, full);
        tma_load_2d(dst + SUB_BYTES, &map_kv, 2 * d + h * DH, row0 + j * TW, full);
      };
      mbar_expect_tx(q_full, 3 * TILE_BYTES);
      tma_load_2d(q_s, &map_q, h * DH, row0 + q0, q_full);
      tma_load_2d(do_s, &map_do, h * DH, row0 + q0, q_full);
      tma_load_2d(ds_s, &map_o, h * DH, row0 + q0, q_full);      // the O tile: read once for delta, then this buffer holds dS
      for (int j = 0; j < NST_Q && j < nsub; j++) load_kv(j);
      const uint32_t id_s = idesc_of(TW, false, false), id_q = idesc_of(DH, false, true);
      bool ok = mbar_wait(q_full, 0);
      if (!ok) set_status(p.status, 21);
      auto issue_dq = [&](int j) {      // dQ += dS_j K_j
        const uint32_t kj = kv_s + (j % NST_Q) * 2 * SUB_BYTES;
#pragma unroll
        for (int kk = 0; kk < TW / 16; kk++) tc_mma(tm_dq, desc_k(ds_s, kk), desc_mn(kj, kk, SUB_BYTES), id_q, (j > 0 || kk > 0) ? 1u : 0u);
      };
      for (int j = 0; j < nsub && ok; j++) {
        const int s = j % NST_Q;
        const uint32_t kj = kv_s + s * 2 * SUB_BYTES, vj = kj + SUB_BYTES;
        if (!mbar_wait(kv_full0 + 8 * s, (j / NST_Q) & 1)) { set_status(p.status, 22); ok = false; break; }
        if (j > 0 && !mbar_wait(ds_full, (j - 1) & 1)) { set_status(p.status, 23); ok = false; break; }   // S, dP read; dS_{j-1} written
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < DH / 16; kk++) tc_mma(tm_s, desc_k(q_s, kk), desc_k(kj, kk), id_s, kk > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < DH / 16; kk++) tc_mma(tm_dp, desc_k(do_s, kk), desc_k(vj, kk), id_s, kk > 0 ? 1u : 0u);
        tc_commit(sdp_full);
        if (j > 0) {
          issue_dq(j - 1);
          tc_commit(ds_free);
          tc_commit(kv_empty0 + 8 * ((j - 1) % NST_Q));
          if (j - 1 + NST_Q < nsub) {     // the freed stage takes the sub-tile NST_Q further on
            if (!mbar_wait(kv_empty0 + 8 * ((j - 1) % NST_Q), ((j - 1) / NST_Q) & 1)) { set_status(p.status, 24); ok = false; break; }
            load_kv(j - 1 + NST_Q);
          }
        }
      }
      if (ok) {
        if (!mbar_wait(ds_full, (nsub - 1) & 1)) { set_status(p.status, 23); ok = false; }
        if (ok) {
          tc_fence_after();
          issue_dq(nsub - 1);
        }
      }
      tc_commit(acc_full);        // fires in any case, so that the softmax warps do not wait for their limit
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const int t = q0 + row;
    const bool row_ok = t < p.T;
    const long long stat = ((long long)b * p.H + h) * p.T + t;
    const float lse2 = row_ok ? p.lse[stat] * LOG2E : 0.f;
    bool ok = true;
    float dl = 0.f;
    {   // delta of this thread's row from the dO and O tiles
      bool w = mbar_wait(q_full, 0);
      if (!w) set_status(p.status, 28);
      w = __all_sync(0xffffffffu, w);
      if (w) {
        dl = row_dot64(smem_raw + (do_s - base), smem_raw + (ds_s - base), row);
        if (half == 0 && row_ok) p.delta[stat] = dl;
      } else {
        ok = false;
      }
      softmax_bar();              // every row of the O tile has been read: the buffer may now take dS
    }
    for (int j = 0; j < nsub && ok; j++) {
      bool w = mbar_wait(sdp_full, j & 1);
      if (!w) set_status(p.status, 25);
      w = __all_sync(0xffffffffu, w);
      if (!w) { ok = false; break; }
      tc_fence_after();
      const int col0 = half * 32;
      const int kcol = j * TW + col0 - q0;                      // key index minus query index = kcol + e - row
      const bool maskable = j * TW + TW - 1 > q0;              // some key of the sub-tile lies beyond some query
      uint32_t rs[32], rp[32];
      tc_ld32_nowait(tm_s + lane_off + col0, rs);
      tc_ld32_nowait(tm_dp + lane_off + col0, rp);
      tc_ld_wait();
      float ds[32];
      if (maskable) {
#pragma unroll
        for (int e = 0; e < 32; e++) {
          const float pe = kcol + e > row ? 0.f : ex2f(fmaf(__uint_as_float(rs[e]), p.scale_log2, -lse2));
          ds[e] = pe * (__uint_as_float(rp[e]) - dl);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 32; e++) ds[e] = ex2f(fmaf(__uint_as_float(rs[e]), p.scale_log2, -lse2)) * (__uint_as_float(rp[e]) - dl);
      }
      if (j > 0) {                  // the previous sub-tile's dQ MMAs must have read dS before it is overwritten
        bool f = mbar_wait(ds_free, (j - 1) & 1);
        if (!f) set_status(p.status, 26);
        f = __all_sync(0xffffffffu, f);
        if (!f) { ok = false; break; }
      }
      store_p32(ds_s, row, col0, ds);
      tc_fence_before();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(ds_full);
    }
    if (ok) {
      bool w = mbar_wait(acc_full, 0);
      if (!w) set_status(p.status, 27);
      w = __all_sync(0xffffffffu, w);
      if (w) {
        tc_fence_after();
        uint32_t r[32];
        tc_ld32(tm_dq + lane_off + half * 32, r);
        if (row_ok) {
          bf16_t* out = p.dqkv + ((long long)b * p.T + t) * (3 * d) + h * DH + half * 32;
#pragma unroll
          for (int g = 0; g < 4; g++) {
            uint4 q;
            q.x = pack_bf(__uint_as_float(r[8 * g]) * p.scale, __uint_as_float(r[8 * g + 1]) * p.scale);
            q.y = pack_bf(__uint_as_float(r[8 * g + 2]) * p.scale, __uint_as_float(r[8 * g + 3]) * p.scale);
            q.z = pack_bf(__uint_as_float(r[8 * g + 4]) * p.scale, __uint_as_float(r[8 * g + 5]) * p.scale);
            q.w = pack_bf(__uint_as_float(r[8 * g + 6]) * p.scale, __uint_as_float(r[8 * g + 7]) * p.scale);
            *reinterpret_cast<uint4*>(out + 8 * g) = q;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

// dK, dV: one CTA per (key tile of 128, head, sequence), query sub-tiles of 64 from the tile's first key to the end of
// the sequence.  Everything is computed transposed, so that a softmax thread owns a KEY row:
//   S^T = K Q^T, dP^T = V dO^T (both operands K-major);  P^T = exp(S^T scale - lse[q]),  dS^T = P^T (.) (dP^T - delta[q])
//   dV += P^T dO   (A = P^T [key, q] K-major from shared memory, B = dO [q, dh] MN-major)
//   dK += dS^T Q   (A = dS^T,                                   B = Q  [q, dh] MN-major), times scale at the end
__global__ void __launch_bounds__(BW_THREADS, 2)
attn_bwd_kv_tc_kernel(const __grid_constant__ CUtensorMap map_kv, const __grid_constant__ CUtensorMap map_q,
                      const __grid_constant__ CUtensorMap map_do, const __grid_constant__ AttnArgs p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = smem_u32(smem_raw);
  const uint32_t k_s = base, v_s = k_s + TILE_BYTES, qdo_s = v_s + TILE_BYTES, pt_s = qdo_s + NST_KV * 2 * SUB_BYTES, dst_s = pt_s + TILE_BYTES;
  const uint32_t vec_s = dst_s + TILE_BYTES;              // lse (log2 units) and delta of the query sub-tile: 2 buffers x 2 x 64 floats
  const uint32_t bar = vec_s + 1024;
  const uint32_t kv_full = bar, qdo_full0 = bar + 8, qdo_empty0 = qdo_full0 + 8 * NST_KV, sdp_full = qdo_empty0 + 8 * NST_KV,
                 pds_full = sdp_full + 8, pds_free = pds_full + 8, acc_full = pds_free + 8, tmem_slot = acc_full + 8;
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - base));
  float* vec = reinterpret_cast<float*>(smem_raw + (vec_s - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kt = blockIdx.x;                               // key tile 0 has the longest walk and comes first
  const int h = blockIdx.y, b = blockIdx.z;
  const int d = p.H * DH;
  const int k0 = kt * TK;
  const int first = 2 * kt, n = (p.T + TW - 1) / TW - first;      // query sub-tiles first .. first+n-1 (n >= 1: k0 < T)
  int st0 = status_peek(p.status);
  if (threadIdx.x == 0 && (base & 1023u)) { set_status(p.status, 10); st0 = 10; }

  if (threadIdx.x == 0) {
    mbar_init(kv_full, 1);
    for (int s = 0; s < NST_KV; s++) { mbar_init(qdo_full0 + 8 * s, 1); mbar_init(qdo_empty0 + 8 * s, 1); }
    mbar_init(sdp_full, 1);
    mbar_init(pds_full, 8);
    mbar_init(pds_free, 1);
    mbar_init(acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_kv) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_do) : "memory");
    }
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem = *tmem_slot_ptr;
  const uint32_t tm_s = tmem, tm_dp = tmem + 64, tm_dv = tmem + 128, tm_dk = tmem + 192;

  if (dead) {
  } else if (warp == 8) {
    if (lane == 0) {
      const int row0 = b * p.T;
      auto load_qdo = [&](int ii) {
        const int s = ii % NST_KV;
        const uint32_t full = qdo_full0 + 8 * s, dst = qdo_s + s * 2 * SUB_BYTES;
        mbar_expect_tx(full, 2 * SUB_BYTES);
        tma_load_2d(dst, &map_q, h * DH, row0 + (first + ii) * TW, full);
        tma_load_2d(dst + SUB_BYTES, &map_do, h * DH, row0 + (first + ii) * TW, full);
      };
      mbar_expect_tx(kv_full, 2 * TILE_BYTES);
      tma_load_2d(k_s, &map_kv, d + h * DH, row0 + k0, kv_full);
      tma_load_2d(v_s, &map_kv, 2 * d + h * DH, row0 + k0, kv_full);
      for (int ii = 0; ii < NST_KV && ii < n; ii++) load_qdo(ii);
      const uint32_t id_s = idesc_of(TW, false, false), id_g = idesc_of(DH, false, true);
      bool ok = mbar_wait(kv_full, 0);
      if (!ok) set_status(p.status, 31);
      auto issue_grads = [&](int ii) {     // dV += P^T dO_i, dK += dS^T Q_i
        const uint32_t qi = qdo_s + (ii % NST_KV) * 2 * SUB_BYTES, doi = qi + SUB_BYTES;
#pragma unroll
        for (int kk = 0; kk < TW / 16; kk++) tc_mma(tm_dv, desc_k(pt_s, kk), desc_mn(doi, kk, SUB_BYTES), id_g, (ii > 0 || kk > 0) ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < TW / 16; kk++) tc_mma(tm_dk, desc_k(dst_s, kk), desc_mn(qi, kk, SUB_BYTES), id_g, (ii > 0 || kk > 0) ? 1u : 0u);
      };
      for (int ii = 0; ii < n && ok; ii++) {
        const int s = ii % NST_KV;
        const uint32_t qi = qdo_s + s * 2 * SUB_BYTES, doi = qi + SUB_BYTES;
        if (!mbar_wait(qdo_full0 + 8 * s, (ii / NST_KV) & 1)) { set_status(p.status, 32); ok = false; break; }
        if (ii > 0 && !mbar_wait(pds_full, (ii - 1) & 1)) { set_status(p.status, 33); ok = false; break; }
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < DH / 16; kk++) tc_mma(tm_s, desc_k(k_s, kk), desc_k(qi, kk), id_s, kk > 0 ? 1u : 0u);
#pragma unroll
        for (int kk = 0; kk < DH / 16; kk++) tc_mma(tm_dp, desc_k(v_s, kk), desc_k(doi, kk), id_s, kk > 0 ? 1u : 0u);
        tc_commit(sdp_full);
        if (ii > 0) {
          issue_grads(ii - 1);
          tc_commit(pds_free);
          tc_commit(qdo_empty0 + 8 * ((ii - 1) % NST_KV));
          if (ii - 1 + NST_KV < n) {
            if (!mbar_wait(qdo_empty0 + 8 * ((ii - 1) % NST_KV), ((ii - 1) / NST_KV) & 1)) { set_status(p.status, 34); ok = false; break; }
            load_qdo(ii - 1 + NST_KV);
          }
        }
      }
      if (ok) {
        if (!mbar_wait(pds_full, (n - 1) & 1)) { set_status(p.status, 33); ok = false; }
        if (ok) {
          tc_fence_after();
          issue_grads(n - 1);
        }
      }
      tc_commit(acc_full);
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;                   // key row of the tile
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const int tid = threadIdx.x;                           // 0..255
    bool ok = true;
    for (int ii = 0; ii < n; ii++) {
      const int q0 = (first + ii) * TW;
      // this query sub-tile's log-sum-exp (in log2 units) and delta, shared by all key rows; +inf marks a query past the sequence
      float* vs = vec + (ii & 1) * 128;
      if (tid < 128) {
        const int t = q0 + (tid & 63);
        const long long stat = ((long long)b * p.H + h) * p.T + t;
        vs[tid] = tid < 64 ? (t < p.T ? p.lse[stat] * LOG2E : INFINITY) : (t < p.T ? p.delta[stat] : 0.f);
      }
      softmax_bar();
      bool w = mbar_wait(sdp_full, ii & 1);
      if (!w) set_status(p.status, 35);
      w = __all_sync(0xffffffffu, w);
      if (!w) { ok = false; break; }
      tc_fence_after();
      const int col0 = half * 32;
      const int qcol = q0 + col0 - k0;                      // query index minus key index = qcol + e - row
      const bool maskable = q0 < k0 + TK - 1;              // some query of the sub-tile lies before some key
      uint32_t rs[32], rp[32];
      tc_ld32_nowait(tm_s + lane_off + col0, rs);
      tc_ld32_nowait(tm_dp + lane_off + col0, rp);
      if (ii > 0) {                 // the previous sub-tile's MMAs must have read P^T and dS^T before they are overwritten
        bool f = mbar_wait(pds_free, (ii - 1) & 1);      // (they were issued right behind this sub-tile's score MMAs)
        if (!f) set_status(p.status, 36);
        f = __all_sync(0xffffffffu, f);
        if (!f) { ok = false; break; }
      }
      tc_ld_wait();
      // eight columns at a time: exponentiate, form dS^T, pack and store both 16-byte pieces
      const uint32_t prow = pt_s + (uint32_t)row * 128u, drow = dst_s + (uint32_t)row * 128u;
#pragma unroll
      for (int g = 0; g < 4; g++) {
        float l2[8], dl[8], pe[8], de[8];
        *reinterpret_cast<float4*>(l2) = *reinterpret_cast<const float4*>(vs + col0 + 8 * g);
        *reinterpret_cast<float4*>(l2 + 4) = *reinterpret_cast<const float4*>(vs + col0 + 8 * g + 4);
        *reinterpret_cast<float4*>(dl) = *reinterpret_cast<const float4*>(vs + 64 + col0 + 8 * g);
        *reinterpret_cast<float4*>(dl + 4) = *reinterpret_cast<const float4*>(vs + 64 + col0 + 8 * g + 4);
#pragma unroll
        for (int j = 0; j < 8; j++) {
          const int e = 8 * g + j;
          float x = ex2f(fmaf(__uint_as_float(rs[e]), p.scale_log2, -l2[j]));      // exp2(-inf) = 0 past the sequence
          if (maskable && qcol + e < row) x = 0.f;
          pe[j] = x;
          de[j] = x * (__uint_as_float(rp[e]) - dl[j]);
        }
        const uint32_t piece = (uint32_t)((((col0 >> 3) + g) ^ (row & 7)) << 4);
        sts_v4(prow + piece, pack_bf(pe[0], pe[1]), pack_bf(pe[2], pe[3]), pack_bf(pe[4], pe[5]), pack_bf(pe[6], pe[7]));
        sts_v4(drow + piece, pack_bf(de[0], de[1]), pack_bf(de[2], de[3]), pack_bf(de[4], de[5]), pack_bf(de[6], de[7]));
      }
      tc_fence_before();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(pds_full);
    }
    if (ok) {
      bool w = mbar_wait(acc_full, 0);
      if (!w) set_status(p.status, 37);
      w = __all_sync(0xffffffffu, w);
      if (w) {
        tc_fence_after();
        const int t = k0 + row;
        uint32_t rv[32], rk[32];
        tc_ld32_nowait(tm_dv + lane_off + half * 32, rv);
        tc_ld32_nowait(tm_dk + lane_off + half * 32, rk);
        tc_ld_wait();
        if (t < p.T) {
          bf16_t* out = p.dqkv + ((long long)b * p.T + t) * (3 * d) + h * DH + half * 32;
#pragma unroll
          for (int g = 0; g < 4; g++) {
            uint4 q;
            q.x = pack_bf(__uint_as_float(rk[8 * g]) * p.scale, __uint_as_float(rk[8 * g + 1]) * p.scale);
            q.y = pack_bf(__uint_as_float(rk[8 * g + 2]) * p.scale, __uint_as_float(rk[8 * g + 3]) * p.scale);
            q.z = pack_bf(__uint_as_float(rk[8 * g + 4]) * p.scale, __uint_as_float(rk[8 * g + 5]) * p.scale);
            q.w = pack_bf(__uint_as_float(rk[8 * g + 6]) * p.scale, __uint_as_float(rk[8 * g + 7]) * p.scale);
            *reinterpret_cast<uint4*>(out + d + 8 * g) = q;
            q.x = pack_bf(__uint_as_float(rv[8 * g]), __uint_as_float(rv[8 * g + 1]));
            q.y = pack_bf(__uint_as_float(rv[8 * g + 2]), __uint_as_float(rv[8 * g + 3]));
            q.z = pack_bf(__uint_as_float(rv[8 * g + 4]), __uint_as_float(rv[8 * g + 5]));
            q.w = pack_bf(__uint_as_float(rv[8 * g + 6]), __uint_as_float(rv[8 * g + 7]));
            *reinterpret_cast<uint4*>(out + 2 * d + 8 * g) = q;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

constexpr size_t BWD_Q_SMEM = TILE_BYTES * 3 + NST_Q * 2 * SUB_BYTES + 128;                 // 96.1 KB: two CTAs per SM
constexpr size_t BWD_KV_SMEM = TILE_BYTES * 4 + NST_KV * 2 * SUB_BYTES + 1024 + 128;       // 97.1 KB: two CTAs per SM

constexpr size_t FWD_SMEM = TILE_BYTES * 5 + P_BYTES + 128;   // two CTAs per SM: 2 x (112.1 KB + 1 KB reserved) <= 228 KB

}  // namespace

bool attention_tc_supported(int dh, int d, const void* qkv, const void* o) {
  return dh == DH && d % DH == 0 && ((reinterpret_cast<uintptr_t>(qkv) | reinterpret_cast<uintptr_t>(o)) & 15) == 0;
}

cudaError_t attention_fwd_tc(const void* qkv, void* o, float* lse, int batch, int T, int heads, int* status, cudaStream_t s) {
  const int d = heads * DH;
  CUtensorMap map;
  if (!tc_encode_rows_bf16(&map, qkv, 3LL * d, (long long)batch * T, 3LL * d, TQ)) return cudaErrorInvalidValue;
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) dev = 0;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FWD_SMEM);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  AttnArgs a;
  a.T = T; a.H = heads; a.batch = batch;
  a.scale = 0.125f;
  a.scale_log2 = 0.125f * LOG2E;
  a.o = (bf16_t*)o; a.lse = lse; a.delta = nullptr; a.dqkv = nullptr; a.status = status;
  dim3 grid((T + TQ - 1) / TQ, heads, batch);
  attn_fwd_tc_kernel<<<grid, AT_THREADS, FWD_SMEM, s>>>(map, a);
  return cudaGetLastError();
}

cudaError_t attention_bwd_tc(const void* qkv, const void* o, const void* dout, const float* lse, float* delta, void* dqkv, int batch,
                             int T, int heads, int* status, cudaStream_t s) {
  const int d = heads * DH;
  const long long rows = (long long)batch * T;
  CUtensorMap qkv128, qkv64, do128, do64, o128;        // the same matrices seen as tiles of 128 or 64 rows
  if (!tc_encode_rows_bf16(&qkv128, qkv, 3LL * d, rows, 3LL * d, 128) || !tc_encode_rows_bf16(&qkv64, qkv, 3LL * d, rows, 3LL * d, TW) ||
      !tc_encode_rows_bf16(&do128, dout, d, rows, d, 128) || !tc_encode_rows_bf16(&do64, dout, d, rows, d, TW) ||
      !tc_encode_rows_bf16(&o128, o, d, rows, d, 128))
    return cudaErrorInvalidValue;
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) dev = 0;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    cudaError_t e = cudaFuncSetAttribute(attn_bwd_q_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BWD_Q_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_kv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BWD_KV_SMEM);
    if (e != cudaSuccess) return e;
    attr_set[dev].store(true, std::memory_order_release);
  }
  AttnArgs a;
  a.T = T; a.H = heads; a.batch = batch;
  a.scale = 0.125f;
  a.scale_log2 = 0.125f * LOG2E;
  a.o = nullptr; a.lse = const_cast<float*>(lse); a.delta = delta; a.dqkv = (bf16_t*)dqkv; a.status = status;
  dim3 grid((T + TQ - 1) / TQ, heads, batch);
  // the dQ kernel also produces delta, which the dK/dV kernel reads: it runs first
  attn_bwd_q_tc_kernel<<<grid, BW_THREADS, BWD_Q_SMEM, s>>>(qkv128, qkv64, do128, o128, a);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  attn_bwd_kv_tc_kernel<<<grid, BW_THREADS, BWD_KV_SMEM, s>>>(qkv128, qkv64, do64, a);
  return cudaGetLastError();
}

}  // namespace erase
