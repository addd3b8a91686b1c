// tcgen05 / TMEM / TMA GEMM for sm_100a.  See gemm_tc.cuh for the contract.
//
// Persistent kernel: one CTA per SM walks over 128 x BN output tiles (one split of K each when
// split-K is on); 320 threads:
//   warp 0      TMA producer: one elected thread fills a ring of STAGES shared-memory stages,
//               each holding a 128 x 64 slab of A and a BN x 64 slab of B (bf16, 128-byte swizzle)
//   warp 1      allocates TMEM (two accumulators), then one elected thread issues tcgen05.mma
//               (M=128, N=BN, K=16), four per stage, commits each stage back to the producer and
//               each finished accumulator to the epilogue through mbarriers
//   warps 2..9  epilogue: wait for an accumulator, read their TMEM lane quarter with tcgen05.ld
//               (two warps per quarter, half of the columns each), apply the fused epilogue,
//               store to global memory, hand the accumulator back; this overlaps the next
//               tile's main loop
// Every mbarrier wait is bounded by a clock limit; on expiry the kernel records a status word,
// skips the rest of its work, still frees its TMEM and returns.
//
// Two more kernels further down share these roles and helpers: tc_gemm_pair_kernel (two CTAs of a
// cluster on one 256 x 256 tile, tcgen05 cta_group::2) for GEMMs with enough tiles to fill the 74
// CTA pairs, and tc_wgrad_group_kernel (up to four small weight-gradient GEMMs in one launch).
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"
#include "ew_math.cuh"

#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

namespace erase {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;          // bf16 elements = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
__host__ __device__ constexpr int stages_for(int bn) { return bn == 256 ? 3 : 4; }   // 3 x 48 KB or 4 x 32 KB (or 24 KB)
constexpr uint32_t EPI_BIAS_BYTES = 512;              // up to 128 bias floats per epilogue warp
constexpr int EPI_WARPS = 8;                       // two per TMEM lane quarter, each takes half the columns
constexpr int TC_THREADS = 32 * (2 + EPI_WARPS);
constexpr uint32_t EPI_STAGE_BYTES = 8192;             // two buffers of 32 rows x 128 bytes per epilogue warp
// (one buffer instead of two, as in the CTA-pair kernel, was measured here as well: C3 2 % faster under the
// overlapped schedule, the 512-wide MLP point 3 % slower, C1, C2 and the 128-wide point unchanged: two stay)
#ifndef SINGLE_EPI_BUFS_N
#define SINGLE_EPI_BUFS_N 2
#endif
constexpr int SINGLE_EPI_BUFS = SINGLE_EPI_BUFS_N;     // the single-CTA GEMM kernel's staging buffers per epilogue warp
constexpr uint32_t SINGLE_EPI_BYTES = 4096u * SINGLE_EPI_BUFS;

struct TcArgs {
  int M, N, K;
  void* C;
  long long ldc;
  int c_f32;
  int splits;
  float* ws;
  Epilogue epi;
  int* status;
  long long* dbg;  // optional: clock64 stamps of CTA 0's first tile (development aid), else null
  int tma_c;       // C (or the split-K partials) leaves through shared memory + TMA store
  int plain;       // 1: the epilogue is the identity; 2: bias add only; 0: general
  int* sched;      // {next tile counter, finished CTAs}, zero between launches; null = static round-robin
  float* xcol_out; // CTA-pair kernel: one more, 16-wide column tile at n = N whose first column goes here (GemmArgs::xcol_out)
};

__device__ __forceinline__ float bf2f(uint32_t bits16) { return __uint_as_float(bits16 << 16); }
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Only ReLU is fused (a compare).  GELU's erf chain on the few epilogue warps, and the instruction
// footprint of its inlined copies, made a fused GEMM slower than the GEMM plus a separate
// elementwise pass, so GEMMs that ask for it (or for a pre-activation copy) use the SIMT kernel.

// 8 bf16 held in a 16-byte register quad -> floats
__device__ __forceinline__ void unpack8_bf16(uint4 q, float* out) {
  out[0] = __uint_as_float(q.x << 16); out[1] = __uint_as_float(q.x & 0xffff0000u);
  out[2] = __uint_as_float(q.y << 16); out[3] = __uint_as_float(q.y & 0xffff0000u);
  out[4] = __uint_as_float(q.z << 16); out[5] = __uint_as_float(q.z & 0xffff0000u);
  out[6] = __uint_as_float(q.w << 16); out[7] = __uint_as_float(q.w & 0xffff0000u);
}

// The epilogue's auxiliary operands (residual; multiplier or activation-derivative source) of one
// output row x 32 columns, as raw bf16.  A warp's 32 lanes read 32 different rows, so each of
// these loads is a full memory round trip: they are issued one chunk ahead -- the first chunk
// before the warp starts waiting for its accumulator -- and consumed from registers.
struct Aux32 { uint4 a[4], b[4]; };
__device__ __forceinline__ void aux_issue(const __nv_bfloat16* pa, const __nv_bfloat16* pb, bool row_ok, int n, int N, Aux32& r) {
#pragma unroll
  for (int g = 0; g < 4; g++) {
    const bool ok = row_ok && n + 8 * g < N;   // N is a multiple of 8 whenever an auxiliary operand is present
    r.a[g] = (pa && ok) ? *reinterpret_cast<const uint4*>(pa + n + 8 * g) : make_uint4(0u, 0u, 0u, 0u);
    r.b[g] = (pb && ok) ? *reinterpret_cast<const uint4*>(pb + n + 8 * g) : make_uint4(0u, 0u, 0u, 0u);
  }
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void store8_bf16(__nv_bfloat16* p, int valid, bool vec, const float* v) {
  if (vec) {
    uint4 q;
    q.x = pack2(v[0], v[1]); q.y = pack2(v[2], v[3]); q.z = pack2(v[4], v[5]); q.w = pack2(v[6], v[7]);
    *reinterpret_cast<uint4*>(p) = q;
  } else {
#pragma unroll
    for (int j = 0; j < 8; j++)
      if (j < valid) p[j] = __float2bfloat16_rn(v[j]);
  }
}


// Fused epilogue on 8 accumulator values of one output row (columns n..n+7), in place:
//   v = alpha*acc + bias; v = relu(v); v *= mul; v += res; v *= relu'(dact_src)
// aux_a: 8 residual values, aux_b: 8 multiplier or derivative-source values (raw bf16).
struct F8 { float v[8]; };

// BIAS_REGS = false: bias8 points at this warp's slice of the bias in shared memory (two 16-byte loads);
// true: at eight values the caller already holds in registers.
template <bool BIAS_REGS = false>
__device__ __forceinline__ F8 epilogue_values8(const TcArgs& p, F8 in, const float* bias8, uint4 aux_a, uint4 aux_b) {
  float* v = in.v;
  const Epilogue& e = p.epi;
  float t[8];
  if (e.alpha != 1.f) {
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] *= e.alpha;
  }
  if (e.bias) {
    if (BIAS_REGS) {
#pragma unroll
      for (int j = 0; j < 8; j++) v[j] += bias8[j];
    } else {
      const float4 b0 = *reinterpret_cast<const float4*>(bias8);
      const float4 b1 = *reinterpret_cast<const float4*>(bias8 + 4);
      v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
      v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
    }
  }
  if (e.act == ACT_RELU) {
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] = fmaxf(v[j], 0.f);
  }
  if (e.mul) {          // aux_b holds the multiplier (never together with a derivative source)
    unpack8_bf16(aux_b, t);
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] *= t[j];
  }
  if (e.res) {
    unpack8_bf16(aux_a, t);
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] += t[j];
  }
  if (e.dact == ACT_RELU) {
    unpack8_bf16(aux_b, t);
#pragma unroll
    for (int j = 0; j < 8; j++) v[j] = t[j] > 0.f ? v[j] : 0.f;
  }
  return in;
}

// Direct global store of 8 finished values (used when the output cannot go through TMA).
__device__ __forceinline__ void direct_store8(const TcArgs& p, F8 in, int row, int n, int split) {
  const float* v = in.v;
  const int valid = min(8, p.N - n);
  if (p.splits > 1 || p.c_f32) {
    float* dst = p.splits > 1 ? p.ws + (long long)split * p.M * p.N + (long long)row * p.N + n
                              : (float*)p.C + (long long)row * p.ldc + n;
    if (valid == 8 && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
      reinterpret_cast<float4*>(dst)[0] = make_float4(v[0], v[1], v[2], v[3]);
      reinterpret_cast<float4*>(dst)[1] = make_float4(v[4], v[5], v[6], v[7]);
    } else {
#pragma unroll
      for (int j = 0; j < 8; j++) if (j < valid) dst[j] = v[j];
    }
  } else {
    __nv_bfloat16* dst = (__nv_bfloat16*)p.C + (long long)row * p.ldc + n;
    store8_bf16(dst, valid, valid == 8 && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0), v);
  }
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(src) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the most recent store of this thread have finished reading their shared-memory source
__device__ __forceinline__ void tma_store_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

// Tile order: splits outermost; inside a split, bands of 8 column tiles, and inside a band m
// outer / n inner.  The ~148 tiles in flight at any time then cover about 18 row tiles x 8
// column tiles, so each operand slab fetched from HBM is reused out of L2 by its neighbours.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& mt, int& nt, int& split) {
  const int per_split = tiles_m * tiles_n;
  split = t / per_split;
  const int r = t - split * per_split;
  const int band = r / (8 * tiles_m);
  const int n_first = band * 8;
  const int width = min(8, tiles_n - n_first);
  const int rr = r - band * 8 * tiles_m;
  mt = rr / width;
  nt = n_first + rr - mt * width;
}

// Persistent kernel: CTA c works on tiles c, c + gridDim.x, ... in the order of tile_coords.
// GENERAL = false compiles the epilogue down to "identity or bias add" (forward Linears without
// activation, every dgrad/wgrad without auxiliary operand): a much smaller loop body, which is what
// bounds the epilogue (instruction fetch), so those GEMMs get their own instantiation.
// CE = true (local softmax cross-entropy head, forward): the epilogue turns a logit l into
// exp(l - ref[row]) with a per-row reference known before the GEMM, stores that (bf16) instead of
// the logit and leaves, per row and group of CPW columns, the fp32 sum of the unrounded
// exponentials in ce_psum[row][group]: the head's loss and gradient then need no pass over logits.
template <int BN, bool A_MN, bool B_MN, bool GENERAL, bool CE = false>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c,
               const __grid_constant__ TcArgs p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr uint32_t A_BYTES = BM * BK * 2;
  constexpr uint32_t B_BYTES = BN * BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;            // two accumulators: epilogue(i) overlaps mainloop(i+1)
  constexpr int STAGES = stages_for(BN);
  constexpr int CPW = BN >= 128 ? BN / 2 : 64;      // tile columns per epilogue warp (two warps per lane quarter)

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;          // EPI_WARPS x 4 KB output staging
  const uint32_t bias_base = epi_base + EPI_WARPS * SINGLE_EPI_BYTES;    // EPI_WARPS x CPW floats of bias
  const uint32_t bar_base = bias_base + EPI_WARPS * EPI_BIAS_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  // tile queue: the producer publishes the tiles this CTA works on (dynamic scheduling) to the MMA
  // and epilogue warps through a 4-entry ring
  auto tq_full = [&](int i) { return bar_base + 8u * (2 * STAGES + 6 + i); };
  auto tq_empty = [&](int i) { return bar_base + 8u * (2 * STAGES + 10 + i); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * (SINGLE_EPI_BYTES + EPI_BIAS_BYTES) + 8u * (2 * STAGES + 4));
  volatile int* tile_ring =
      reinterpret_cast<volatile int*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * (SINGLE_EPI_BYTES + EPI_BIAS_BYTES) + 8u * (2 * STAGES + 14));
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int st0 = status_peek(p.status);
#ifdef ERASE_DEV_AIDS   // clock stamps of CTA 0's first tile: compiled in only with -DERASE_DEV_AIDS
  const bool dbg = p.dbg != nullptr && blockIdx.x == 0;
#else
  constexpr bool dbg = false;
#endif
  if (dbg && threadIdx.x == 0) p.dbg[0] = clock64();
  if (threadIdx.x == 32) {   // descriptor fetches overlap the barrier and TMEM set-up
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    if (p.tma_c) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
  }
  const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
  const int total = tiles_m * tiles_n * p.splits;
  const int kchunk = (((p.K + p.splits - 1) / p.splits) + BK - 1) / BK * BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS);
    }
    for (int i = 0; i < 4; i++) {
      mbar_init(tq_full(i), 1);
      mbar_init(tq_empty(i), 1 + EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  if (dbg && threadIdx.x == 0) p.dbg[1] = clock64();

  if (dead) {
    // the step is already void: do nothing but free TMEM below
  } else if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0, slot = 0;
      bool ok = true;
      int t = (int)blockIdx.x < total ? (int)blockIdx.x : -1;
      while (ok) {
        // publish the tile (or the end marker -1) to the other roles
        if (!mbar_wait(tq_empty(slot & 3), ((slot >> 2) & 1) ^ 1)) { atomicExch(p.status, 5); ok = false; break; }
        tile_ring[slot & 3] = t;
        mbar_arrive(tq_full(slot & 3));
        slot++;
        if (t < 0) break;
        // claim the next tile now: the atomic's latency hides behind this tile's loads
        int next = p.sched ? (int)gridDim.x + atomicAdd(p.sched, 1) : t + (int)gridDim.x;
        int mt, nt, split;
        tile_coords(t, tiles_m, tiles_n, mt, nt, split);
        const int m0 = mt * BM, n0 = nt * BN;
        const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicExch(p.status, 1); ok = false; break; }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          const uint32_t a_dst = smem_base + s * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const int k0 = kbeg + kb * BK;
          if (!A_MN) {
            tma_load_2d(a_dst, &map_a, k0, m0, full_bar(s));
          } else {
#pragma unroll
            for (int a = 0; a < BM / 64; a++) tma_load_2d(a_dst + a * (BK * 128), &map_a, m0 + a * 64, k0, full_bar(s));
          }
          if (!B_MN) {
            tma_load_2d(b_dst, &map_b, k0, n0, full_bar(s));
          } else {
#pragma unroll
            for (int a = 0; a < BN / 64; a++) tma_load_2d(b_dst + a * (BK * 128), &map_b, n0 + a * 64, k0, full_bar(s));
          }
          if (dbg && it == 0) p.dbg[2] = clock64();
          if (dbg && it == 3) p.dbg[8] = clock64();
        }
        t = next < total ? next : -1;
      }
      if (!ok) {  // give copies already in flight time to land before the CTA's shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 x bf16, majors, N>>3 at bit 17, M>>4 at bit 24
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (;; lt++) {
        if (!mbar_wait(tq_full(lt & 3), (lt >> 2) & 1)) { atomicExch(p.status, 6); break; }
        const int t = tile_ring[lt & 3];
        mbar_arrive(tq_empty(lt & 3));
        if (t < 0 || !ok) break;
        const int split = t / (tiles_m * tiles_n);
        const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
        if (!mbar_wait(tempty_bar(ab), aph ^ 1)) { atomicExch(p.status, 4); ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + ab * BN;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(full_bar(s), ph)) { atomicExch(p.status, 2); ok = false; break; }
          tc_fence_after();
          if (dbg && it == 0) p.dbg[3] = clock64();
          if (dbg && it == 3) p.dbg[9] = clock64();
          const uint32_t a_src = smem_base + s * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            // K-major: rows of 128 bytes, 8-row groups 1024 bytes apart; a K step of 16 elements is
            //          32 bytes inside the swizzled row.
            // MN-major: 64-element (128-byte) runs along M/N, one per K index; 8 K rows form a
            //          1024-byte group (stride offset), the next 64 M/N elements sit BK*128 bytes
            //          further (leading offset); a K step of 16 is 16 rows = 2048 bytes.
            const uint64_t ad = A_MN ? smem_desc(a_src + k * (UMMA_K * 128), BK * 128, 1024)
                                     : smem_desc(a_src + k * (UMMA_K * 2), 16, 1024);
            const uint64_t bd = B_MN ? smem_desc(b_src + k * (UMMA_K * 128), BK * 128, 1024)
                                     : smem_desc(b_src + k * (UMMA_K * 2), 16, 1024);
            tc_mma(tmem_d, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));  // stage may be refilled once these MMAs have read it
        }
        tc_commit(tfull_bar(ab));   // accumulator ab complete (also fires when the loop bailed out)
        if (dbg && lt == 0) p.dbg[4] = clock64();
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    // A warp owns 32 rows (its TMEM lane quarter) x 64 columns of the tile, as two 32-column
    // chunks.  Finished values go to a 4 KB staging buffer in shared memory (one 128-byte row
    // per lane, 16-byte pieces XOR-swizzled with the row so that writes are conflict-free and
    // match the tensor map's 128-byte swizzle) and leave with one TMA store per 128-byte-wide
    // box, which also clips the M and N tails.  Outputs that cannot be described to TMA
    // (unaligned leading dimension) are stored directly.
    const int ew = warp - 2;
    const int q = warp & 3;                       // TMEM lane quarter this warp may read
    const int cbeg = (ew / 4) * CPW;              // first tile column of this warp
    const bool active = cbeg < BN;                // BN = 64: only one warp per quarter has columns
    const uint32_t stage0 = epi_base + ew * SINGLE_EPI_BYTES;   // two 4 KB buffers, used alternately
    uint32_t sbuf = 0;
    float* bias_s = reinterpret_cast<float*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * SINGLE_EPI_BYTES + ew * EPI_BIAS_BYTES);
    const bool out_f32 = p.splits > 1 || p.c_f32;
    bool store_pending = false;                   // lane 0: TMA stores may still be reading the staging buffers
    uint32_t lt = 0;
    for (;; lt++) {
      int t = -1;
      if (lane == 0) {
        if (mbar_wait(tq_full(lt & 3), (lt >> 2) & 1)) {
          t = tile_ring[lt & 3];
          mbar_arrive(tq_empty(lt & 3));
        } else {
          atomicExch(p.status, 7);
        }
      }
      t = __shfl_sync(0xffffffffu, t, 0);
      if (t < 0) break;
      int mt, nt, split;
      tile_coords(t, tiles_m, tiles_n, mt, nt, split);
      const int m0 = mt * BM, n0 = nt * BN;
      const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
      const bool empty_k = kend <= kbeg;          // a trailing split with no K range: partial sum is zero
      const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
      if (p.epi.bias && active) {   // fetch this warp's bias slice now; the latency hides behind the MMAs
        __syncwarp();
        for (int j = lane; j < CPW; j += 32) {
          const int n = n0 + cbeg + j;
          bias_s[j] = n < p.N ? __ldg(p.epi.bias + n) : 0.f;
        }
        __syncwarp();
      }
      const int row = m0 + q * 32 + lane;
      const bool row_ok = row < p.M;
      float ce_ref2 = 0.f, ce_sum = 0.f;          // CE: this row's reference (in log2 units) and its running sum
      if (CE && row_ok) ce_ref2 = __ldg(p.epi.ce_ref + row) * 1.4426950408889634f;
      // auxiliary operands of this thread's row (raw bf16), fetched one 32-column chunk ahead
      const __nv_bfloat16* aux_pa = nullptr;
      const __nv_bfloat16* aux_pb = nullptr;
      Aux32 aux_cur, aux_nxt;
      if (GENERAL && !p.plain && p.splits == 1) {
        const long long ro = (long long)row * p.epi.ld_aux;
        if (p.epi.res) aux_pa = (const __nv_bfloat16*)p.epi.res + ro;
        const void* bsrc = p.epi.mul ? p.epi.mul : (p.epi.dact != ACT_NONE ? p.epi.dact_src : nullptr);
        if (bsrc) aux_pb = (const __nv_bfloat16*)bsrc + ro;
        if (active && n0 + cbeg < p.N && (aux_pa || aux_pb)) {   // in flight while the MMAs still run
          aux_issue(aux_pa, aux_pb, row_ok, n0 + cbeg, p.N, aux_nxt);
        }
      }
      const bool use_aux = GENERAL && (aux_pa || aux_pb);
      bool ok = mbar_wait(tfull_bar(ab), aph);
      if (!ok) atomicExch(p.status, 3);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      if (dbg && lt == 0 && threadIdx.x == 64) p.dbg[5] = clock64();
#ifdef ERASE_DEV_AIDS
      const long long dflags = p.dbg ? p.dbg[15] : 0;
#else
      constexpr long long dflags = 0;
#endif
      if (active && n0 + cbeg < p.N) {
        {
          const bool via_tma = p.tma_c != 0;
          const bool f32 = out_f32;
#pragma unroll 1
          for (int cc = 0; cc < CPW; cc += 32) {
            const int c0 = cbeg + cc;
            if (n0 + c0 >= p.N) break;  // warp-uniform
            if (GENERAL && use_aux) {
              aux_cur = aux_nxt;
              if (cc + 32 < CPW && n0 + c0 + 32 < p.N) aux_issue(aux_pa, aux_pb, row_ok, n0 + c0 + 32, p.N, aux_nxt);
            }
            uint32_t r[32];
            if (!empty_k && !(dflags & 2)) {
              tc_ld32(tmem_base + ab * BN + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
            } else {
#pragma unroll
              for (int j = 0; j < 32; j++) r[j] = 0u;
            }
            if (via_tma && (f32 || (cc & 63) == 0)) { // next staging buffer: its previous store (two stores ago) must have read it
              if (SINGLE_EPI_BUFS == 2) {
                sbuf ^= 1;
                if (lane == 0 && store_pending) tma_store_wait_read1();
              } else if (lane == 0 && store_pending) {
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
              }
              __syncwarp();
            }
            const uint32_t stage = stage0 + sbuf * 4096;
            const uint32_t my_row = stage + lane * 128;
#pragma unroll
            for (int g8 = 0; g8 < 4; g8++) {
              const int n = n0 + c0 + g8 * 8;
              F8 f;
#pragma unroll
              for (int j = 0; j < 8; j++) f.v[j] = __uint_as_float(r[g8 * 8 + j]);
              if (CE) {                    // logit -> exp(logit - reference); columns past N contribute nothing
                const float4 b0 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8);
                const float4 b1 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8 + 4);
                const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                const bool full = n + 8 <= p.N;
#pragma unroll
                for (int j = 0; j < 8; j++) {
                  float e = ex2_approx(fmaf(f.v[j] + bb[j], 1.4426950408889634f, -ce_ref2));
                  if (!full && n + j >= p.N) e = 0.f;
                  ce_sum += e;
                  f.v[j] = e;
                }
              } else if (p.plain == 2) {          // bias only: the common forward case, kept free of the general path
                const float4 b0 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8);
                const float4 b1 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8 + 4);
                f.v[0] += b0.x; f.v[1] += b0.y; f.v[2] += b0.z; f.v[3] += b0.w;
                f.v[4] += b1.x; f.v[5] += b1.y; f.v[6] += b1.z; f.v[7] += b1.w;
              } else if (GENERAL && row_ok && n < p.N && p.splits == 1 && !p.plain) {
                f = epilogue_values8(p, f, bias_s + cc + g8 * 8, aux_cur.a[g8], aux_cur.b[g8]);
              }
              const float* v = f.v;
              if (!via_tma) {
                if (row_ok && n < p.N && !(dflags & 1)) direct_store8(p, f, row, n, split);
              } else if (f32) {                      // 32 floats per row: pieces 2*g8 and 2*g8+1 of the 128-byte row
                const uint32_t s0 = my_row + (((2 * g8) ^ (lane & 7)) << 4), s1 = my_row + (((2 * g8 + 1) ^ (lane & 7)) << 4);
                st_shared_v4(s0, __float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
                st_shared_v4(s1, __float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
              } else {                               // 64 bf16 per row: piece (cc mod 64)/8 + g8
                const uint32_t s0 = my_row + (((((cc & 63) >> 3) + g8) ^ (lane & 7)) << 4);
                st_shared_v4(s0, pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
              }
            }
            const bool last_chunk = (cc & 63) == 32 || n0 + c0 + 32 >= p.N;
            if (via_tma && (f32 || last_chunk)) {
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (dbg && lt == 0 && threadIdx.x == 64 && p.dbg[10] == 0) p.dbg[10] = clock64();
              if (lane == 0 && !(dflags & 1)) {
                const int x = f32 ? n0 + c0 : n0 + cbeg + (cc & ~63), y = m0 + q * 32;
                if (p.splits > 1) tma_store_3d(&map_c, stage, x, y, split);
                else tma_store_2d(&map_c, stage, x, y);
                tma_store_commit();
                store_pending = true;
                if (dbg && lt == 0 && threadIdx.x == 64 && p.dbg[11] == 0) p.dbg[11] = clock64();
              }
            }
          }
        }
      }
      if (CE && active && row_ok && n0 + cbeg < p.N)
        p.epi.ce_psum[(long long)row * p.epi.ce_groups + (n0 + cbeg) / CPW] = ce_sum;
      // all TMEM reads of this warp are complete (tcgen05.wait::ld): hand the accumulator back
      if (dbg && lt == 0 && threadIdx.x == 64) p.dbg[12] = clock64();
      tc_fence_before();
      __syncwarp();
      if (dbg && lt == 0 && threadIdx.x == 64) p.dbg[13] = clock64();
      if (lane == 0) mbar_arrive(tempty_bar(ab));
      if (dbg && lt == 0 && threadIdx.x == 64) p.dbg[6] = clock64();
    }
    if (lane == 0 && store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores complete before exit
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (p.sched && threadIdx.x == 0) {   // the CTA that finishes last leaves the scheduler words at zero
    __threadfence();
    if (atomicAdd(p.sched + 1, 1) == (int)gridDim.x - 1) {
      p.sched[0] = 0;
      p.sched[1] = 0;
      __threadfence();
    }
  }
  if (dbg && threadIdx.x == 0) p.dbg[7] = clock64();
}

// =================================================================================================
// CTA-pair kernel (tcgen05 cta_group::2): two CTAs of a cluster, on neighbouring SMs, share one
// 256 x 256 output tile.  Each CTA stages its own 128 rows of A and HALF of the B slab (128 of the
// 256 columns) per K block; the pair's tensor cores read both halves, so every SM moves 32 KB per
// K block through shared memory and L2 instead of the 48 KB of the single-CTA 128 x 256 tile --
// which is what bounds the large GEMMs.  The leader CTA (cluster rank 0) issues the MMAs
// (M = 256, N = 256, K = 16) for both; the accumulator rows 0..127 land in the leader's TMEM,
// rows 128..255 in the peer's, and each CTA's epilogue warps drain their own.
//   full[s]    leader only: TMA bytes of BOTH CTAs' stage s have landed (both CTAs' copies signal it)
//   empty[s]   per CTA: the MMAs that read stage s are done (one commit, delivered to both CTAs)
//   tfull[a]   per CTA: accumulator a is complete (delivered to both CTAs)
//   tempty[a]  leader only: both CTAs' epilogue warps have drained accumulator a (the peer's warps
//              arrive on it through the cluster's shared-memory window)
// Tiles are assigned round-robin to clusters, in the order of tile_coords.  The output must be
// describable to TMA (it leaves through staged TMA stores); GENERAL as in tc_gemm_kernel.
constexpr int PAIR_BN = 256;
#ifndef PAIR_STAGES_N
#define PAIR_STAGES_N 5
#endif
// One staging buffer per epilogue warp, not two: the warp then waits for its previous store to have read the
// buffer before refilling it, which costs the epilogue-bound short contractions a few per cent when they run
// alone, but the CTA takes 194 KB of shared memory instead of 226 KB and other streams' small kernels find
// room beside it: under the overlapped schedule every configuration measured 0.5-1 % faster.
#ifndef PAIR_EPI_BUFS_N
#define PAIR_EPI_BUFS_N 1
#endif
constexpr int PAIR_STAGES = PAIR_STAGES_N;
constexpr int PAIR_EPI_BUFS = PAIR_EPI_BUFS_N;                      // 4 KB output staging buffers per epilogue warp
constexpr uint32_t PAIR_EPI_BYTES = 4096u * PAIR_EPI_BUFS;
constexpr uint32_t PAIR_BIAS_BYTES = 2u * 2u * (PAIR_BN / 2) * 4u;   // two column halves x two tile parities x 128 floats
constexpr uint32_t PAIR_STAGE_BYTES = 2u * BM * BK * 2u;   // 128 x 64 of A + 128 x 64 of B, bf16

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {   // same offset in CTA `rank` of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// copy into this CTA's shared memory; the byte count is credited to `bar`, which may be the peer's
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {   // arrives on `bar` in both CTAs of the pair
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

template <bool A_MN, bool B_MN, bool GENERAL, bool CE = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_c, const __grid_constant__ TcArgs p, const uint32_t tmem_cols) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  constexpr int BN = PAIR_BN;
  constexpr int STAGES = PAIR_STAGES;
  constexpr uint32_t A_BYTES = BM * BK * 2;
  constexpr uint32_t STAGE_BYTES = PAIR_STAGE_BYTES;
  constexpr int CPW = BN / 2;

  // The operand stages need a 1024-byte aligned base (128-byte swizzle); the kernel has no static shared
  // memory, so the dynamic array starts the CTA's window.  Should it ever not, the kernel reports it and works on nothing.
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;
  const uint32_t bar_base = epi_base + EPI_WARPS * PAIR_EPI_BYTES + PAIR_BIAS_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * PAIR_EPI_BYTES + PAIR_BIAS_BYTES + 8u * (2 * STAGES + 4));
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* dead_flag_ptr = reinterpret_cast<volatile int*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * PAIR_EPI_BYTES + PAIR_BIAS_BYTES + 8u * (2 * STAGES + 6));
  if (threadIdx.x == 0) {
    const bool misaligned = (smem_base & 1023u) != 0;
    if (misaligned) atomicExch(p.status, 9);
    *dead_flag_ptr = (misaligned || status_peek(p.status) != 0) ? 1 : 0;
  }
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int naccum = tmem_cols >= 2u * BN ? 2 : 1;      // accumulators in TMEM (two: epilogue overlaps the next main loop)
  if (threadIdx.x == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
  }
  // xcol: behind the column tiles of C comes one narrow tile per row tile, at n = N (a multiple of BN), 16 wide
  const bool xcol = p.xcol_out != nullptr;
  const int tiles_n_main = (p.N + BN - 1) / BN;
  const int tiles_m = (p.M + 2 * BM - 1) / (2 * BM), tiles_n = tiles_n_main + (xcol ? 1 : 0);
  constexpr int XCOL_N = 16;
  const int total = tiles_m * tiles_n * p.splits;
  const int kchunk = (((p.K + p.splits - 1) / p.splits) + BK - 1) / BK * BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 2 * EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {   // one warp of EACH CTA of the pair takes part in the allocation
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();      // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
#ifdef ERASE_DEV_AIDS
  if (p.dbg && threadIdx.x == 0 && cluster_id == 0) p.dbg[8 + rank] = (long long)tmem_base;
#endif
  int dead;   // both CTAs of the pair take the LEADER's reading, so that they skip (or work) together
  asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(dead) : "r"(map_to_cta(bar_base + 8u * (2 * STAGES + 6), 0)) : "memory");

  if (dead) {
    // the step is already void: do nothing but free TMEM below
  } else if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = cluster_id; t < total && ok; t += n_clusters) {
        int mt, nt, split;
        tile_coords(t, tiles_m, tiles_n, mt, nt, split);
        const int m0 = mt * 2 * BM + (int)rank * BM;        // this CTA's 128 rows of A
        const bool narrow = xcol && nt == tiles_n_main;
        const int nb0 = narrow ? p.N + (int)rank * (XCOL_N / 2) : nt * BN + (int)rank * (BN / 2);     // this CTA's half of the tile's B columns
        const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
#ifdef ERASE_DEV_AIDS
          const long long w0 = clock64();
#endif
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicExch(p.status, 1); ok = false; break; }
#ifdef ERASE_DEV_AIDS
          if (p.dbg && blockIdx.x == 0) p.dbg[7] += clock64() - w0;      // producer: waiting for a free stage
#endif
          if (leader) mbar_expect_tx(full_bar(s), narrow ? 2 * (A_BYTES + BK * 128) : 2 * STAGE_BYTES);   // this CTA's bytes and the peer's
          const uint32_t lfull = map_to_cta(full_bar(s), 0);
          const uint32_t a_dst = smem_base + s * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const int k0 = kbeg + kb * BK;
          if (!A_MN) {
            tma_load_2d_pair(a_dst, &map_a, k0, m0, lfull);
          } else {
#pragma unroll
            for (int a = 0; a < BM / 64; a++) tma_load_2d_pair(a_dst + a * (BK * 128), &map_a, m0 + a * 64, k0, lfull);
          }
          if (!B_MN) {
            tma_load_2d_pair(b_dst, &map_b, k0, nb0, lfull);
          } else {
#pragma unroll
            for (int a = 0; a < (narrow ? 1 : BN / 128); a++) tma_load_2d_pair(b_dst + a * (BK * 128), &map_b, nb0 + a * 64, k0, lfull);
          }
        }
      }
      if (!ok) {  // give copies already in flight time to land before the CTA's shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only) ------------------------------
    if (lane == 0 && leader) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int t = cluster_id; t < total && ok; t += n_clusters, lt++) {
        int mt_, nt_, split;
        tile_coords(t, tiles_m, tiles_n, mt_, nt_, split);
        const bool narrow = xcol && nt_ == tiles_n_main;
        const uint32_t idesc_t = narrow ? ((idesc & ~(0x3Fu << 17)) | ((uint32_t)(XCOL_N >> 3) << 17)) : idesc;
        const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        const uint32_t ab = naccum == 2 ? (lt & 1) : 0u, aph = naccum == 2 ? ((lt >> 1) & 1) : (lt & 1);
#ifdef ERASE_DEV_AIDS
        const bool acct = p.dbg && blockIdx.x == 0;
        long long w0 = acct ? clock64() : 0;
        if (acct && lt == 0) p.dbg[0] = w0;
#endif
        if (!mbar_wait(tempty_bar(ab), aph ^ 1)) { atomicExch(p.status, 4); ok = false; break; }
#ifdef ERASE_DEV_AIDS
        if (acct) { p.dbg[1] += clock64() - w0; p.dbg[10] += 1; }       // MMA thread: waiting for a drained accumulator
#endif
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + ab * BN;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
#ifdef ERASE_DEV_AIDS
          w0 = acct ? clock64() : 0;
#endif
          if (!mbar_wait(full_bar(s), ph)) { atomicExch(p.status, 2); ok = false; break; }
#ifdef ERASE_DEV_AIDS
          if (acct) { const long long w1 = clock64(); p.dbg[2] += w1 - w0; p.dbg[3] = w1; }   // MMA thread: waiting for operands
#endif
          tc_fence_after();
          const uint32_t a_src = smem_base + s * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            // the same descriptors address this CTA's and the peer's shared memory (identical layout)
            const uint64_t ad = A_MN ? smem_desc(a_src + k * (UMMA_K * 128), BK * 128, 1024)
                                     : smem_desc(a_src + k * (UMMA_K * 2), 16, 1024);
            const uint64_t bd = B_MN ? smem_desc(b_src + k * (UMMA_K * 128), BK * 128, 1024)
                                     : smem_desc(b_src + k * (UMMA_K * 2), 16, 1024);
            tc_mma_pair(tmem_d, ad, bd, idesc_t, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(s));
        }
        tc_commit_pair(tfull_bar(ab));
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs, own 128 rows) ------------------------------
    const int ew = warp - 2;
    const int q = warp & 3;
    const int cbeg = (ew / 4) * CPW;
    const uint32_t stage0 = epi_base + ew * PAIR_EPI_BYTES;
    uint32_t sbuf = 0;
    const bool f32 = p.splits > 1 || p.c_f32;
    const uint32_t ltempty0 = map_to_cta(tempty_bar(0), 0), ltempty1 = map_to_cta(tempty_bar(1), 0);
    bool store_pending = false;
    uint32_t lt = 0;
    for (int t = cluster_id; t < total; t += n_clusters, lt++) {
      int mt, nt, split;
      tile_coords(t, tiles_m, tiles_n, mt, nt, split);
      const int m0 = mt * 2 * BM + (int)rank * BM, n0 = nt * BN;
      const int kbeg = split * kchunk, kend = min(p.K, kbeg + kchunk);
      const bool empty_k = kend <= kbeg;
      const uint32_t ab = naccum == 2 ? (lt & 1) : 0u, aph = naccum == 2 ? ((lt >> 1) & 1) : (lt & 1);
      // Bias: the four warps that share a column half share one 128-float slice per tile parity.  Each warp
      // fetches the slice into registers now (the latency hides behind the MMAs) and writes it -- every warp
      // the same values -- once the tile's accumulator is complete: by then every warp of the pair has drained
      // the tile before the previous one, the last reader of this parity's slice.  A warp reads only behind
      // its own writes, so no barrier between the warps is needed.
      const bool need_bias = p.epi.bias != nullptr && p.splits == 1;
      float* bias_s = reinterpret_cast<float*>(gen_base + STAGES * STAGE_BYTES + EPI_WARPS * PAIR_EPI_BYTES) + ((ew / 4) * 2 + (lt & 1)) * CPW;
      float4 bias_pre = make_float4(0.f, 0.f, 0.f, 0.f);
      if (need_bias) {
        const int n = n0 + cbeg + lane * 4;
        const float* bp = p.epi.bias + n;
        if (n + 4 <= p.N) {
          bias_pre = __ldg(reinterpret_cast<const float4*>(bp));
        } else {
          if (n < p.N) bias_pre.x = __ldg(bp);
          if (n + 1 < p.N) bias_pre.y = __ldg(bp + 1);
          if (n + 2 < p.N) bias_pre.z = __ldg(bp + 2);
        }
      }
      const int row = m0 + q * 32 + lane;
      const bool row_ok = row < p.M;
      float ce_ref2 = 0.f, ce_sum = 0.f;          // CE: this row's reference (in log2 units) and its running sum
      if (CE && row_ok) ce_ref2 = __ldg(p.epi.ce_ref + row) * 1.4426950408889634f;
      // auxiliary operands of this thread's row (raw bf16), fetched one 32-column chunk ahead
      const __nv_bfloat16* aux_pa = nullptr;
      const __nv_bfloat16* aux_pb = nullptr;
      Aux32 aux_cur, aux_nxt;
      if (GENERAL && !p.plain && p.splits == 1) {
        const long long ro = (long long)row * p.epi.ld_aux;
        if (p.epi.res) aux_pa = (const __nv_bfloat16*)p.epi.res + ro;
        const void* bsrc = p.epi.mul ? p.epi.mul : (p.epi.dact != ACT_NONE ? p.epi.dact_src : nullptr);
        if (bsrc) aux_pb = (const __nv_bfloat16*)bsrc + ro;
        if (n0 + cbeg < p.N && (aux_pa || aux_pb)) aux_issue(aux_pa, aux_pb, row_ok, n0 + cbeg, p.N, aux_nxt);
      }
      const bool use_aux = GENERAL && (aux_pa || aux_pb);
#ifdef ERASE_DEV_AIDS
      const bool acct = p.dbg && blockIdx.x == 0 && threadIdx.x == 64;
      const long long e0 = acct ? clock64() : 0;
#endif
      bool ok = mbar_wait(tfull_bar(ab), aph);
      if (!ok) atomicExch(p.status, 3);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#ifdef ERASE_DEV_AIDS
      const long long e1 = acct ? clock64() : 0;
      if (acct) p.dbg[4] += e1 - e0;                                   // epilogue warp 0: waiting for a finished accumulator
#endif
      if (need_bias) {
        *reinterpret_cast<float4*>(bias_s + lane * 4) = bias_pre;
        __syncwarp();
      }
      const bool rows_in = m0 + q * 32 < p.M;      // warp-uniform: any of this warp's 32 rows inside the matrix
#ifdef ERASE_DEV_AIDS
      const long long dflags = p.dbg ? p.dbg[15] : 0;   // 1: no TMA stores, 2: no TMEM loads, 4: no staging writes
#else
      constexpr long long dflags = 0;
#endif
      if (xcol && nt == tiles_n_main) {            // the narrow tile: its first column is the extra product
        if (cbeg == 0 && rows_in) {
          uint32_t r[32];
          if (!empty_k) {
            tc_ld32(tmem_base + ab * BN + ((uint32_t)(q * 32) << 16), r);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j++) r[j] = 0u;
          }
          if (row_ok) p.xcol_out[row] = __uint_as_float(r[0]);
        }
      } else if (n0 + cbeg < p.N) {
#pragma unroll 1
        for (int cc = 0; cc < CPW; cc += 32) {
          const int c0 = cbeg + cc;
          if (n0 + c0 >= p.N) break;  // warp-uniform
          if (GENERAL && use_aux) {
            aux_cur = aux_nxt;
            if (cc + 32 < CPW && n0 + c0 + 32 < p.N) aux_issue(aux_pa, aux_pb, row_ok, n0 + c0 + 32, p.N, aux_nxt);
          }
          uint32_t r[32];
          const bool from_tmem = !empty_k && !(dflags & 2);
          if (from_tmem) tc_ld32_issue(tmem_base + ab * BN + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
          if (from_tmem) {
            tc_ld_wait(r);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j++) r[j] = 0u;
          }
          if (f32 || (cc & 63) == 0) {
            if (PAIR_EPI_BUFS == 2) {
              sbuf ^= 1;
              if (lane == 0 && store_pending) tma_store_wait_read1();
            } else if (lane == 0 && store_pending) {
              asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            }
            __syncwarp();
          }
          const uint32_t stage = stage0 + sbuf * 4096;
          const uint32_t my_row = stage + lane * 128;
#pragma unroll
          for (int g8 = 0; g8 < 4; g8++) {
            F8 f;
            float* v = f.v;
#pragma unroll
            for (int j = 0; j < 8; j++) v[j] = __uint_as_float(r[g8 * 8 + j]);
            if (CE) {                      // logit -> exp(logit - reference); columns past N contribute nothing
              const float4 b0 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8);
              const float4 b1 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8 + 4);
              const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
              const int n = n0 + c0 + g8 * 8;
              const bool full = n + 8 <= p.N;
#pragma unroll
              for (int j = 0; j < 8; j++) {
                float e = ex2_approx(fmaf(v[j] + bb[j], 1.4426950408889634f, -ce_ref2));
                if (!full && n + j >= p.N) e = 0.f;
                ce_sum += e;
                v[j] = e;
              }
            } else if (p.plain == 2) {
              const float4 b0 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8);
              const float4 b1 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8 + 4);
              v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
              v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
            } else if (GENERAL && !p.plain && p.splits == 1 && row_ok && n0 + c0 + g8 * 8 < p.N) {
              f = epilogue_values8(p, f, bias_s + cc + g8 * 8, aux_cur.a[g8], aux_cur.b[g8]);
            }
            if (dflags & 4) {
              if (v[0] == 123.456f) st_shared_v4(my_row, 0u, 0u, 0u, 0u);     // keeps the values alive without the writes
            } else if (f32) {
              const uint32_t s0 = my_row + (((2 * g8) ^ (lane & 7)) << 4), s1 = my_row + (((2 * g8 + 1) ^ (lane & 7)) << 4);
              st_shared_v4(s0, __float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
              st_shared_v4(s1, __float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
            } else {
              const uint32_t s0 = my_row + (((((cc & 63) >> 3) + g8) ^ (lane & 7)) << 4);
              st_shared_v4(s0, pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
            }
          }
          const bool last_chunk = (cc & 63) == 32 || n0 + c0 + 32 >= p.N;
          if (f32 || last_chunk) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0 && rows_in && !(dflags & 1)) {
              const int x = f32 ? n0 + c0 : n0 + cbeg + (cc & ~63), y = m0 + q * 32;
              if (p.splits > 1) tma_store_3d(&map_c, stage, x, y, split);
              else tma_store_2d(&map_c, stage, x, y);
              tma_store_commit();
              store_pending = true;
            }
          }
        }
      }
      if (CE && row_ok && n0 + cbeg < p.N)
        p.epi.ce_psum[(long long)row * p.epi.ce_groups + (n0 + cbeg) / CPW] = ce_sum;
      tc_fence_before();
      __syncwarp();
#ifdef ERASE_DEV_AIDS
      if (acct) p.dbg[5] += clock64() - e1;                            // epilogue warp 0: draining one accumulator
#endif
      if (lane == 0) {   // accumulator drained: tell the leader's MMA thread
        if (leader) mbar_arrive(tempty_bar(ab));
        else mbar_arrive_cluster(ab ? ltempty1 : ltempty0);
      }
    }
    if (lane == 0 && store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // Neither CTA may leave (or free its TMEM) while the other can still read its shared memory,
  // write its TMEM or signal its barriers.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// =================================================================================================
// Grouped weight-gradient kernel: up to four small wgrad GEMMs (dW_i = dY_i^T X_i, both operands
// MN-major, fp32 split-K partials) in ONE launch.  A block's weight gradients are each a few
// 128 x 128 tiles; launched one by one they pay launch, prologue, pipeline fill and drain four
// times with most SMs idle.  Here a tile index runs over all problems (problem, split, m, n), one
// CTA per SM takes tiles round-robin, and the roles are those of tc_gemm_kernel (BN = 128,
// identity epilogue, partials TMA-stored through each problem's 3-D map).
constexpr int GROUP_MAX = 4;
struct GroupProblem {
  int M, N, K, splits, kchunk, tiles_m, tiles_n, tile_begin;
};
struct GroupArgs {
  int nprob, total;
  int* status;
  GroupProblem prob[GROUP_MAX];
};
struct GroupMaps {
  CUtensorMap a[GROUP_MAX], b[GROUP_MAX], c[GROUP_MAX];
};

__device__ __forceinline__ void group_tile(const GroupArgs& g, int t, int& pi, int& mt, int& nt, int& split) {
  pi = 0;
  while (pi + 1 < g.nprob && t >= g.prob[pi + 1].tile_begin) pi++;
  const GroupProblem& q = g.prob[pi];
  const int local = t - q.tile_begin, per = q.tiles_m * q.tiles_n;
  split = local / per;
  const int r = local - split * per;
  mt = r / q.tiles_n;
  nt = r - mt * q.tiles_n;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_wgrad_group_kernel(const __grid_constant__ GroupMaps maps, const __grid_constant__ GroupArgs g) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int BN = 128;
  constexpr uint32_t A_BYTES = BM * BK * 2;
  constexpr uint32_t B_BYTES = BN * BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;
  constexpr int STAGES = 4;
  constexpr int CPW = BN / 2;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;
  const uint32_t bar_base = epi_base + EPI_WARPS * EPI_STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(gen_base + (bar_base - smem_base) + 8u * (2 * STAGES + 4));
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int st0 = status_peek(g.status);
  if (threadIdx.x == 32) {
    for (int i = 0; i < g.nprob; i++) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.a[i]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.b[i]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.c[i]) : "memory");
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  if (dead) {
    // the step is already void: do nothing but free TMEM below
  } else if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < g.total && ok; t += gridDim.x) {
        int pi, mt, nt, split;
        group_tile(g, t, pi, mt, nt, split);
        const GroupProblem& q = g.prob[pi];
        const int m0 = mt * BM, n0 = nt * BN;
        const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicExch(g.status, 1); ok = false; break; }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          const uint32_t a_dst = smem_base + s * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const int k0 = kbeg + kb * BK;
#pragma unroll
          for (int a = 0; a < BM / 64; a++) tma_load_2d(a_dst + a * (BK * 128), &maps.a[pi], m0 + a * 64, k0, full_bar(s));
#pragma unroll
          for (int a = 0; a < BN / 64; a++) tma_load_2d(b_dst + a * (BK * 128), &maps.b[pi], n0 + a * 64, k0, full_bar(s));
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < g.total && ok; t += gridDim.x, lt++) {
        int pi, mt, nt, split;
        group_tile(g, t, pi, mt, nt, split);
        const GroupProblem& q = g.prob[pi];
        const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
        if (!mbar_wait(tempty_bar(ab), aph ^ 1)) { atomicExch(g.status, 4); ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + ab * BN;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(full_bar(s), ph)) { atomicExch(g.status, 2); ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = smem_base + s * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            const uint64_t ad = smem_desc(a_src + k * (UMMA_K * 128), BK * 128, 1024);
            const uint64_t bd = smem_desc(b_src + k * (UMMA_K * 128), BK * 128, 1024);
            tc_mma(tmem_d, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));
        }
        tc_commit(tfull_bar(ab));
      }
    }
  } else {
    const int ew = warp - 2;
    const int q4 = warp & 3;
    const int cbeg = (ew / 4) * CPW;
    const uint32_t stage0 = epi_base + ew * EPI_STAGE_BYTES;
    uint32_t sbuf = 0;
    bool store_pending = false;
    uint32_t lt = 0;
    for (int t = blockIdx.x; t < g.total; t += gridDim.x, lt++) {
      int pi, mt, nt, split;
      group_tile(g, t, pi, mt, nt, split);
      const GroupProblem& q = g.prob[pi];
      const int m0 = mt * BM, n0 = nt * BN;
      const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
      const bool empty_k = kend <= kbeg;
      const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
      bool ok = mbar_wait(tfull_bar(ab), aph);
      if (!ok) atomicExch(g.status, 3);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool rows_in = m0 + q4 * 32 < q.M;
      if (n0 + cbeg < q.N) {
#pragma unroll 1
        for (int cc = 0; cc < CPW; cc += 32) {
          const int c0 = cbeg + cc;
          if (n0 + c0 >= q.N) break;
          uint32_t r[32];
          if (!empty_k) {
            tc_ld32(tmem_base + ab * BN + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, r);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j++) r[j] = 0u;
          }
          sbuf ^= 1;
          if (lane == 0 && store_pending) tma_store_wait_read1();
          __syncwarp();
          const uint32_t stage = stage0 + sbuf * 4096;
          const uint32_t my_row = stage + lane * 128;
#pragma unroll
          for (int g8 = 0; g8 < 4; g8++) {
            const uint32_t s0 = my_row + (((2 * g8) ^ (lane & 7)) << 4), s1 = my_row + (((2 * g8 + 1) ^ (lane & 7)) << 4);
            st_shared_v4(s0, r[g8 * 8 + 0], r[g8 * 8 + 1], r[g8 * 8 + 2], r[g8 * 8 + 3]);
            st_shared_v4(s1, r[g8 * 8 + 4], r[g8 * 8 + 5], r[g8 * 8 + 6], r[g8 * 8 + 7]);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0 && rows_in) {
            tma_store_3d(&maps.c[pi], stage, n0 + c0, m0 + q4 * 32, split);
            tma_store_commit();
            store_pending = true;
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(ab));
    }
    if (lane == 0 && store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// =================================================================================================
// Dual-list persistent kernel: the forward of block b+1 and the backward of block b in ONE launch,
// each on its own share of the SMs (paper Section 2.2: B_b overlaps F_{b+1}; Sections 1 and 3.1:
// small GEMMs leave SMs idle and can share the device).  A launch carries up to DUAL_MAX problems
// in two ordered lists.  CTAs [0, split) work through list 0, the others through list 1; inside a
// list the tiles of all problems form one sequence that the list's CTAs take round-robin.  A problem
// may name an earlier problem of its list whose output it reads: before a CTA touches such a tile
// it waits (bounded) until a device counter says every tile of that problem has been stored.
// Every CTA walks its list in order and never waits for a later problem, all CTAs of the launch
// are resident (grid <= SMs, one CTA per SM), so the waits always resolve.
//   kind 0: GEMM tile (128 x 128), roles and pipeline as in tc_wgrad_group_kernel, operand majors
//           chosen per problem; epilogue: bias, ReLU, ReLU derivative; bf16 or fp32 output or
//           fp32 split-K partials, all through TMA stores
//   kind 1: y = gelu(u), kind 2: g = g * gelu'(u) on 32 Ki-element chunks of bf16 data, done by the
//           eight epilogue warps with the same functions as the stand-alone elementwise kernel
// The arithmetic of a tile does not depend on which CTA computes it or when: the results are the
// bits of the same operations launched one by one.
constexpr int DUAL_MAX = 8;
constexpr int DUAL_EW_CHUNK = 32768;
constexpr long long DUAL_WAIT_CYCLES = 500000000LL;
struct DualProblem {
  int kind;                       // 0 GEMM, 1 gelu, 2 gelu derivative
  int M, N, K, splits, kchunk, tiles_m, tiles_n;
  int a_mn, b_mn;
  int out_mode;                   // 0: bf16 [M, N]; 1: fp32 [M, N]; 2: fp32 split-K partials [splits, M, N]
  int relu, dact_relu;
  int dep;                        // problem whose completion this one waits for, or -1
  int signal;                     // a later problem waits for this one: count finished tiles
  int ntiles, tile_begin;         // tiles of this problem; index of its first tile in its list's sequence
  const float* bias;
  const __nv_bfloat16* dact_src;
  long long ld_aux;
  const __nv_bfloat16* ew_src;
  __nv_bfloat16* ew_dst;
  long long ew_n;
};
struct DualArgs {
  int nprob, split;
  int first[2], count[2], total[2];   // per list: first problem, number of problems, tiles
  int* done;                          // [DUAL_MAX] finished epilogue-warp tiles per problem, zero at launch
  int* status;
  DualProblem prob[DUAL_MAX];
};
struct DualMaps {
  CUtensorMap a[DUAL_MAX], b[DUAL_MAX], c[DUAL_MAX];
};

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// waits until problem `dep` has stored all its tiles (8 epilogue warps each); false on expiry
__device__ __forceinline__ bool dual_wait_dep(const DualArgs& g, int dep) {
  if (dep < 0) return true;
  const int need = g.prob[dep].ntiles * EPI_WARPS;
  if (ld_acquire(g.done + dep) >= need) return true;
  const long long t0 = clock64();
  while (ld_acquire(g.done + dep) < need) {
    if (clock64() - t0 > DUAL_WAIT_CYCLES) return false;
    __nanosleep(64);
  }
  return true;
}
__device__ __forceinline__ int dual_find(const DualArgs& g, int list, int t) {
  int pi = g.first[list];
  const int end = g.first[list] + g.count[list];
  while (pi + 1 < end && t >= g.prob[pi + 1].tile_begin) pi++;
  return pi;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
tc_dual_kernel(const __grid_constant__ DualMaps maps, const __grid_constant__ DualArgs g) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int BN = 128;
  constexpr uint32_t A_BYTES = BM * BK * 2;
  constexpr uint32_t B_BYTES = BN * BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;
  constexpr int STAGES = 4;
  constexpr int CPW = BN / 2;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;
  const uint32_t bias_base = epi_base + EPI_WARPS * EPI_STAGE_BYTES;
  const uint32_t bar_base = bias_base + EPI_WARPS * EPI_BIAS_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(gen_base + (bar_base - smem_base) + 8u * (2 * STAGES + 4));
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int list = (int)blockIdx.x < g.split ? 0 : 1;
  const int rank = list == 0 ? (int)blockIdx.x : (int)blockIdx.x - g.split;
  const int nrank = list == 0 ? g.split : (int)gridDim.x - g.split;
  const int total = g.total[list];
  const int st0 = status_peek(g.status);
  if (threadIdx.x == 32) {
    for (int i = 0; i < g.nprob; i++) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.a[i]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.b[i]) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.c[i]) : "memory");
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  const bool dead = __syncthreads_or(st0 != 0) != 0;
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  if (dead) {
    // the step is already void: do nothing but free TMEM below
  } else if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = rank; t < total && ok; t += nrank) {
        const int pi = dual_find(g, list, t);
        const DualProblem& q = g.prob[pi];
        if (q.kind != 0) continue;                      // elementwise chunks need no staging
        if (!dual_wait_dep(g, q.dep)) { atomicExch(g.status, 41); ok = false; break; }
        asm volatile("fence.proxy.async;" ::: "memory");   // the other CTAs' stores are ordered before this CTA's TMA reads
        const int local = t - q.tile_begin, per = q.tiles_m * q.tiles_n;
        const int split = local / per, r = local - split * per;
        const int mt = r / q.tiles_n, nt = r - mt * q.tiles_n;
        const int m0 = mt * BM, n0 = nt * BN;
        const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(empty_bar(s), ph ^ 1)) { atomicExch(g.status, 1); ok = false; break; }
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          const uint32_t a_dst = smem_base + s * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
          const int k0 = kbeg + kb * BK;
          if (!q.a_mn) {
            tma_load_2d(a_dst, &maps.a[pi], k0, m0, full_bar(s));
          } else {
#pragma unroll
            for (int a = 0; a < BM / 64; a++) tma_load_2d(a_dst + a * (BK * 128), &maps.a[pi], m0 + a * 64, k0, full_bar(s));
          }
          if (!q.b_mn) {
            tma_load_2d(b_dst, &maps.b[pi], k0, n0, full_bar(s));
          } else {
#pragma unroll
            for (int a = 0; a < BN / 64; a++) tma_load_2d(b_dst + a * (BK * 128), &maps.b[pi], n0 + a * 64, k0, full_bar(s));
          }
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int t = rank; t < total && ok; t += nrank) {
        const int pi = dual_find(g, list, t);
        const DualProblem& q = g.prob[pi];
        if (q.kind != 0) continue;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((q.a_mn ? 1u : 0u) << 15) | ((q.b_mn ? 1u : 0u) << 16) |
                               ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        const int local = t - q.tile_begin, split = local / (q.tiles_m * q.tiles_n);
        const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
        const int num_kb = kend > kbeg ? (kend - kbeg + BK - 1) / BK : 0;
        const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
        if (!mbar_wait(tempty_bar(ab), aph ^ 1)) { atomicExch(g.status, 4); ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + ab * BN;
        for (int kb = 0; kb < num_kb; kb++, it++) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(full_bar(s), ph)) { atomicExch(g.status, 2); ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = smem_base + s * STAGE_BYTES;
          const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            const uint64_t ad = q.a_mn ? smem_desc(a_src + k * (UMMA_K * 128), BK * 128, 1024) : smem_desc(a_src + k * (UMMA_K * 2), 16, 1024);
            const uint64_t bd = q.b_mn ? smem_desc(b_src + k * (UMMA_K * 128), BK * 128, 1024) : smem_desc(b_src + k * (UMMA_K * 2), 16, 1024);
            tc_mma(tmem_d, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));
        }
        tc_commit(tfull_bar(ab));
        lt++;
      }
    }
  } else {
    // ------------------------------ epilogue / elementwise warps ------------------------------
    const int ew = warp - 2;
    const int q4 = warp & 3;
    const int cbeg = (ew / 4) * CPW;
    const uint32_t stage0 = epi_base + ew * EPI_STAGE_BYTES;
    float* bias_s = reinterpret_cast<float*>(gen_base + (bias_base - smem_base) + ew * EPI_BIAS_BYTES);
    uint32_t sbuf = 0;
    bool store_pending = false;
    uint32_t lt = 0;
    for (int t = rank; t < total; t += nrank) {
      const int pi = dual_find(g, list, t);
      const DualProblem& q = g.prob[pi];
      if (q.kind != 0) {
        // ---- elementwise chunk: the 256 threads of these warps, 16 bytes per access ----
        bool ok = true;
        if (lane == 0) ok = dual_wait_dep(g, q.dep);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) { if (lane == 0) atomicExch(g.status, 42); break; }
        asm volatile("fence.proxy.async;" ::: "memory");
        const long long beg = (long long)(t - q.tile_begin) * DUAL_EW_CHUNK;
        const long long end = beg + DUAL_EW_CHUNK < q.ew_n ? beg + DUAL_EW_CHUNK : q.ew_n;
        for (long long i = beg + (long long)(ew * 32 + lane) * 8; i < end; i += 256 * 8) {     // ew_n % 8 == 0
          const uint4 u = *reinterpret_cast<const uint4*>(q.ew_src + i);
          float x[8], y[8];
          unpack8_bf16(u, x);
          if (q.kind == 1) {
#pragma unroll
            for (int j = 0; j < 8; j++) y[j] = gelu_bf16_value(x[j]);
          } else {
            unpack8_bf16(*reinterpret_cast<const uint4*>(q.ew_dst + i), y);
#pragma unroll
            for (int j = 0; j < 8; j++) y[j] = y[j] * gelu_bf16_deriv(x[j]);
          }
          uint4 o;
          o.x = pack2(y[0], y[1]); o.y = pack2(y[2], y[3]); o.z = pack2(y[4], y[5]); o.w = pack2(y[6], y[7]);
          *reinterpret_cast<uint4*>(q.ew_dst + i) = o;
        }
        if (q.signal) {
          __threadfence();
          __syncwarp();
          if (lane == 0) atomicAdd(g.done + pi, 1);
        }
        continue;
      }
      const int local = t - q.tile_begin, per = q.tiles_m * q.tiles_n;
      const int split = local / per, r = local - split * per;
      const int mt = r / q.tiles_n, nt = r - mt * q.tiles_n;
      const int m0 = mt * BM, n0 = nt * BN;
      const int kbeg = split * q.kchunk, kend = min(q.K, kbeg + q.kchunk);
      const bool empty_k = kend <= kbeg;
      const uint32_t ab = lt & 1, aph = (lt >> 1) & 1;
      lt++;
      if (q.bias) {
        __syncwarp();
        for (int j = lane; j < CPW; j += 32) {
          const int n = n0 + cbeg + j;
          bias_s[j] = n < q.N ? __ldg(q.bias + n) : 0.f;
        }
        __syncwarp();
      }
      const int row = m0 + q4 * 32 + lane;
      const bool row_ok = row < q.M;
      bool ok = mbar_wait(tfull_bar(ab), aph);
      if (!ok) atomicExch(g.status, 3);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool rows_in = m0 + q4 * 32 < q.M;
      const bool f32 = q.out_mode != 0;
      if (n0 + cbeg < q.N) {
#pragma unroll 1
        for (int cc = 0; cc < CPW; cc += 32) {
          const int c0 = cbeg + cc;
          if (n0 + c0 >= q.N) break;
          uint32_t rr[32];
          if (!empty_k) {
            tc_ld32(tmem_base + ab * BN + ((uint32_t)(q4 * 32) << 16) + (uint32_t)c0, rr);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j++) rr[j] = 0u;
          }
          if (f32 || (cc & 63) == 0) {
            sbuf ^= 1;
            if (lane == 0 && store_pending) tma_store_wait_read1();
            __syncwarp();
          }
          const uint32_t stage = stage0 + sbuf * 4096;
          const uint32_t my_row = stage + lane * 128;
#pragma unroll
          for (int g8 = 0; g8 < 4; g8++) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; j++) v[j] = __uint_as_float(rr[g8 * 8 + j]);
            const int n = n0 + c0 + g8 * 8;
            if (q.bias) {
              const float4 b0 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8);
              const float4 b1 = *reinterpret_cast<const float4*>(bias_s + cc + g8 * 8 + 4);
              v[0] += b0.x; v[1] += b0.y; v[2] += b0.z; v[3] += b0.w;
              v[4] += b1.x; v[5] += b1.y; v[6] += b1.z; v[7] += b1.w;
            }
            if (q.relu) {
#pragma unroll
              for (int j = 0; j < 8; j++) v[j] = fmaxf(v[j], 0.f);
            }
            if (q.dact_relu && row_ok && n < q.N) {       // N % 8 == 0 whenever an auxiliary operand is present
              float tsrc[8];
              unpack8_bf16(*reinterpret_cast<const uint4*>(q.dact_src + (long long)row * q.ld_aux + n), tsrc);
#pragma unroll
              for (int j = 0; j < 8; j++) v[j] = tsrc[j] > 0.f ? v[j] : 0.f;
            }
            if (f32) {
              const uint32_t s0 = my_row + (((2 * g8) ^ (lane & 7)) << 4), s1 = my_row + (((2 * g8 + 1) ^ (lane & 7)) << 4);
              st_shared_v4(s0, __float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
              st_shared_v4(s1, __float_as_uint(v[4]), __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
            } else {
              const uint32_t s0 = my_row + (((((cc & 63) >> 3) + g8) ^ (lane & 7)) << 4);
              st_shared_v4(s0, pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
            }
          }
          const bool last_chunk = (cc & 63) == 32 || n0 + c0 + 32 >= q.N;
          if (f32 || last_chunk) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0 && rows_in) {
              const int x = f32 ? n0 + c0 : n0 + cbeg + (cc & ~63), y = m0 + q4 * 32;
              if (q.out_mode == 2) tma_store_3d(&maps.c[pi], stage, x, y, split);
              else tma_store_2d(&maps.c[pi], stage, x, y);
              tma_store_commit();
              store_pending = true;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(ab));
      if (q.signal) {     // a later problem reads this output: report the tile once its stores have landed
        if (lane == 0) {
          if (store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
          store_pending = false;
          asm volatile("fence.proxy.async;" ::: "memory");
          __threadfence();
          atomicAdd(g.done + pi, 1);
        }
        __syncwarp();
      }
    }
    if (lane == 0 && store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// The bounded wait on its own: one thread waits, with the given limit, on a barrier that nothing
// ever signals, records status code 8 and returns.  It returns by construction (the wait is
// clock-bounded) and touches no tensor memory; used to check that an expired wait surfaces as
// ERASE_ETIMEOUT and leaves the context usable.
__global__ void wait_selftest_kernel(int* status, long long limit_cycles) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait(smem_u32(&bar), 0, limit_cycles)) atomicExch(status, 8);
  }
}

// Host-side caches are per device: a process may drive several GPUs.
constexpr int MAX_DEVICES = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) dev = 0;
  return dev;
}
int sm_count() {
  static std::atomic<int> cache[MAX_DEVICES];
  const int dev = current_device();
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 2) n = 148;
    cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel, device); `done` is the kernel's own table
template <typename K>
cudaError_t ensure_smem(K kernel, size_t smem, std::atomic<bool>* done) {
  const int dev = current_device();
  if (done[dev].load(std::memory_order_acquire)) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess) done[dev].store(true, std::memory_order_release);
  return e;
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static const EncodeFn fn = []() -> EncodeFn {   // initialised once, thread-safe (the entry point is process-wide)
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return (EncodeFn)p;
    cudaGetLastError();
    return nullptr;
  }();
  return fn;
}

// Tensor map of a row-major bf16 or fp32 matrix (rank 2) or stack of matrices (rank 3):
// dims[0] contiguous elements per row, rows stride_bytes[0] apart, 128-byte swizzle; the box's
// inner extent is 128 bytes.  Out-of-bounds elements read as zero and are not written.
bool encode_map(void* out, const void* base, bool f32, int rank, const cuuint64_t* dims, const cuuint64_t* stride_bytes,
                const cuuint32_t* box) {
  EncodeFn fn = encode_fn();
  if (!fn) return false;
  for (int i = 0; i + 1 < rank; i++)
    if (stride_bytes[i] % 16) return false;
  if (reinterpret_cast<uintptr_t>(base) & 15) return false;
  CUtensorMap tmp;
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = fn(&tmp, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                  const_cast<void*>(base), dims, stride_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r == CUDA_SUCCESS) memcpy(out, &tmp, sizeof(tmp));
  return r == CUDA_SUCCESS;
}

// operand map: `inner` contiguous bf16 elements per row, `outer` rows `ld` elements apart; box 64 x box_outer
bool encode_2d(void* out, const void* base, long long inner, long long outer, long long ld, int box_outer) {
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
  return encode_map(out, base, false, 2, dims, strides, box);
}

template <int BN, bool A_MN, bool B_MN, bool GENERAL, bool CE = false>
cudaError_t launch_t(const GemmArgs& g, const TcPlan& plan, cudaStream_t s, int max_ctas) {
  constexpr int STAGES = stages_for(BN);
  constexpr size_t smem = (size_t)STAGES * (BM * BK * 2 + BN * BK * 2) + EPI_WARPS * (SINGLE_EPI_BYTES + EPI_BIAS_BYTES) + 8 * (2 * STAGES + 16) + 1024;
  static std::atomic<bool> attr_set[MAX_DEVICES];
  if (cudaError_t e = ensure_smem(tc_gemm_kernel<BN, A_MN, B_MN, GENERAL, CE>, smem, attr_set)) return e;
  TcArgs p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.C = g.C; p.ldc = g.ldc; p.c_f32 = g.c_f32;
  p.splits = g.splits; p.ws = g.ws; p.epi = g.epi; p.status = plan.status; p.dbg = plan.dbg; p.sched = plan.sched;
  p.xcol_out = nullptr;
  const int num_sms = sm_count();
  const long long total = (long long)((g.N + BN - 1) / BN) * ((g.M + BM - 1) / BM) * g.splits;
  long long cap = (max_ctas > 0 && max_ctas < num_sms) ? max_ctas : num_sms;
  dim3 grid((unsigned)(total < cap ? total : cap));
  CUtensorMap ma, mb, mc;
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  memcpy(&ma, plan.map_a, sizeof(ma));
  memcpy(&mb, plan.map_b, sizeof(mb));
  memcpy(&mc, plan.map_c, sizeof(mc));
  p.tma_c = plan.tma_c;
  const Epilogue& e = g.epi;
  const bool no_aux = e.alpha == 1.f && e.act == ACT_NONE && !e.pre_out && !e.mul && !e.res && e.dact == ACT_NONE;
  p.plain = no_aux ? (e.bias ? (g.splits == 1 ? 2 : 1) : 1) : 0;   // 1: identity, 2: bias only, 0: general
  if (total <= (long long)grid.x) p.sched = nullptr;   // one tile per CTA: nothing to balance
  tc_gemm_kernel<BN, A_MN, B_MN, GENERAL, CE><<<grid, TC_THREADS, smem, s>>>(ma, mb, mc, p);
  return cudaGetLastError();
}

template <bool A_MN, bool B_MN, bool GENERAL, bool CE = false>
cudaError_t launch_pair_t(const GemmArgs& g, const TcPlan& plan, cudaStream_t s, int max_ctas) {
  constexpr size_t smem = (size_t)PAIR_STAGES * PAIR_STAGE_BYTES + EPI_WARPS * PAIR_EPI_BYTES + PAIR_BIAS_BYTES + 8 * (2 * PAIR_STAGES + 16);
  static_assert(smem <= 232448, "pair kernel: shared memory over the per-CTA limit");
  static std::atomic<bool> attr_set[MAX_DEVICES];
  if (cudaError_t e = ensure_smem(tc_gemm_pair_kernel<A_MN, B_MN, GENERAL, CE>, smem, attr_set)) return e;
  TcArgs p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.C = g.C; p.ldc = g.ldc; p.c_f32 = g.c_f32;
  p.splits = g.splits; p.ws = g.ws; p.epi = g.epi; p.status = plan.status; p.dbg = plan.dbg; p.sched = nullptr;
  p.xcol_out = plan.xcol ? g.xcol_out : nullptr;
  p.tma_c = 1;
  const Epilogue& e = g.epi;
  const bool no_aux = e.alpha == 1.f && e.act == ACT_NONE && !e.pre_out && !e.mul && !e.res && e.dact == ACT_NONE;
  p.plain = no_aux ? (e.bias ? (g.splits == 1 ? 2 : 1) : 1) : 0;   // 1: identity, 2: bias only, 0: general
  const int num_sms = sm_count();
  const long long total = (long long)((g.N + PAIR_BN - 1) / PAIR_BN + (plan.xcol ? 1 : 0)) * ((g.M + 2 * BM - 1) / (2 * BM)) * g.splits;
  long long cap = ((max_ctas > 1 && max_ctas < num_sms) ? max_ctas : num_sms) / 2;
  dim3 grid(2u * (unsigned)(total < cap ? total : cap));
  CUtensorMap ma, mb, mc;
  memcpy(&ma, plan.map_a, sizeof(ma));
  memcpy(&mb, plan.b_mn ? plan.map_b : plan.map_b_half, sizeof(mb));
  memcpy(&mc, plan.map_c, sizeof(mc));
  tc_gemm_pair_kernel<A_MN, B_MN, GENERAL, CE><<<grid, TC_THREADS, smem, s>>>(ma, mb, mc, p, (uint32_t)plan.pair_tmem_cols);
  return cudaGetLastError();
}

static bool epilogue_is_simple(const GemmArgs& g) {
  const Epilogue& e = g.epi;
  return g.splits > 1 || (e.alpha == 1.f && e.act == ACT_NONE && !e.pre_out && !e.mul && !e.res && e.dact == ACT_NONE);
}

template <int BN, bool GENERAL>
cudaError_t launch_bn(const GemmArgs& g, const TcPlan& plan, cudaStream_t s, int max_ctas) {
  if (!plan.a_mn && !plan.b_mn) return launch_t<BN, false, false, GENERAL>(g, plan, s, max_ctas);
  if (!plan.a_mn && plan.b_mn) return launch_t<BN, false, true, GENERAL>(g, plan, s, max_ctas);
  if (plan.a_mn && !plan.b_mn) return launch_t<BN, true, false, GENERAL>(g, plan, s, max_ctas);
  return launch_t<BN, true, true, GENERAL>(g, plan, s, max_ctas);
}

}  // namespace

// ---- dual-list persistent kernel: host side ---------------------------------------------------
struct TcDualPlan {
  DualArgs args;
  DualMaps maps;
  int grid;
};

int tc_dual_max() { return DUAL_MAX; }

TcDualPlan* tc_dual_plan(const DualItem* items_in, int n, int* done_dev, int* status) {
  if (n < 1 || n > DUAL_MAX || !done_dev) return nullptr;
  // list 0 first, then list 1, each in the given order
  DualItem items[DUAL_MAX];
  int cnt = 0, first1 = 0;
  for (int l = 0; l < 2; l++) {
    if (l == 1) first1 = cnt;
    for (int i = 0; i < n; i++)
      if (items_in[i].list == l) items[cnt++] = items_in[i];
  }
  if (cnt != n) return nullptr;
  for (int i = 0; i < n; i++)
    if (items[i].kind == 0 && items[i].g.xcol_out) return nullptr;   // the extra-column product exists in the pair kernel only
  TcDualPlan* plan = new TcDualPlan();
  DualArgs& a = plan->args;
  memset(&a, 0, sizeof(a));
  a.nprob = n;
  a.done = done_dev;
  a.status = status;
  a.first[0] = 0; a.count[0] = first1;
  a.first[1] = first1; a.count[1] = n - first1;
  double work[2] = {0, 0};
  auto fail = [&]() { delete plan; return (TcDualPlan*)nullptr; };
  for (int l = 0; l < 2; l++) {
    int tiles = 0, last_chain = -1;
    for (int i = a.first[l]; i < a.first[l] + a.count[l]; i++) {
      const DualItem& it = items[i];
      DualProblem& q = a.prob[i];
      q.kind = it.kind;
      q.dep = last_chain;
      q.tile_begin = tiles;
      if (it.kind == 0) {
        const GemmArgs& g = it.g;
        const Epilogue& e = g.epi;
        if (!tc_gemm_supported(g) || e.alpha != 1.f || e.mul || e.res || e.pre_out || e.ce_ref || (e.act != ACT_NONE && e.act != ACT_RELU) ||
            (e.dact != ACT_NONE && e.dact != ACT_RELU) || (g.splits > 1 && (!g.ws || e.bias || e.act != ACT_NONE || e.dact != ACT_NONE)))
          return fail();
        q.M = g.M; q.N = g.N; q.K = g.K; q.splits = g.splits;
        q.kchunk = (((g.K + g.splits - 1) / g.splits) + BK - 1) / BK * BK;
        q.tiles_m = (g.M + BM - 1) / BM;
        q.tiles_n = (g.N + 127) / 128;
        q.a_mn = g.sa_k != 1; q.b_mn = g.sb_k != 1;
        q.relu = e.act == ACT_RELU; q.dact_relu = e.dact == ACT_RELU;
        q.bias = e.bias;
        q.dact_src = (const __nv_bfloat16*)e.dact_src;
        q.ld_aux = e.ld_aux ? e.ld_aux : g.N;
        q.ntiles = q.tiles_m * q.tiles_n * g.splits;
        bool ok = q.a_mn ? encode_2d(&plan->maps.a[i], g.A, g.M, g.K, g.sa_k, BK) : encode_2d(&plan->maps.a[i], g.A, g.K, g.M, g.sa_m, BM);
        ok = ok && (q.b_mn ? encode_2d(&plan->maps.b[i], g.B, g.N, g.K, g.sb_k, BK) : encode_2d(&plan->maps.b[i], g.B, g.K, g.N, g.sb_n, 128));
        if (!ok) return fail();
        if (g.splits > 1) {
          q.out_mode = 2;
          cuuint64_t dims[3] = {(cuuint64_t)g.N, (cuuint64_t)g.M, (cuuint64_t)g.splits};
          cuuint64_t str[2] = {(cuuint64_t)g.N * 4, (cuuint64_t)g.M * g.N * 4};
          cuuint32_t box[3] = {32u, 32u, 1u};
          ok = encode_map(&plan->maps.c[i], g.ws, true, 3, dims, str, box);
        } else if (g.c_f32) {
          q.out_mode = 1;
          cuuint64_t dims[2] = {(cuuint64_t)g.N, (cuuint64_t)g.M};
          cuuint64_t str[1] = {(cuuint64_t)g.ldc * 4};
          cuuint32_t box[2] = {32u, 32u};
          ok = encode_map(&plan->maps.c[i], g.C, true, 2, dims, str, box);
        } else {
          q.out_mode = 0;
          cuuint64_t dims[2] = {(cuuint64_t)g.N, (cuuint64_t)g.M};
          cuuint64_t str[1] = {(cuuint64_t)g.ldc * 2};
          cuuint32_t box[2] = {64u, 32u};
          ok = encode_map(&plan->maps.c[i], g.C, false, 2, dims, str, box);
        }
        if (!ok) return fail();
        work[l] += (double)q.ntiles * ((q.kchunk + BK - 1) / BK + 6);
      } else {
        if (it.ew_n < 8 || it.ew_n % 8 || ((reinterpret_cast<uintptr_t>(it.ew_src) | reinterpret_cast<uintptr_t>(it.ew_dst)) & 15)) return fail();
        q.ew_src = (const __nv_bfloat16*)it.ew_src;
        q.ew_dst = (__nv_bfloat16*)it.ew_dst;
        q.ew_n = it.ew_n;
        q.ntiles = (int)((it.ew_n + DUAL_EW_CHUNK - 1) / DUAL_EW_CHUNK);
        plan->maps.a[i] = plan->maps.a[0]; plan->maps.b[i] = plan->maps.b[0]; plan->maps.c[i] = plan->maps.c[0];
        work[l] += (double)q.ntiles * 8;
      }
      tiles += q.ntiles;
      if (!it.leaf) last_chain = i;
    }
    a.total[l] = tiles;
  }
  for (int i = 0; i < n; i++)
    for (int j = i + 1; j < n; j++)
      if (a.prob[j].dep == i) a.prob[i].signal = 1;
  for (int i = n; i < DUAL_MAX; i++) { plan->maps.a[i] = plan->maps.a[0]; plan->maps.b[i] = plan->maps.b[0]; plan->maps.c[i] = plan->maps.c[0]; }
  const int sms = sm_count();
  plan->grid = sms;
  if (a.total[0] == 0) a.split = 0;
  else if (a.total[1] == 0) a.split = sms;
  else {
    int sp = (int)(sms * work[0] / (work[0] + work[1]) + 0.5);
    a.split = sp < 1 ? 1 : (sp > sms - 1 ? sms - 1 : sp);
  }
  return plan;
}

void tc_dual_free(TcDualPlan* plan) { delete plan; }

cudaError_t tc_dual_launch(const TcDualPlan* plan, cudaStream_t s) {
  constexpr size_t smem = (size_t)4 * (BM * BK * 2 + 128 * BK * 2) + EPI_WARPS * (EPI_STAGE_BYTES + EPI_BIAS_BYTES) + 8 * (2 * 4 + 16) + 1024;
  static std::atomic<bool> attr_set[MAX_DEVICES];
  if (cudaError_t e = ensure_smem(tc_dual_kernel, smem, attr_set)) return e;
  cudaError_t e = cudaMemsetAsync(plan->args.done, 0, DUAL_MAX * sizeof(int), s);
  if (e != cudaSuccess) return e;
  tc_dual_kernel<<<plan->grid, TC_THREADS, smem, s>>>(plan->maps, plan->args);
  return cudaGetLastError();
}

bool tc_encode_rows_bf16(void* map128, const void* base, long long inner, long long outer, long long ld, int box_rows) {
  return encode_2d(map128, base, inner, outer, ld, box_rows);
}

cudaError_t tc_wait_selftest(int* status, long long limit_cycles, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(status, limit_cycles);
  return cudaGetLastError();
}

bool tc_wgrad_group_plan(const GemmArgs* gs, int n, int* status, TcGroupPlan* plan) {
  if (n < 1 || n > GROUP_MAX) return false;
  plan->n = n;
  plan->status = status;
  int total = 0;
  for (int i = 0; i < n; i++) {
    const GemmArgs& g = gs[i];
    if (!tc_gemm_supported(g) || g.sa_k == 1 || g.sb_k == 1 || g.splits < 1 || !g.ws) return false;   // both operands MN-major
    plan->M[i] = g.M; plan->N[i] = g.N; plan->K[i] = g.K; plan->splits[i] = g.splits;
    plan->kchunk[i] = (((g.K + g.splits - 1) / g.splits) + BK - 1) / BK * BK;
    plan->tiles_m[i] = (g.M + BM - 1) / BM;
    plan->tiles_n[i] = (g.N + 127) / 128;
    plan->tile_begin[i] = total;
    total += plan->tiles_m[i] * plan->tiles_n[i] * g.splits;
    if (!encode_2d(plan->map_a[i], g.A, g.M, g.K, g.sa_k, BK)) return false;
    if (!encode_2d(plan->map_b[i], g.B, g.N, g.K, g.sb_k, BK)) return false;
    cuuint64_t dims[3] = {(cuuint64_t)g.N, (cuuint64_t)g.M, (cuuint64_t)g.splits};
    cuuint64_t str[2] = {(cuuint64_t)g.N * 4, (cuuint64_t)g.M * g.N * 4};
    cuuint32_t box[3] = {32u, 32u, 1u};
    if (!encode_map(plan->map_c[i], g.ws, true, 3, dims, str, box)) return false;
  }
  plan->total = total;
  return true;
}

cudaError_t tc_wgrad_group_launch(const TcGroupPlan& plan, cudaStream_t s, int max_ctas) {
  constexpr size_t smem = (size_t)4 * (BM * BK * 2 + 128 * BK * 2) + EPI_WARPS * EPI_STAGE_BYTES + 8 * (2 * 4 + 16) + 1024;
  static std::atomic<bool> attr_set[MAX_DEVICES];
  if (cudaError_t e = ensure_smem(tc_wgrad_group_kernel, smem, attr_set)) return e;
  GroupMaps maps;
  GroupArgs g;
  memset(&g, 0, sizeof(g));
  g.nprob = plan.n; g.total = plan.total; g.status = plan.status;
  for (int i = 0; i < plan.n; i++) {
    memcpy(&maps.a[i], plan.map_a[i], 128);
    memcpy(&maps.b[i], plan.map_b[i], 128);
    memcpy(&maps.c[i], plan.map_c[i], 128);
    g.prob[i] = GroupProblem{plan.M[i], plan.N[i], plan.K[i], plan.splits[i], plan.kchunk[i], plan.tiles_m[i], plan.tiles_n[i], plan.tile_begin[i]};
  }
  for (int i = plan.n; i < GROUP_MAX; i++) { maps.a[i] = maps.a[0]; maps.b[i] = maps.b[0]; maps.c[i] = maps.c[0]; }
  const int num_sms = sm_count();
  int cap = (max_ctas > 0 && max_ctas < num_sms) ? max_ctas : num_sms;
  dim3 grid((unsigned)(plan.total < cap ? plan.total : cap));
  tc_wgrad_group_kernel<<<grid, TC_THREADS, smem, s>>>(maps, g);
  return cudaGetLastError();
}

bool tc_gemm_supported(const GemmArgs& g) {
  if (g.K < 64 || g.N < 16 || g.M < 1) return false;
  auto operand_ok = [](const void* p, long long s_mn, long long s_k) {
    if (reinterpret_cast<uintptr_t>(p) & 15) return false;
    if (s_k == 1) return s_mn % 8 == 0 && s_mn > 0;
    if (s_mn == 1) return s_k % 8 == 0 && s_k > 0;
    return false;
  };
  if (!operand_ok(g.A, g.sa_m, g.sa_k) || !operand_ok(g.B, g.sb_n, g.sb_k)) return false;
  // a [1 x K] operand is ambiguous (both strides may be 1): leave such GEMVs to the SIMT kernel
  if ((g.sa_m == 1 && g.sa_k == 1) || (g.sb_n == 1 && g.sb_k == 1)) return false;
  // the fused epilogue reads its auxiliary operands as aligned 16-byte pieces of 8 columns, and keeps
  // one register set for "multiplier or activation-derivative source"
  const Epilogue& e = g.epi;
  if (g.splits == 1 && (e.pre_out || e.act == ACT_GELU || e.dact == ACT_GELU)) return false;   // SIMT kernel
  if (g.splits == 1 && (e.mul || e.res || e.dact != ACT_NONE)) {
    if (e.mul && e.dact != ACT_NONE) return false;
    const long long ld = e.ld_aux ? e.ld_aux : g.N;
    if (ld % 8 != 0 || g.N % 8 != 0) return false;
    const void* aux[3] = {e.mul, e.res, e.dact != ACT_NONE ? e.dact_src : nullptr};
    for (const void* a : aux)
      if (a && (reinterpret_cast<uintptr_t>(a) & 15)) return false;
  }
  return true;
}

bool tc_gemm_plan(const GemmArgs& g, int* status, TcPlan* plan) {
  if (!tc_gemm_supported(g)) return false;
  plan->a_mn = g.sa_k != 1;
  plan->b_mn = g.sb_k != 1;
  // tile width: 256 halves the A-operand traffic per FLOP, taken when it still leaves every SM a tile
  const long long tiles256 = (long long)((g.M + BM - 1) / BM) * ((g.N + 255) / 256) * g.splits;
  plan->bn = g.N <= 64 ? 64 : (g.N >= 256 && tiles256 >= 148 ? 256 : 128);
  // CTA-pair kernel (256 x 256 tiles over two SMs) when its tiles keep most of the 74 pairs busy
  static const int env_pair = getenv("ERASE_TC_PAIR") ? atoi(getenv("ERASE_TC_PAIR")) : 1;
  // (a request for the extra-column product brings one narrow tile per row tile: they count)
  const bool xcol_shape = g.xcol_out != nullptr && g.sa_k != 1 && g.sb_k != 1 && g.splits == 1 && g.N % PAIR_BN == 0;
  const long long pair_tiles = (long long)((g.M + 2 * BM - 1) / (2 * BM)) * ((g.N + PAIR_BN - 1) / PAIR_BN + (xcol_shape ? 1 : 0)) * g.splits;
  // (GEMMs with a little more than one wave of pair tiles, e.g. C4's 96-tile N = 768 ones, were also tried as
  // 128 x 256 single-CTA tiles, which fill two waves of 148 evenly: 3-14 % slower, so the pair kernel keeps them.)
  const bool want_pair = env_pair && (epilogue_is_simple(g) || !plan->a_mn) && g.M >= 256 && g.N > 128 && pair_tiles >= 56;
  if (want_pair) plan->bn = 256;
  if (getenv("ERASE_TC_BN")) { int f = atoi(getenv("ERASE_TC_BN")); if ((f == 64 || f == 128 || f == 256) && f <= (g.N + 63) / 64 * 64) plan->bn = f; }
  plan->status = status;
  plan->launches = 1;
  bool ok;
  if (!plan->a_mn) ok = encode_2d(plan->map_a, g.A, g.K, g.M, g.sa_m, BM);
  else ok = encode_2d(plan->map_a, g.A, g.M, g.K, g.sa_k, BK);
  if (!ok) return false;
  // extra-column product: weight-gradient layout on the pair kernel, no split, N a multiple of the tile width
  const bool want_xcol = g.xcol_out != nullptr && want_pair && plan->a_mn && plan->b_mn && g.splits == 1 && g.N % PAIR_BN == 0 &&
                         plan->bn == 256;
  if (!plan->b_mn) ok = encode_2d(plan->map_b, g.B, g.K, g.N, g.sb_n, plan->bn);
  else ok = encode_2d(plan->map_b, g.B, g.N + (want_xcol ? 16 : 0), g.K, g.sb_k, BK);
  if (!ok) return false;
  // outputs through TMA stores where their layout allows it (else the kernel stores directly)
  memset(plan->map_c, 0, sizeof(plan->map_c));
  plan->tma_c = 0;
  if (g.splits > 1) {
    cuuint64_t dims[3] = {(cuuint64_t)g.N, (cuuint64_t)g.M, (cuuint64_t)g.splits};
    cuuint64_t str[2] = {(cuuint64_t)g.N * 4, (cuuint64_t)g.M * g.N * 4};
    cuuint32_t box[3] = {32u, 32u, 1u};
    plan->tma_c = g.ws && encode_map(plan->map_c, g.ws, true, 3, dims, str, box) ? 1 : 0;
  } else if (g.c_f32) {
    cuuint64_t dims[2] = {(cuuint64_t)g.N, (cuuint64_t)g.M};
    cuuint64_t str[1] = {(cuuint64_t)g.ldc * 4};
    cuuint32_t box[2] = {32u, 32u};
    plan->tma_c = encode_map(plan->map_c, g.C, true, 2, dims, str, box) ? 1 : 0;
  } else {
    cuuint64_t dims[2] = {(cuuint64_t)g.N, (cuuint64_t)g.M};
    cuuint64_t str[1] = {(cuuint64_t)g.ldc * 2};
    cuuint32_t box[2] = {64u, 32u};
    plan->tma_c = encode_map(plan->map_c, g.C, false, 2, dims, str, box) ? 1 : 0;
  }
  // CTA-pair kernel (256 x 256 tiles over two SMs): identity / bias-only epilogue, TMA-stored output
  plan->pair = 0;
  {
    static const int env_cols = getenv("ERASE_TC_PAIR_COLS") ? atoi(getenv("ERASE_TC_PAIR_COLS")) : 512;
    plan->pair_tmem_cols = env_cols == 256 ? 256 : 512;
    if (want_pair && plan->tma_c && plan->bn == 256) {
      bool okp = true;
      if (!plan->b_mn) okp = encode_2d(plan->map_b_half, g.B, g.K, g.N, g.sb_n, PAIR_BN / 2);
      plan->pair = okp ? 1 : 0;
    }
  }
  plan->xcol = (want_xcol && plan->pair) ? 1 : 0;
  if (want_xcol && !plan->xcol)     // the map was encoded 16 columns too wide for a kernel that will not read them: encode it again
    if (!encode_2d(plan->map_b, g.B, g.N, g.K, g.sb_k, BK)) return false;
  return true;
}

int tc_ce_group_cols(const TcPlan& plan) { return (plan.pair || plan.bn >= 128) ? plan.bn / 2 : 64; }

cudaError_t tc_gemm_launch(const GemmArgs& g, const TcPlan& plan, cudaStream_t s, int max_ctas) {
  if (g.epi.ce_ref) {   // cross-entropy head forward: both operands K-major, bias, bf16 output through TMA
    if (plan.a_mn || plan.b_mn || !plan.tma_c || g.splits != 1 || !g.epi.bias || !g.epi.ce_psum) return cudaErrorInvalidValue;
    if (plan.pair) return launch_pair_t<false, false, false, true>(g, plan, s, max_ctas);
    switch (plan.bn) {
      case 64: return launch_t<64, false, false, false, true>(g, plan, s, max_ctas);
      case 256: return launch_t<256, false, false, false, true>(g, plan, s, max_ctas);
      default: return launch_t<128, false, false, false, true>(g, plan, s, max_ctas);
    }
  }
  const bool simple = epilogue_is_simple(g);
  if (plan.pair) {
    if (simple) {
      if (!plan.a_mn && !plan.b_mn) return launch_pair_t<false, false, false>(g, plan, s, max_ctas);
      if (!plan.a_mn && plan.b_mn) return launch_pair_t<false, true, false>(g, plan, s, max_ctas);
      if (plan.a_mn && !plan.b_mn) return launch_pair_t<true, false, false>(g, plan, s, max_ctas);
      return launch_pair_t<true, true, false>(g, plan, s, max_ctas);
    }
    // fused epilogues occur on forward (both operands K-major) and dgrad (B MN-major) GEMMs only
    if (!plan.a_mn && !plan.b_mn) return launch_pair_t<false, false, true>(g, plan, s, max_ctas);
    if (!plan.a_mn && plan.b_mn) return launch_pair_t<false, true, true>(g, plan, s, max_ctas);
  }
  switch (plan.bn) {
    case 64: return simple ? launch_bn<64, false>(g, plan, s, max_ctas) : launch_bn<64, true>(g, plan, s, max_ctas);
    case 256: return simple ? launch_bn<256, false>(g, plan, s, max_ctas) : launch_bn<256, true>(g, plan, s, max_ctas);
    default: return simple ? launch_bn<128, false>(g, plan, s, max_ctas) : launch_bn<128, true>(g, plan, s, max_ctas);
  }
}

}  // namespace erase
