// Tensor-core GEMM path for bf16 models on sm_100a: operands staged in shared memory by TMA
// (cp.async.bulk.tensor, 128-byte swizzle), tcgen05.mma issued by one thread with the fp32
// accumulator in tensor memory (TMEM), epilogue warps reading it back with tcgen05.ld and
// applying the fused epilogue (bias, ReLU, residual, DCN-v2 cross, ReLU derivative; GEMMs that ask
// for GELU or a pre-activation copy are refused here and use the SIMT kernel).
// One kernel serves the forward (both operands K-major), the dgrad (B MN-major) and the wgrad
// (both MN-major), so no operand is ever transposed in memory.  tc_gemm_plan picks the single-CTA
// kernel (128 x BN tiles) or the CTA-pair kernel (256 x 256 tiles over two SMs, cta_group::2).
#pragma once
#include <cuda_runtime.h>

#include "kernels.cuh"

namespace erase {

struct TcPlan {
  unsigned char map_a[128];  // CUtensorMap of A (copied into an aligned object at launch)
  unsigned char map_b[128];  // CUtensorMap of B
  unsigned char map_c[128];  // CUtensorMap of the output (or of the split-K partials), if tma_c
  unsigned char map_b_half[128];  // CTA-pair kernel, K-major B: box of 128 rows (each CTA stages half of the 256 columns)
  int tma_c = 0;
  int pair = 0;       // run the CTA-pair kernel (tcgen05 cta_group::2, 256 x 256 tiles)
  int pair_tmem_cols = 512;
  int bn = 128;       // tile width (N)
  int a_mn = 0;       // A is contiguous along M (not along K)
  int b_mn = 0;
  int launches = 1;
  int* status = nullptr;  // device word set non-zero when a bounded wait expired
  int* sched = nullptr;   // two zero-initialised device ints for dynamic tile scheduling (null: static order)
  long long* dbg = nullptr;  // optional device buffer (16 slots) for clock64 stamps of CTA 0, development aid
  int xcol = 0;              // the launch also forms GemmArgs::xcol_out (extra-column product)
};

// True if the tensor-core kernel can take this GEMM: bf16 operands, 16-byte aligned bases,
// leading strides that are multiples of 8 elements, K >= 64 and N >= 16.
bool tc_gemm_supported(const GemmArgs& g);
// Encodes the TMA descriptors.  g.ws must already point at splits*M*N floats when g.splits > 1.
// Returns false (and leaves the GEMM to the SIMT kernel) if a descriptor cannot be encoded.
bool tc_gemm_plan(const GemmArgs& g, int* status, TcPlan* plan);
// Cross-entropy head forward (g.epi.ce_ref set): columns per partial-sum group of ce_psum for this plan;
// ce_groups must be ceil(N / that).
int tc_ce_group_cols(const TcPlan& plan);
// max_ctas > 0 caps the persistent grid (an SM budget: lets kernels of other streams run beside it);
// the tile-to-CTA assignment does not enter the arithmetic, so results do not depend on it.
cudaError_t tc_gemm_launch(const GemmArgs& g, const TcPlan& plan, cudaStream_t s, int max_ctas = 0);

// Up to four weight-gradient GEMMs (both operands MN-major, g.splits >= 1, g.ws set: fp32 partials)
// in one launch; each problem's partials still need splitk_reduce.
struct TcGroupPlan {
  int n = 0, total = 0;
  int M[4], N[4], K[4], splits[4], kchunk[4], tiles_m[4], tiles_n[4], tile_begin[4];
  unsigned char map_a[4][128], map_b[4][128], map_c[4][128];
  int* status = nullptr;
};
bool tc_wgrad_group_plan(const GemmArgs* gs, int n, int* status, TcGroupPlan* plan);
cudaError_t tc_wgrad_group_launch(const TcGroupPlan& plan, cudaStream_t s, int max_ctas = 0);

// Dual-list persistent kernel: up to tc_dual_max() problems in two ordered lists (list 0: the forward of
// one block, list 1: the backward of another), each list on its own share of the SMs, in ONE launch.
//   kind 0: GEMM g (bf16, tensor-core shapes; epilogue: bias, ReLU, ReLU derivative; split-K writes its
//           fp32 partials to g.ws, which the caller reduces afterwards as for tc_gemm_launch)
//   kind 1: ew_dst = gelu(ew_src); kind 2: ew_dst *= gelu'(ew_src)   (bf16, ew_n % 8 == 0)
// A problem that is not a leaf is waited for by the problems behind it in its list (they read its
// output); a leaf (a weight gradient) is read by nothing inside the launch.  done_dev: tc_dual_max() ints of
// device memory owned by the caller (cleared by every launch).  Returns null if a problem does not fit.
struct DualItem {
  int kind = 0;
  GemmArgs g;
  const void* ew_src = nullptr;
  void* ew_dst = nullptr;
  long long ew_n = 0;
  int list = 0;
  int leaf = 0;
};
struct TcDualPlan;
int tc_dual_max();
TcDualPlan* tc_dual_plan(const DualItem* items, int n, int* done_dev, int* status);
void tc_dual_free(TcDualPlan* plan);
cudaError_t tc_dual_launch(const TcDualPlan* plan, cudaStream_t s);

// TMA descriptor (128 bytes, a CUtensorMap) of a row-major bf16 matrix with `inner` contiguous
// elements per row and `outer` rows `ld` elements apart: tiles of 64 columns x box_rows rows,
// 128-byte swizzle, zero fill outside.  False if the layout cannot be described (alignment).
bool tc_encode_rows_bf16(void* map128, const void* base, long long inner, long long outer, long long ld, int box_rows);

// Launches one thread that waits, for at most limit_cycles SM clocks, on a barrier nothing signals,
// then sets *status to 8 and returns: the bounded-wait helper of the GEMM kernels on its own.
cudaError_t tc_wait_selftest(int* status, long long limit_cycles, cudaStream_t s);

}  // namespace erase
