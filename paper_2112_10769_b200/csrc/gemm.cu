// 4-bit training GEMMs on tcgen05 / tensor memory (sm_100a).
//
//   D[Mo x No] = scale * sum_s sum_k opA_s[mo, k] * opB[no, k]
//
// serves the three products of the path (forward, backward, update); the
// operands are packed 4-bit codes in global memory, stored either k-contiguous
// ("K-major": rows are mo / no) or contraction-major ("MN-major": rows are k).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0       TMA producer for packed slabs (128 rows x 64 bytes) -> packed ring
//   warp 6       TMA producer for operand planes (128 rows x 128 bytes, already
//                8-bit, 128-byte swizzle) -> straight into the operand ring
//   warps 7-..   converters (8 or 16 warps, by how many operands arrive packed): packed
//                nibbles -> 8-bit operands, written in the 128-byte swizzled layout the
//                tensor core reads
//   warp 1       one thread issues tcgen05.mma (128 x 256 x 32 per instruction),
//                accumulators live in tensor memory, two buffers of 256 columns
//   warps 2-5    epilogue: tcgen05.ld -> scale -> swizzled staging -> TMA store
// Every slab, in either orientation, expands to 128 rows x 128 bytes; only the
// matrix descriptor differs between orientations.
//
// Shared-memory bandwidth bounds the in-kernel expansion (TMA write + converter
// read + converter write + tensor-core read of every operand byte).  An operand
// that many tiles re-read (the weights; the gradient in the backward and update
// products) is therefore fetched as bytes, by TMA in its final layout: the bytes
// the quantizer wrote beside the codes if the caller passes them, else an 8-bit
// "plane" that a small kernel expands into the context workspace.  Only operands
// used by a single row or column of tiles are expanded inside the GEMM.
//
// A second kernel (luq_gemm_pair_kernel, option LUQ_OPT_PAIRS) runs products
// whose operands both arrive as bytes on CTA pairs: tcgen05 cta_group::2, one
// 256-row tile per pair, each CTA fetching half of B.
//
// Operand bytes.  kind::f8f6f4: e4m3 through a 16-entry byte table (PRMT).
// kind::i8: LUQ levels +-2^(c-1) through the table; INT4 integers without a
// table - the two's-complement nibble moved to the high half of a byte is the
// int8 value 16*q, and the epilogue divides by 16 per INT4 operand (exact).
//
// Few output tiles (the update GEMM): the contraction is split over CTAs, each
// stores its partial tile to a workspace and a second kernel adds them in a fixed
// order (deterministic; no atomics).
// All waits are bounded; on expiry the CTA flags LUQ_STATUS_TIMEOUT, drains its
// copies, frees its tensor memory and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "int4_math.cuh"

namespace {

using namespace luqdev;

constexpr int BM = 128;            // output rows per tile (tensor-memory lanes)
constexpr int BN = 256;            // output columns per tile
constexpr int BK = 128;            // contraction elements per pipeline stage
constexpr int kSlabRows = 128;
constexpr int kPackedSlab = kSlabRows * 64;      // bytes
constexpr int kExpandedSlab = kSlabRows * 128;   // bytes
constexpr int kSlabs = 1 + BN / 128;             // A, B0, B1
constexpr int kExpandedStage = kSlabs * kExpandedSlab;
constexpr int kFirstEpiWarp = 2;
constexpr int kPlaneWarp = 6;
constexpr int kFirstConvWarp = 7;
constexpr int kTmemCols = 2 * BN;
constexpr int kTileFloats = BM * BN;
// Returns once every lane of the warp holds the words it loaded into w[0..count): the vote
// consumes a value computed from all of them, so it cannot complete while a load is outstanding, and
// it doubles as the warp barrier.  The side effect (an atomic OR with zero, taken when some lane's
// words happen to OR to one particular pattern) only keeps the compiler from discarding the chain.
__device__ __forceinline__ uint32_t loads_landed(const uint4* w, int count, unsigned int* status) {
  uint32_t seen = 0u;
#pragma unroll
  for (int j = 0; j < count; ++j) seen |= w[j].x | w[j].y | w[j].z | w[j].w;
  const uint32_t rare = __any_sync(0xFFFFFFFFu, seen == 0x9E3779B9u);
  if (rare && (threadIdx.x & 31) == 0) atomicOr(status, 0u);
  return rare;
}
// an arrival that carries the value returned above as an operand, so that it cannot be issued before the vote
__device__ __forceinline__ void mbar_arrive_after(uint32_t bar, uint32_t token) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];   // after %1" ::"r"(bar), "r"(token) : "memory");
}

constexpr int kStageBox = 32 * 32 * 4;           // one 32 x 32 fp32 store box
constexpr int kMaxBarriers = 24;

// Ring depths and shared-memory map for one choice of "which operands arrive as planes".
// ROWS (both operands planes, short contraction, fp32 output): the epilogue stages whole 1 KB output
// rows (32 KB per warp) and stores a strip with one 3-D copy; the operand ring is two stages deep.
constexpr int kStripBytes = 32 * BN * 4;         // 32 rows x 256 fp32
template <bool A_PLANE, bool B_PLANE, bool ROWS = false>
struct Cfg {
  static_assert(!ROWS || (A_PLANE && B_PLANE), "whole-row staging needs the room of the packed ring");
  static constexpr int packed_slabs = (A_PLANE ? 0 : 1) + (B_PLANE ? 0 : BN / 128);
  static constexpr int packed_stage = packed_slabs * kPackedSlab;
  static constexpr int b_packed_off = A_PLANE ? 0 : kPackedSlab;        // first B slab inside a packed stage
  static constexpr int ES = ROWS ? 2 : (A_PLANE && B_PLANE) ? 4 : ((A_PLANE || B_PLANE) ? 3 : 2);
  static constexpr int PS = packed_slabs == 0 ? 0 : (packed_slabs == 2 ? 3 : 4);
  static constexpr int plane_bytes = (A_PLANE ? kExpandedSlab : 0) + (B_PLANE ? (BN / 128) * kExpandedSlab : 0);
  // sixteen converter warps when all three slabs are expanded here, eight otherwise; with the
  // smaller CTA the register budget allows the epilogue to double-buffer its tensor-memory loads
  static constexpr int conv_warps = packed_slabs == 3 ? 16 : 8;
  static constexpr int conv_threads = conv_warps * 32;
  static constexpr int threads = 32 * (kFirstConvWarp + conv_warps);
  static constexpr bool epi_double = threads <= 512;
  static constexpr int tasks_per_thread = packed_slabs * 512 / conv_threads;
  // shared-memory offsets from the 1024-byte aligned base
  static constexpr int expanded = 0;
  static constexpr int packed = expanded + ES * kExpandedStage;
  static constexpr int staging = packed + PS * packed_stage;             // 4 warps x 2 boxes, or 4 strips
  static constexpr int barriers = staging + (ROWS ? 4 * kStripBytes : 4 * 2 * kStageBox);
  static constexpr int tmem_slot = barriers + 8 * kMaxBarriers;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int total = abort_flag + 4;
  static constexpr int smem_bytes = total + 1024;                        // slack to align the base
  static_assert(smem_bytes <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
  static_assert(2 * PS + 2 * ES + 4 <= kMaxBarriers, "barrier area too small");
  static_assert(packed_slabs * 512 % conv_threads == 0, "converter tasks must divide evenly");
};

struct GemmParams {
  const float* scale_a;
  const float* scale_b;
  unsigned int* status;
  long long Mo, No, Kc;
  int n_samples;
  int tiles_m, tiles_n;
  int out_bf16;          // the output tensor is bf16 (round to nearest even of the fp32 result), not fp32
  int num_kb;          // contraction blocks per sample plane
  int splits;          // contraction splits per tile
  int iters_per_split;
  float post_scale;    // 1/n_samples times the power of two that undoes the int8 operand scaling
  uint4 lut_a, lut_b;  // nibble -> operand byte
};

// tcgen05.ld of 32 accumulator columns, checked against the allocation in the checking build
// (the condition is the same in every lane of the warp; a violation reads zeros instead)
__device__ __forceinline__ void tmem_ld_32x32_chk(uint32_t tmem_base, unsigned int* status, uint32_t taddr, uint32_t (&r)[32]) {
  if (tmem_in(taddr, tmem_base, 512, status)) {
    tmem_ld_32x32(taddr, r);
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = 0u;
  }
}

// eight nibbles of `w` -> eight operand bytes through a 16-entry table
__device__ __forceinline__ void expand8_lut(uint32_t w, const uint4& lut, uint32_t& lo, uint32_t& hi) {
  const uint32_t sel0 = w & 0x7777u;
  const uint32_t sel1 = (w >> 16) & 0x7777u;
  const uint32_t pick0 = 0x3210u | ((w >> 1) & 0x4444u);
  const uint32_t pick1 = 0x3210u | ((w >> 17) & 0x4444u);
  lo = __byte_perm(__byte_perm(lut.x, lut.y, sel0), __byte_perm(lut.z, lut.w, sel0), pick0);
  hi = __byte_perm(__byte_perm(lut.x, lut.y, sel1), __byte_perm(lut.z, lut.w, sel1), pick1);
}
// eight two's-complement nibbles -> eight int8 values 16*q.  PERMUTED keeps the
// even elements in `lo` and the odd ones in `hi` (a fixed permutation of the
// contraction index, legal when both operands of the product apply it).
template <bool PERMUTED>
__device__ __forceinline__ void expand8_int4_x16(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const uint32_t even = (w << 4) & 0xF0F0F0F0u;
  const uint32_t odd = w & 0xF0F0F0F0u;
  if constexpr (PERMUTED) { lo = even; hi = odd; }
  else { lo = __byte_perm(even, odd, 0x5140); hi = __byte_perm(even, odd, 0x7362); }
}
// two fp32 values -> two bf16 (round to nearest even), the first in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// 32 packed codes (16 bytes) -> 32 operand bytes in element order
template <int KIND, bool LUQ_CODES, bool PERMUTED>
__device__ __forceinline__ void expand32(const uint4& w, const uint4& lut, uint4& o0, uint4& o1) {
  if constexpr (KIND == 1 && !LUQ_CODES) {
    expand8_int4_x16<PERMUTED>(w.x, o0.x, o0.y);
    expand8_int4_x16<PERMUTED>(w.y, o0.z, o0.w);
    expand8_int4_x16<PERMUTED>(w.z, o1.x, o1.y);
    expand8_int4_x16<PERMUTED>(w.w, o1.z, o1.w);
  } else {
    expand8_lut(w.x, lut, o0.x, o0.y);
    expand8_lut(w.y, lut, o0.z, o0.w);
    expand8_lut(w.z, lut, o1.x, o1.y);
    expand8_lut(w.w, lut, o1.z, o1.w);
  }
}

// Expands a whole packed tensor into an 8-bit operand plane (element order kept).
template <int KIND, bool LUQ_CODES>
__global__ void __launch_bounds__(256) expand_plane_kernel(const uint4* __restrict__ codes, uint4* __restrict__ plane,
                                                           size_t pieces, uint4 lut) {
  pdl_wait();
  pdl_trigger();
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < pieces; i += stride) {
    uint4 o0, o1;
    expand32<KIND, LUQ_CODES, false>(__ldg(codes + i), lut, o0, o1);
    plane[2 * i] = o0;
    plane[2 * i + 1] = o1;
  }
}

// KIND 0 f8f6f4 / 1 i8; A_MN, B_MN operand orientation; A_LUQ: A holds LUQ codes (B is always
// INT4); A_PLANE / B_PLANE: the operand arrives as an 8-bit plane instead of packed codes
template <int KIND, bool A_MN, bool B_MN, bool A_LUQ, bool A_PLANE, bool B_PLANE, bool ROWS = false>
__global__ void __launch_bounds__((Cfg<A_PLANE, B_PLANE, ROWS>::threads), 1)
luq_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_out, const GemmParams p) {
  using C = Cfg<A_PLANE, B_PLANE, ROWS>;
  constexpr int PS = C::PS, ES = C::ES;
  constexpr int kConvWarps = C::conv_warps, kConvThreads = C::conv_threads;
  constexpr bool kAnyPacked = C::packed_slabs > 0;
  constexpr bool kAnyPlane = A_PLANE || B_PLANE;
  // with int8 operands and both INT4 operands expanded here and k-contiguous, the expansion may permute k
  constexpr bool kPermuteK = KIND == 1 && !A_MN && !B_MN && !A_LUQ && !A_PLANE && !B_PLANE;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* const gen = smem_raw + (base - raw);

  const uint32_t bar0 = base + C::barriers;
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_empty = [&](int s) { return bar0 + 8u * (PS + s); };
  auto ex_full = [&](int s) { return bar0 + 8u * (2 * PS + s); };
  auto ex_empty = [&](int s) { return bar0 + 8u * (2 * PS + ES + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * PS + 2 * ES + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * PS + 2 * ES + 2 + b); };
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + C::tmem_slot);
  volatile uint32_t* const abort_flag = reinterpret_cast<volatile uint32_t*>(gen + C::abort_flag);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PS; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), kConvWarps); }
    for (int s = 0; s < ES; ++s) {
      mbar_init(ex_full(s), (kAnyPacked ? kConvWarps : 0) + (kAnyPlane ? 1 : 0));
      mbar_init(ex_empty(s), 1);
    }
    // whole-row staging has two epilogue warps per quarter of the accumulator's rows
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), ROWS ? 8 : 4); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tm_a); tma_prefetch_desc(&tm_b); tma_prefetch_desc(&tm_out); }
  if (warp == 1) {  // this warp owns the tensor-memory allocation
    tmem_alloc(base + C::tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done (barriers, tensor memory, descriptor prefetch): from here on global memory is
  // touched, which has to wait for the preceding kernel of the stream
  pdl_wait();
  pdl_trigger();

  const int units = p.tiles_m * p.tiles_n * p.splits;
  const int total_iters = p.n_samples * p.num_kb;

  // Tile order.  Unsplit products walk along the rows of the output: the CTAs that run at the same
  // time then write whole output rows (an output-bound product gains 6 % of write bandwidth,
  // measured with the bare store pattern) and share the row panel of A.  Split products keep the
  // order of the reduction kernel, down the columns.
  auto tile_m = [&](int tile) { return p.splits == 1 ? tile / p.tiles_n : tile % p.tiles_m; };
  auto tile_n = [&](int tile) { return p.splits == 1 ? tile % p.tiles_n : tile / p.tiles_m; };
  const int u_begin = static_cast<int>(blockIdx.x), u_end = units, u_step = static_cast<int>(gridDim.x);
  auto unit_range = [&](int u, int& tile, int& it_begin, int& it_end) {
    tile = u / p.splits;
    const int sp = u - tile * p.splits;
    it_begin = sp * p.iters_per_split;
    it_end = min(total_iters, it_begin + p.iters_per_split);
  };

  if (warp == 0) {
    // ------------------------------------------------- producer of packed slabs
    if (kAnyPacked && lane == 0) {
      // stage index and phase are counted, not divided: this loop is one thread's serial
      // instruction stream and must stay well below the time of a stage
      uint32_t issued = 0, stage = 0, phase = 0;
      bool ok = true;
      for (int u = u_begin; ok && u < u_end; u += u_step) {
        int tile, it_begin, it_end;
        unit_range(u, tile, it_begin, it_end);
        const int m0 = tile_m(tile) * BM;
        const int n0 = tile_n(tile) * BN;
        int sample = it_begin / p.num_kb;
        int kb = it_begin - sample * p.num_kb;
        for (int k_it = it_begin; k_it < it_end; ++k_it) {
          const uint32_t full = pk_full(stage);
          if (!mbar_wait(pk_empty(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = base + C::packed + stage * C::packed_stage;
          mbar_arrive_expect_tx(full, C::packed_stage);
          if constexpr (!A_PLANE) {
            if constexpr (A_MN) tma_load_3d(dst, &tm_a, full, m0 / 2, kb * BK, sample);
            else tma_load_3d(dst, &tm_a, full, kb * (BK / 2), m0, sample);
          }
          if constexpr (!B_PLANE) {
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) {
              const uint32_t d = dst + C::b_packed_off + j * kPackedSlab;
              if constexpr (B_MN) tma_load_2d(d, &tm_b, full, n0 / 2 + 64 * j, kb * BK);
              else tma_load_2d(d, &tm_b, full, kb * (BK / 2), n0 + 128 * j);
            }
          }
          ++issued;
          if (++kb == p.num_kb) { kb = 0; ++sample; }
          if (++stage == static_cast<uint32_t>(PS)) { stage = 0; phase ^= 1u; }
        }
      }
      // drain: every copy this thread issued must have landed before the CTA may exit
      for (int s = 0; s < PS; ++s) {
        if (issued > static_cast<uint32_t>(s)) {
          const uint32_t last = ((issued - 1 - s) / (PS > 0 ? PS : 1));  // last fill index of stage s
          mbar_wait(pk_full(s), last & 1u, abort_flag);
        }
      }
    }
  } else if (warp == kPlaneWarp) {
    // ------------------------------------------------ producer of operand planes
    if (kAnyPlane && lane == 0) {
      uint32_t issued = 0, stage = 0, phase = 0;
      bool ok = true;
      for (int u = u_begin; ok && u < u_end; u += u_step) {
        int tile, it_begin, it_end;
        unit_range(u, tile, it_begin, it_end);
        const int m0 = tile_m(tile) * BM;
        const int n0 = tile_n(tile) * BN;
        int sample = it_begin / p.num_kb;
        int kb = it_begin - sample * p.num_kb;
        for (int k_it = it_begin; k_it < it_end; ++k_it) {
          const uint32_t full = ex_full(stage);
          if (!mbar_wait(ex_empty(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t dst = base + C::expanded + stage * kExpandedStage;
          mbar_arrive_expect_tx(full, C::plane_bytes);
          if constexpr (A_PLANE) {
            if constexpr (A_MN) tma_load_3d(dst, &tm_a, full, m0, kb * BK, sample);
            else tma_load_3d(dst, &tm_a, full, kb * BK, m0, sample);
          }
          if constexpr (B_PLANE) {
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) {
              const uint32_t d = dst + (1 + j) * kExpandedSlab;
              if constexpr (B_MN) tma_load_2d(d, &tm_b, full, n0 + 128 * j, kb * BK);
              else tma_load_2d(d, &tm_b, full, kb * BK, n0 + 128 * j);
            }
          }
          ++issued;
          if (++kb == p.num_kb) { kb = 0; ++sample; }
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
      }
      for (int s = 0; s < ES; ++s) {
        if (issued > static_cast<uint32_t>(s)) {
          const uint32_t last = ((issued - 1 - s) / ES);
          mbar_wait(ex_full(s), last & 1u, abort_flag);
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = (KIND == 0 ? (1u << 4) : (2u << 4))        // accumulator: F32 / S32
                                 | ((KIND == 0 ? 0u : 1u) << 7)             // A: E4M3 / signed 8-bit
                                 | ((KIND == 0 ? 0u : 1u) << 10)            // B: E4M3 / signed 8-bit
                                 | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16)
                                 | (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
      // descriptors of stage 0; a stage or a 32-deep step further only moves the 14-bit
      // address field (shared memory is below 256 KB, the field cannot carry out)
      const uint32_t a0 = base + C::expanded, b0 = a0 + kExpandedSlab;
      const uint64_t da0 = A_MN ? umma_desc_sw128(a0, kExpandedSlab, 1024) : umma_desc_sw128(a0, 16, 1024);
      const uint64_t db0 = B_MN ? umma_desc_sw128(b0, kExpandedSlab, 1024) : umma_desc_sw128(b0, 16, 1024);
      constexpr uint64_t kStepA = (A_MN ? 32 * 128 : 32) >> 4, kStepB = (B_MN ? 32 * 128 : 32) >> 4;
      constexpr uint64_t kStageStep = kExpandedStage >> 4;
      uint32_t stage = 0, phase = 0, tile_it = 0;
      bool ok = true;
      for (int u = u_begin; ok && u < u_end; u += u_step, ++tile_it) {
        int tile, it_begin, it_end;
        unit_range(u, tile, it_begin, it_end);
        const uint32_t buf = tile_it & 1u;
        if (!mbar_wait(acc_empty(buf), ((tile_it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        uint32_t accumulate = 0;
        for (int k_it = it_begin; k_it < it_end; ++k_it) {
          if (!mbar_wait(ex_full(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = da0 + stage * kStageStep, db = db0 + stage * kStageStep;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            tc_mma<KIND>(tmem_d, da + kk * kStepA, db + kk * kStepB, idesc, accumulate);
            accumulate = 1;
          }
          tc_commit(ex_empty(stage));
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(acc_full(buf));
      }
    }
  } else if (warp < kPlaneWarp || (ROWS && warp >= kFirstConvWarp && warp < kFirstConvWarp + 4)) {
    // ---------------------------------------------------------------- epilogue
    // (whole-row staging: the kernel has no converters, and four of their warps form a second
    // epilogue group - a warp may only read the quarter of tensor memory given by its index mod 4,
    // so the two warps of a quarter share its rows and take four 32-column chunks each)
    const int quarter = warp & 3;  // tensor-memory lanes this warp may read
    const int half = warp >= kFirstConvWarp ? 1 : 0;
    const float scale = p.splits == 1 ? (__ldg(p.scale_a) * __ldg(p.scale_b)) * p.post_scale : 1.0f;
    const uint32_t stage0 = base + C::staging + ((warp - kFirstEpiWarp) & 3) * 2 * kStageBox;
    uint8_t* const stage0_gen = gen + C::staging + ((warp - kFirstEpiWarp) & 3) * 2 * kStageBox;
    const int sw = lane & 7;
    const bool out_bf16 = p.out_bf16 && p.splits == 1;   // partial tiles of a split stay fp32
    uint32_t tile_it = 0, box_it = 0;
    bool ok = true;
    for (int u = u_begin; ok && u < u_end; u += u_step, ++tile_it) {
      int tile, it_begin, it_end;
      unit_range(u, tile, it_begin, it_end);
      // a split stores its whole partial tile at row u*128 of the workspace
      const long long row0 = (p.splits == 1 ? static_cast<long long>(tile_m(tile)) * BM
                                            : static_cast<long long>(u) * BM) + quarter * 32;
      const long long col_base = p.splits == 1 ? static_cast<long long>(tile_n(tile)) * BN : 0;
      const long long row_limit = p.splits == 1 ? p.Mo : static_cast<long long>(units) * BM;
      const long long col_limit = p.splits == 1 ? p.No : BN;
      const uint32_t buf = tile_it & 1u;
      if (!mbar_wait(acc_full(buf), (tile_it >> 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN;
      // scale one 32 x 32 block held in registers, stage it (swizzled) and hand it to the TMA store
      auto emit = [&](const uint32_t (&r)[32], int c) {
        const long long col0 = col_base + c * 32;
        if (row0 < row_limit && col0 < col_limit) {   // warp-uniform
          const uint32_t b = box_it & 1u;
          ++box_it;
          if (lane == 0) bulk_wait_read<1>();          // the store that last read this box is done
          __syncwarp();
          auto value = [&](int i) {
            const float acc = KIND == 0 ? __uint_as_float(r[i]) : static_cast<float>(static_cast<int>(r[i]));
            return acc * scale;
          };
          if (out_bf16) {
            // 32 columns of bf16 = 64 bytes per row: four 16-byte pieces, 64-byte swizzle (piece ^ row/2)
            uint8_t* const rowp = stage0_gen + b * kStageBox + lane * 64;
            const int sw64 = (lane >> 1) & 3;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint4 v;
              v.x = pack_bf16x2(value(8 * j), value(8 * j + 1));
              v.y = pack_bf16x2(value(8 * j + 2), value(8 * j + 3));
              v.z = pack_bf16x2(value(8 * j + 4), value(8 * j + 5));
              v.w = pack_bf16x2(value(8 * j + 6), value(8 * j + 7));
              if (smem_in(rowp + ((j ^ sw64) << 4), gen, C::staging, C::barriers, 16, p.status))
                *reinterpret_cast<uint4*>(rowp + ((j ^ sw64) << 4)) = v;
            }
          } else {
            uint8_t* const rowp = stage0_gen + b * kStageBox + lane * 128;
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (smem_in(rowp + ((j ^ sw) << 4), gen, C::staging, C::barriers, 16, p.status))
                *reinterpret_cast<float4*>(rowp + ((j ^ sw) << 4)) =
                    make_float4(value(4 * j), value(4 * j + 1), value(4 * j + 2), value(4 * j + 3));
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tm_out, stage0 + b * kStageBox, static_cast<int>(col0), static_cast<int>(row0));
            bulk_commit();
          }
        }
      };
      if constexpr (ROWS) {
        // Whole rows: the strip of this warp (32 rows x 256 columns) is staged as the image of ONE 3-D
        // box [row][32-column chunk][32 floats] - rows are 1 KB apart, so the 128-byte swizzle is keyed
        // on the chunk: 16-byte unit u of chunk c lies at slot u ^ c.  A thread holds one row; were all
        // threads to write unit s at step s they would hit one bank.  So thread `lane` writes unit
        // s ^ (lane & 7) at step s: its units are first permuted by that XOR (three rounds of
        // conditional swaps), and eight consecutive lanes then cover the eight slots of a 128-byte line.
        // The two warps of a quarter fill the same strip (chunks 0-3 and 4-7) and meet at a
        // named barrier of 64 threads before and after: the first warp waits for the previous
        // store to have read the strip, and issues this tile's store.
        const int slot = (warp - kFirstEpiWarp) & 3;
        const uint32_t strip = base + C::staging + slot * kStripBytes;
        uint8_t* const rowp = gen + C::staging + slot * kStripBytes + lane * (BN * 4);
        const bool in_range = row0 < row_limit;       // warp-uniform
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + slot) : "memory"); };
        auto emit_rows = [&](uint32_t (&r)[32], int c) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float acc = KIND == 0 ? __uint_as_float(r[i]) : static_cast<float>(static_cast<int>(r[i]));
            r[i] = __float_as_uint(acc * scale);
          }
#pragma unroll
          for (int bit = 0; bit < 3; ++bit) {
            const bool flip = (sw >> bit) & 1;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              if (u & (1 << bit)) continue;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t x = r[4 * u + e], y = r[4 * (u | (1 << bit)) + e];
                r[4 * u + e] = flip ? y : x;
                r[4 * (u | (1 << bit)) + e] = flip ? x : y;
              }
            }
          }
          uint8_t* const line = rowp + c * 128;
          const int key = sw ^ (c & 7);
#pragma unroll
          for (int s = 0; s < 8; ++s)   // position s holds unit s ^ sw, whose slot is (s ^ sw) ^ c
            if (smem_in(line + ((s ^ key) << 4), gen, C::staging, C::barriers, 16, p.status))
              *reinterpret_cast<uint4*>(line + ((s ^ key) << 4)) = make_uint4(r[4 * s], r[4 * s + 1], r[4 * s + 2], r[4 * s + 3]);
        };
        constexpr int kChunks = BN / 32 / 2;          // chunks per warp
        const int c_first = half * kChunks;
        uint32_t r0[32], r1[32];
        tmem_ld_32x32_chk(tmem_base, p.status, taddr + c_first * 32, r0);
        // first write of this tile: the previous tile's store must have read the strip
        if (half == 0 && lane == 0) bulk_wait_read<0>();
        pair_sync();
        tmem_ld_wait();
#pragma unroll 1
        for (int c = c_first; c < c_first + kChunks; c += 2) {
          tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 1) * 32, r1);
          emit_rows(r0, c);
          tmem_ld_wait();
          if (c + 2 < c_first + kChunks) tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 2) * 32, r0);
          emit_rows(r1, c + 1);
          tmem_ld_wait();
        }
        fence_proxy_async();
        pair_sync();
        if (half == 0 && lane == 0 && in_range) {   // chunks and rows beyond the tensor are clipped by the copy
          tma_store_3d(&tm_out, strip, 0, static_cast<int>(col_base / 32), static_cast<int>(row0));
          bulk_commit();
        }
      } else if constexpr (C::epi_double) {
        // two register sets: the tensor-memory load of the next block is in flight while this one is emitted
        uint32_t r0[32], r1[32];
        tmem_ld_32x32_chk(tmem_base, p.status, taddr, r0);
        tmem_ld_wait();
#pragma unroll 1
        for (int c = 0; c < BN / 32; c += 2) {
          tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 1) * 32, r1);
          emit(r0, c);
          tmem_ld_wait();
          if (c + 2 < BN / 32) tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 2) * 32, r0);
          emit(r1, c + 1);
          tmem_ld_wait();
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32_chk(tmem_base, p.status, taddr + c * 32, r);
          tmem_ld_wait();
          emit(r, c);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(buf));
    }
    if (lane == 0) bulk_wait<0>();   // all stores of this warp are complete before the CTA exits
  } else if (kAnyPacked) {
    // -------------------------------------------------------------- converters
    const int ctid = threadIdx.x - kFirstConvWarp * 32;
    uint32_t ps = 0, pphase = 0, es = 0, ephase = 0;
    bool ok = true;
    for (int u = u_begin; ok && u < u_end; u += u_step) {
      int tile, it_begin, it_end;
      unit_range(u, tile, it_begin, it_end);
      for (int k_it = it_begin; k_it < it_end; ++k_it) {
        if (!mbar_wait(pk_full(ps), pphase, abort_flag)) { ok = false; break; }
        if (!mbar_wait(ex_empty(es), ephase ^ 1u, abort_flag)) { ok = false; break; }
        const uint8_t* src = gen + C::packed + ps * C::packed_stage;
        uint8_t* dst = gen + C::expanded + es * kExpandedStage;
        constexpr int kTasks = C::tasks_per_thread > 0 ? C::tasks_per_thread : 1;
        uint4 w[kTasks];
#pragma unroll
        for (int j = 0; j < C::tasks_per_thread; ++j)
          w[j] = smem_in(src + (ctid + j * kConvThreads) * 16, gen, C::packed, C::staging, 16, p.status)
                     ? *reinterpret_cast<const uint4*>(src + (ctid + j * kConvThreads) * 16) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int j = 0; j < C::tasks_per_thread; ++j) {
          const int id = ctid + j * kConvThreads;
          const int pslab = id >> 9;                         // slab inside the packed stage, compile-time per j
          const int slab = A_PLANE ? pslab + 1 : pslab;      // slab inside the operand stage (0 = A)
          const int idx = id & 511;
          const int row = idx >> 2;
          const int q = idx & 3;
          uint4 o0, o1;
          if (slab == 0) expand32<KIND, A_LUQ, kPermuteK>(w[j], p.lut_a, o0, o1);
          else expand32<KIND, false, kPermuteK>(w[j], p.lut_b, o0, o1);
          uint8_t* drow = dst + slab * kExpandedSlab + row * 128;
          const int swz = row & 7;
          if (smem_in(drow + (((2 * q) ^ swz) << 4), gen, C::expanded, C::packed, 16, p.status))
            *reinterpret_cast<uint4*>(drow + (((2 * q) ^ swz) << 4)) = o0;
          if (smem_in(drow + (((2 * q + 1) ^ swz) << 4), gen, C::expanded, C::packed, 16, p.status))
            *reinterpret_cast<uint4*>(drow + (((2 * q + 1) ^ swz) << 4)) = o1;
        }
        fence_proxy_async();   // make the generic-proxy writes visible to the tensor core
        __syncwarp();
        if (lane == 0) { mbar_arrive(pk_empty(ps)); mbar_arrive(ex_full(es)); }
        if (++ps == static_cast<uint32_t>(PS > 0 ? PS : 1)) { ps = 0; pphase ^= 1u; }
        if (++es == static_cast<uint32_t>(ES)) { es = 0; ephase ^= 1u; }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, LUQ_STATUS_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------
// CTA-pair kernel (cluster of two, tcgen05 cta_group::2) for products whose two
// operands both arrive as planes.  A pair computes a 256 x 256 tile: each CTA
// loads its own 128 rows of A and its own 128 columns of B, one thread of the
// leader issues 256 x 256 x 32 MMAs that run on both SMs, each SM accumulates its
// 128 rows in its own tensor memory.  Per SM and stage that is 32 KB of operands
// instead of 48 KB - the operand fetch, not the tensor core, bounded the
// single-CTA kernel.
//   warp 0      TMA producer (its own A slab and B half; bytes counted on the leader's barrier)
//   warp 1      MMA issue (leader only); owns the tensor-memory allocation in both CTAs
//   warps 2-5   epilogue of this CTA's 128 rows
// Barriers: full[s] lives in the leader (one arrival, 64 KB of transactions from both
// CTAs); empty[s] and acc_full[b] exist in both CTAs and are signalled by one
// multicast commit; acc_empty[b] lives in the leader and counts the eight epilogue warps.
// ---------------------------------------------------------------------------
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kExpandedSlab;             // A slab + half of B
constexpr int kPairThreads = 32 * 6;
struct PairSmem {
  static constexpr int ring = 0;
  static constexpr int staging = ring + kPairStages * kPairStageBytes;
  static constexpr int barriers = staging + 4 * 2 * kStageBox;
  static constexpr int num_barriers = 2 * kPairStages + 4;
  static constexpr int tmem_slot = barriers + 8 * num_barriers;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int total = abort_flag + 4;
  static constexpr int smem_bytes = total + 1024;
  static_assert(smem_bytes <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
};

template <int KIND, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kPairThreads, 1)
luq_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_out, const GemmParams p) {
  constexpr int ES = kPairStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* const gen = smem_raw + (base - raw);
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  const uint32_t bar0 = base + PairSmem::barriers;
  auto full = [&](uint32_t s) { return bar0 + 8u * s; };
  auto empty = [&](uint32_t s) { return bar0 + 8u * (ES + s); };
  auto acc_full = [&](uint32_t b) { return bar0 + 8u * (2 * ES + b); };
  auto acc_empty = [&](uint32_t b) { return bar0 + 8u * (2 * ES + 2 + b); };
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + PairSmem::tmem_slot);
  volatile uint32_t* const abort_flag = reinterpret_cast<volatile uint32_t*>(gen + PairSmem::abort_flag);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < ES; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 8); }
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tm_a); tma_prefetch_desc(&tm_b); tma_prefetch_desc(&tm_out); }
  if (warp == 1) {  // the same warp of both CTAs allocates tensor memory for the pair
    tmem_alloc_pair(base + PairSmem::tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();   // barriers of both CTAs are initialised before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // set-up done (barriers, tensor memory, descriptor prefetch): from here on global memory is
  // touched, which has to wait for the preceding kernel of the stream
  pdl_wait();
  pdl_trigger();

  const int tiles_m2 = (p.tiles_m + 1) / 2;               // 256-row tiles
  const int tiles = tiles_m2 * p.tiles_n;
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
  const int total_iters = p.n_samples * p.num_kb;

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      uint32_t issued = 0, stage = 0, phase = 0;
      bool ok = true;
      for (int t = pair; ok && t < tiles; t += pairs) {
        const int m0 = (t % tiles_m2) * 256 + static_cast<int>(rank) * 128;    // this CTA's rows of A
        const int n0 = (t / tiles_m2) * BN + static_cast<int>(rank) * 128;     // this CTA's columns of B
        int sample = 0, kb = 0;
        for (int k_it = 0; k_it < total_iters; ++k_it) {
          if (!mbar_wait(empty(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t full_leader = mapa_shared(full(stage), 0);
          const uint32_t dst = base + PairSmem::ring + stage * kPairStageBytes;
          if (leader) mbar_arrive_expect_tx(full(stage), 2 * kPairStageBytes);   // both CTAs' bytes
          if constexpr (A_MN) tma_pair_load_3d(dst, &tm_a, full_leader, m0, kb * BK, sample);
          else tma_pair_load_3d(dst, &tm_a, full_leader, kb * BK, m0, sample);
          if constexpr (B_MN) tma_pair_load_2d(dst + kExpandedSlab, &tm_b, full_leader, n0, kb * BK);
          else tma_pair_load_2d(dst + kExpandedSlab, &tm_b, full_leader, kb * BK, n0);
          ++issued;
          if (++kb == p.num_kb) { kb = 0; ++sample; }
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
      }
      // drain: every copy of the pair counts its bytes on the leader's barriers, so the leader waits
      // for the last fill of every stage (both CTAs' copies have then landed); its peer leaves only
      // after the cluster barrier of the teardown, i.e. after this drain
      if (leader) {
        for (int s = 0; s < ES; ++s) {
          if (issued > static_cast<uint32_t>(s)) {
            const uint32_t last = (issued - 1 - s) / ES;
            mbar_wait_cluster(full(s), last & 1u, abort_flag);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------- MMA issue (leader only)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = (KIND == 0 ? (1u << 4) : (2u << 4)) | ((KIND == 0 ? 0u : 1u) << 7) |
                                 ((KIND == 0 ? 0u : 1u) << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                                 (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
      const uint32_t a0 = base + PairSmem::ring, b0 = a0 + kExpandedSlab;
      const uint64_t da0 = A_MN ? umma_desc_sw128(a0, kExpandedSlab, 1024) : umma_desc_sw128(a0, 16, 1024);
      const uint64_t db0 = B_MN ? umma_desc_sw128(b0, kExpandedSlab, 1024) : umma_desc_sw128(b0, 16, 1024);
      constexpr uint64_t kStepA = (A_MN ? 32 * 128 : 32) >> 4, kStepB = (B_MN ? 32 * 128 : 32) >> 4;
      constexpr uint64_t kStageStep = kPairStageBytes >> 4;
      uint32_t stage = 0, phase = 0, tile_it = 0;
      bool ok = true;
      for (int t = pair; ok && t < tiles; t += pairs, ++tile_it) {
        const uint32_t buf = tile_it & 1u;
        if (!mbar_wait_cluster(acc_empty(buf), ((tile_it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        uint32_t accumulate = 0;
        for (int k_it = 0; k_it < total_iters; ++k_it) {
          if (!mbar_wait_cluster(full(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = da0 + stage * kStageStep, db = db0 + stage * kStageStep;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            tc_mma_pair<KIND>(tmem_d, da + kk * kStepA, db + kk * kStepB, idesc, accumulate);
            accumulate = 1;
          }
          tc_commit_pair(empty(stage));
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit_pair(acc_full(buf));
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;
    const float scale = (__ldg(p.scale_a) * __ldg(p.scale_b)) * p.post_scale;
    const uint32_t stage0 = base + PairSmem::staging + (warp - kFirstEpiWarp) * 2 * kStageBox;
    uint8_t* const stage0_gen = gen + PairSmem::staging + (warp - kFirstEpiWarp) * 2 * kStageBox;
    const int sw = lane & 7;
    uint32_t tile_it = 0, box_it = 0;
    bool ok = true;
    for (int t = pair; ok && t < tiles; t += pairs, ++tile_it) {
      const long long row0 = static_cast<long long>(t % tiles_m2) * 256 + rank * 128 + quarter * 32;
      const long long col_base = static_cast<long long>(t / tiles_m2) * BN;
      const uint32_t buf = tile_it & 1u;
      if (!mbar_wait(acc_full(buf), (tile_it >> 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN;
      auto emit = [&](const uint32_t (&r)[32], int c) {
        const long long col0 = col_base + c * 32;
        if (row0 < p.Mo && col0 < p.No) {   // warp-uniform
          const uint32_t b = box_it & 1u;
          ++box_it;
          if (lane == 0) bulk_wait_read<1>();
          __syncwarp();
          uint8_t* const rowp = stage0_gen + b * kStageBox + lane * 128;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float4 v;
            if constexpr (KIND == 0) {
              v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                              __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
            } else {
              v = make_float4(static_cast<float>(static_cast<int>(r[4 * j])), static_cast<float>(static_cast<int>(r[4 * j + 1])),
                              static_cast<float>(static_cast<int>(r[4 * j + 2])), static_cast<float>(static_cast<int>(r[4 * j + 3])));
            }
            v.x *= scale; v.y *= scale; v.z *= scale; v.w *= scale;
            if (smem_in(rowp + ((j ^ sw) << 4), gen, PairSmem::staging, PairSmem::barriers, 16, p.status))
              *reinterpret_cast<float4*>(rowp + ((j ^ sw) << 4)) = v;
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tm_out, stage0 + b * kStageBox, static_cast<int>(col0), static_cast<int>(row0));
            bulk_commit();
          }
        }
      };
      uint32_t r0[32], r1[32];
      tmem_ld_32x32_chk(tmem_base, p.status, taddr, r0);
      tmem_ld_wait();
#pragma unroll 1
      for (int c = 0; c < BN / 32; c += 2) {
        tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 1) * 32, r1);
        emit(r0, c);
        tmem_ld_wait();
        if (c + 2 < BN / 32) tmem_ld_32x32_chk(tmem_base, p.status, taddr + (c + 2) * 32, r0);
        emit(r1, c + 1);
        tmem_ld_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(acc_empty(buf), 0));   // tell the leader this half is drained
    }
    if (lane == 0) bulk_wait<0>();
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while its peer may still signal it
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, LUQ_STATUS_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------
// Activation quantizer fused into the forward GEMM (Eq. Forward with Q_INT of
// Sec. 3.3 applied on the way in), for layers with one column of output tiles
// (N <= 256): every 128-row block of A is then read by exactly one tile, so the
// GEMM can take the HIGH-PRECISION activations, quantize them itself and write
// the packed codes (the update GEMM needs them) as a by-product.  The kernel
// streams A once at HBM speed and the tensor-core work hides under that stream.
//   warp 0       TMA producer of raw activations: boxes of 128 rows x 32 elements
//                (128-byte swizzle for fp32, 64-byte for bf16), two boxes per raw stage
//   warp 6       TMA producer of W's operand bytes (two 128 x 128 slabs per stage)
//   warps 7-22   converters, two groups of eight warps that take the raw stages in turn (one
//                group computes while the other waits at its barrier): one row of one box
//                per thread -> 32 INT4 codes; the codes go packed into a staging box that
//                one thread of the group stores with TMA (32-byte swizzle), and widened
//                (16 * q) into the A slab of the operand stage
//   warp 1       tcgen05.mma issue, kind::i8, accumulators in tensor memory (2 x 256 columns)
//   warps 2-5    epilogue (one 32 x 32 staging box per warp)
// An operand stage (128 deep) is made of two raw stages (64 deep).  Codes are
// bit-identical to the streaming quantizer's: same arithmetic (int4_math.cuh).
// ---------------------------------------------------------------------------
template <bool BF16>
struct FusedCfg {
  static constexpr int box_bytes = 128 * 32 * (BF16 ? 2 : 4);   // one raw box
  static constexpr int raw_stage = 2 * box_bytes;               // 64 contraction elements of 128 rows
  static constexpr int RS = BF16 ? 6 : 3;                       // raw stages: 96 KB
  static constexpr int ES = 2;                                  // operand stages (A slab + W's two slabs, 48 KB)
  static constexpr int code_box = 128 * 32;                     // packed codes of one raw stage
  static constexpr int conv_groups = 2;                         // converter groups, eight warps each
  static constexpr int threads = 32 * (kFirstConvWarp + 8 * conv_groups);
  static constexpr int expanded = 0;
  static constexpr int raw = expanded + ES * kExpandedStage;
  static constexpr int codes = raw + RS * raw_stage;            // two code boxes per converter group
  static constexpr int staging = codes + 2 * conv_groups * code_box;   // 4 warps x 1 box
  static constexpr int barriers = staging + 4 * kStageBox;
  static constexpr int num_barriers = 2 * RS + 2 * ES + 4;
  static constexpr int tmem_slot = barriers + 8 * num_barriers;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int cta_max = abort_flag + 4;     // largest |a| bit pattern this CTA has seen (in-hindsight form)
  static constexpr int total = cta_max + 4;
  static constexpr int smem_bytes = total + 1024;
  static_assert(smem_bytes <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
};

struct FusedParams {

  const float* clip;      // max|A| (or a caller's clip)
  const float* scale_b;   // weight scale
  float* scale_a_out;     // receives clip / 7
  // In-hindsight form (estimate != null, and clip == estimate): the kernel also measures max|A|, writes its
  // bit pattern to `measured` and replaces the estimate - see luq_quant_int4_hindsight.
  float* estimate; unsigned int* measured; unsigned int* scratch; float eta;
  unsigned int* status;
  long long Mo, No, Kc;
  int tiles_m, num_kb;
};

// the 256 threads of a converter group meet at named barrier `id`; returns true when every one of them passed `ok`
__device__ __forceinline__ bool conv_barrier_all(bool ok, uint32_t id) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred q, r;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred r, %2, 256, q;\n\t"
      "selp.u32 %0, 1, 0, r;\n\t}"
      : "=r"(out) : "r"(static_cast<uint32_t>(ok)), "r"(id) : "memory");
  return out != 0;
}

template <bool BF16>
__global__ void __launch_bounds__((FusedCfg<BF16>::threads), 1)
luq_quant_fwd_kernel(const __grid_constant__ CUtensorMap tm_raw, const __grid_constant__ CUtensorMap tm_b,
                     const __grid_constant__ CUtensorMap tm_codes, const __grid_constant__ CUtensorMap tm_out,
                     const FusedParams p) {
  using C = FusedCfg<BF16>;
  constexpr int RS = C::RS, ES = C::ES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* const gen = smem_raw + (base - raw);

  const uint32_t bar0 = base + C::barriers;
  auto raw_full = [&](int s) { return bar0 + 8u * s; };
  auto raw_empty = [&](int s) { return bar0 + 8u * (RS + s); };
  auto ex_full = [&](int s) { return bar0 + 8u * (2 * RS + s); };
  auto ex_empty = [&](int s) { return bar0 + 8u * (2 * RS + ES + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * RS + 2 * ES + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * RS + 2 * ES + 2 + b); };
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + C::tmem_slot);
  volatile uint32_t* const abort_flag = reinterpret_cast<volatile uint32_t*>(gen + C::abort_flag);
  uint32_t* const cta_max = reinterpret_cast<uint32_t*>(gen + C::cta_max);
  const bool track = p.estimate != nullptr;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < RS; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), 16); }   // all converter warps release a stage
    for (int s = 0; s < ES; ++s) {
      mbar_init(ex_full(s), 2 * 8 + 1);   // eight converter warps for each half of the A slab, and W's producer
      mbar_init(ex_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    *abort_flag = 0;
    *cta_max = 0u;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tm_raw); tma_prefetch_desc(&tm_b); tma_prefetch_desc(&tm_codes); tma_prefetch_desc(&tm_out);
  }
  if (warp == 1) {
    tmem_alloc(base + C::tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();
  pdl_trigger();
  // in-hindsight form: the estimate every CTA quantizes with; its replacement is written by the CTA
  // that finishes last, when no CTA can read it any more
  const float given = (track && threadIdx.x == 0) ? *p.clip : 0.0f;

  const int raw_iters = 2 * p.num_kb;   // raw stages per tile
  // Tiles are walked from the END of the tensor: the max reduction that precedes this kernel read
  // A front to back, so A's tail is what the L2 would still hold.  (Measured on a 462 MB tensor it
  // holds none of it - the two kernels take as long back to back as apart, also when the max pass
  // loads the tail with an evict-last hint - so the order costs nothing and gains nothing there.)

  if (warp == 0) {
    // ------------------------------------------ producer of raw activations
    if (lane == 0) {
      uint32_t issued = 0, stage = 0, phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < p.tiles_m; t += gridDim.x) {
        const int m0 = (p.tiles_m - 1 - t) * BM;   // back to front, see below
        for (int it = 0; it < raw_iters; ++it) {
          if (!mbar_wait(raw_empty(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t full = raw_full(stage);
          const uint32_t dst = base + C::raw + stage * C::raw_stage;
          mbar_arrive_expect_tx(full, C::raw_stage);
          tma_load_2d(dst, &tm_raw, full, it * 64, m0);                      // columns beyond K read as zero
          tma_load_2d(dst + C::box_bytes, &tm_raw, full, it * 64 + 32, m0);
          ++issued;
          if (++stage == static_cast<uint32_t>(RS)) { stage = 0; phase ^= 1u; }
        }
      }
      for (int s = 0; s < RS; ++s) {   // drain: every copy issued here has landed before the CTA exits
        if (issued > static_cast<uint32_t>(s)) {
          const uint32_t last = (issued - 1 - s) / RS;
          mbar_wait(raw_full(s), last & 1u, abort_flag);
        }
      }
    }
  } else if (warp == kPlaneWarp) {
    // ------------------------------------------ producer of W's operand bytes
    if (lane == 0) {
      uint32_t issued = 0, stage = 0, phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < p.tiles_m; t += gridDim.x) {
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!mbar_wait(ex_empty(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t full = ex_full(stage);
          const uint32_t dst = base + C::expanded + stage * kExpandedStage;
          mbar_arrive_expect_tx(full, 2 * kExpandedSlab);
          tma_load_2d(dst + kExpandedSlab, &tm_b, full, kb * BK, 0);
          tma_load_2d(dst + 2 * kExpandedSlab, &tm_b, full, kb * BK, 128);
          ++issued;
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
      }
      for (int s = 0; s < ES; ++s) {
        if (issued > static_cast<uint32_t>(s)) {
          const uint32_t last = (issued - 1 - s) / ES;
          mbar_wait(ex_full(s), last & 1u, abort_flag);
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10)      // S32 accumulator, signed 8-bit A and B
                                 | (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(BM >> 4) << 24);
      const uint32_t a0 = base + C::expanded, b0 = a0 + kExpandedSlab;
      const uint64_t da0 = umma_desc_sw128(a0, 16, 1024), db0 = umma_desc_sw128(b0, 16, 1024);
      constexpr uint64_t kStep = 32 >> 4, kStageStep = kExpandedStage >> 4;
      uint32_t stage = 0, phase = 0, tile_it = 0;
      bool ok = true;
      for (int t = blockIdx.x; ok && t < p.tiles_m; t += gridDim.x, ++tile_it) {
        const uint32_t buf = tile_it & 1u;
        if (!mbar_wait(acc_empty(buf), ((tile_it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        uint32_t accumulate = 0;
        for (int kb = 0; kb < p.num_kb; ++kb) {
          if (!mbar_wait(ex_full(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint64_t da = da0 + stage * kStageStep, db = db0 + stage * kStageStep;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            tc_mma<1>(tmem_d, da + kk * kStep, db + kk * kStep, idesc, accumulate);
            accumulate = 1;
          }
          tc_commit(ex_empty(stage));
          if (++stage == static_cast<uint32_t>(ES)) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(acc_full(buf));
      }
    }
  } else if (warp < kPlaneWarp) {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;
    const float clip = __ldg(p.clip);
    const float sa = scale_usable(clip, nullptr) ? clip / 7.0f : 0.0f;
    const float scale = (sa * __ldg(p.scale_b)) * (1.0f / 256.0f);   // both operands carry 16 * q
    const uint32_t box = base + C::staging + (warp - kFirstEpiWarp) * kStageBox;
    uint8_t* const rowp = gen + C::staging + (warp - kFirstEpiWarp) * kStageBox + lane * 128;
    const int sw = lane & 7;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int t = blockIdx.x; ok && t < p.tiles_m; t += gridDim.x, ++tile_it) {
      const long long row0 = static_cast<long long>(p.tiles_m - 1 - t) * BM + quarter * 32;
      const uint32_t buf = tile_it & 1u;
      if (!mbar_wait(acc_full(buf), (tile_it >> 1) & 1u, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN;
      auto emit = [&](const uint32_t (&r)[32], int c) {
        const long long col0 = c * 32;
        if (row0 < p.Mo && col0 < p.No) {   // warp-uniform
          if (lane == 0) bulk_wait_read<0>();          // the store that last read this box is done
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float4 v;
            v.x = static_cast<float>(static_cast<int>(r[4 * j])) * scale;
            v.y = static_cast<float>(static_cast<int>(r[4 * j + 1])) * scale;
            v.z = static_cast<float>(static_cast<int>(r[4 * j + 2])) * scale;
            v.w = static_cast<float>(static_cast<int>(r[4 * j + 3])) * scale;
            if (smem_in(rowp + ((j ^ sw) << 4), gen, C::staging, C::barriers, 16, p.status))
              *reinterpret_cast<float4*>(rowp + ((j ^ sw) << 4)) = v;
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tm_out, box, static_cast<int>(col0), static_cast<int>(row0));
            bulk_commit();
          }
        }
      };
      // one register set: with 23 warps in the CTA a thread has 88 registers, and this epilogue has
      // the whole main loop of the next tile (tens of microseconds) to finish in
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32_chk(tmem_base, p.status, taddr + c * 32, r);
        tmem_ld_wait();
        emit(r, c);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(buf));
    }
    if (lane == 0) bulk_wait<0>();
  } else if (warp >= kFirstConvWarp) {
    // -------------------------------------------------------------- converters
    const int group = (warp - kFirstConvWarp) >> 3;   // takes the raw stages of this parity
    const int cw = (warp - kFirstConvWarp) & 7;
    const int ctid = threadIdx.x - (kFirstConvWarp + 8 * group) * 32;   // 0..255 inside the group
    const int boxi = cw >> 2;                      // which box of the raw stage
    const int row = (cw & 3) * 32 + lane;          // row of the tile
    const float clip = track ? *p.clip : __ldg(p.clip);   // the in-hindsight form writes the estimate at its very end
    const bool first = blockIdx.x == 0 && group == 0 && ctid == 0;
    const bool usable = scale_usable(clip, first ? p.status : nullptr);
    const float inv = usable ? 7.0f / clip : 0.0f;   // an unusable clip gives zero codes and a zero scale
    if (first) *p.scale_a_out = usable ? clip / 7.0f : 0.0f;
    constexpr int kUnits = BF16 ? 4 : 8;           // 16-byte units of a box row
    // position of unit u of this row inside the swizzled box image
    const int rkey = BF16 ? ((row >> 1) & 3) : (row & 7);
    const uint32_t row_off = row * (BF16 ? 64 : 128);
    // raw stage number q (over the whole CTA): ring slot q % RS; operand stage q / 2, half q % 2.
    // raw_iters is even, so a group always fills the same half.  Both groups follow EVERY raw stage
    // (wait for it, release it) although each converts only its own: a waiter that skipped phases of
    // a barrier could no longer tell them apart by their parity, and a slot must not be refilled
    // before both groups have seen it filled.
    uint32_t q = 0, stored = 0;
    uint32_t seen = 0u;   // largest |a| bit pattern among this thread's elements (in-hindsight form)
    bool alive = true, ok = true;
    for (int t = blockIdx.x; alive && t < p.tiles_m; t += gridDim.x) {
      const int m0 = (p.tiles_m - 1 - t) * BM;
      for (int it = 0; it < raw_iters; ++it, ++q) {
        const uint32_t rs = q % RS, rphase = (q / RS) & 1u;
        const uint32_t es = (q >> 1) % ES, ephase = ((q >> 1) / ES) & 1u;
        ok = ok && mbar_wait_idle(raw_full(rs), rphase, abort_flag);
        if ((it & 1) != group) {          // the other group's stage
          __syncwarp();
          if (ok && lane == 0) mbar_arrive(raw_empty(rs));
          continue;
        }
        const uint32_t cbox_off = C::codes + (2 * group + (stored & 1u)) * C::code_box;
        uint4 u[kUnits];
        if (ok) {
          const uint8_t* src = gen + C::raw + rs * C::raw_stage + boxi * C::box_bytes + row_off;
#pragma unroll
          for (int j = 0; j < kUnits; ++j)
            u[j] = smem_in(src + ((j ^ rkey) << 4), gen, C::raw, C::codes, 16, p.status)
                       ? *reinterpret_cast<const uint4*>(src + ((j ^ rkey) << 4)) : make_uint4(0u, 0u, 0u, 0u);
          // The raw slot is given back as soon as this warp HOLDS its rows - before the operand stage is
          // free, before the conversion: what one SM can stream is the bytes its three raw slots keep in
          // flight, and a slot that waits for arithmetic, stores and a barrier is not in flight.  "Holds"
          // must be literal: the refill is a write of the async proxy, which the release semantics of an
          // arrival do not order against this warp's reads (arriving straight after issuing the loads
          // gave wrong codes about once in 150 calls).  loads_landed() returns only when every lane's
          // words are in registers.
          {
            const uint32_t token = loads_landed(u, kUnits, p.status);
            if (lane == 0) mbar_arrive_after(raw_empty(rs), token);
          }
          ok = mbar_wait_idle(ex_empty(es), ephase ^ 1u, abort_flag);
        }
        if (ok) {
          // 32 elements -> 32 codes (element e in nibble e % 8 of word e / 8) and 32 operand bytes 16 * q
          float v[32];
          if constexpr (BF16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t h[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                v[8 * j + 2 * i] = __uint_as_float(h[i] << 16);
                v[8 * j + 2 * i + 1] = __uint_as_float(h[i] & 0xFFFF0000u);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              v[4 * j] = __uint_as_float(u[j].x); v[4 * j + 1] = __uint_as_float(u[j].y);
              v[4 * j + 2] = __uint_as_float(u[j].z); v[4 * j + 3] = __uint_as_float(u[j].w);
            }
          }
          if (track) {   // copied columns beyond K and rows beyond M arrive as zeros
#pragma unroll
            for (int e = 0; e < 32; ++e) seen = max(seen, __float_as_uint(v[e]) & 0x7FFFFFFFu);
          }
          uint32_t lowb[8], any = 0u;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint32_t t0 = int4_round_bits(v[4 * g], inv), t1 = int4_round_bits(v[4 * g + 1], inv);
            const uint32_t t2 = int4_round_bits(v[4 * g + 2], inv), t3 = int4_round_bits(v[4 * g + 3], inv);
            any |= t0 | t1 | t2 | t3;
            lowb[g] = int4_low_bytes(t0, t1, t2, t3);
          }
          uint4 packed = make_uint4(int4_pack8(lowb[0], lowb[1]), int4_pack8(lowb[2], lowb[3]),
                                    int4_pack8(lowb[4], lowb[5]), int4_pack8(lowb[6], lowb[7]));
          uint4 o0 = make_uint4(int4_operand_bytes(lowb[0]), int4_operand_bytes(lowb[1]),
                                int4_operand_bytes(lowb[2]), int4_operand_bytes(lowb[3]));
          uint4 o1 = make_uint4(int4_operand_bytes(lowb[4]), int4_operand_bytes(lowb[5]),
                                int4_operand_bytes(lowb[6]), int4_operand_bytes(lowb[7]));
          if (any & 0x20000000u) {   // a NaN among the 32 products (rare): the element-wise rule, NaN -> 0
            uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int e = 0; e < 32; ++e) w[e >> 3] |= int4_code(v[e], inv) << (4 * (e & 7));
            packed = make_uint4(w[0], w[1], w[2], w[3]);
            expand32<1, false, false>(packed, make_uint4(0u, 0u, 0u, 0u), o0, o1);
          }
          // operand bytes, element order, into this row of the A slab (128-byte swizzle)
          uint8_t* drow = gen + C::expanded + es * kExpandedStage + row * 128;
          const int unit = group * 4 + boxi * 2;
          if (smem_in(drow + ((unit ^ (row & 7)) << 4), gen, C::expanded, C::raw, 16, p.status))
            *reinterpret_cast<uint4*>(drow + ((unit ^ (row & 7)) << 4)) = o0;
          if (smem_in(drow + (((unit + 1) ^ (row & 7)) << 4), gen, C::expanded, C::raw, 16, p.status))
            *reinterpret_cast<uint4*>(drow + (((unit + 1) ^ (row & 7)) << 4)) = o1;
          // packed codes into the staging box of this raw stage: 128 rows x 32 bytes, 32-byte swizzle
          if (smem_in(gen + cbox_off + row * 32 + ((boxi ^ ((row >> 2) & 1)) << 4), gen, C::codes, C::staging, 16, p.status))
            *reinterpret_cast<uint4*>(gen + cbox_off + row * 32 + ((boxi ^ ((row >> 2) & 1)) << 4)) = packed;
          fence_proxy_async();   // both writes are read by the async proxy (tensor core, TMA store)
        }
        // The group's two code boxes alternate.  Here the store issued one turn ago must have read its
        // box: after the barrier below every thread may go on to the next turn and write that box again.
        if (ctid == 0) bulk_wait_read<0>();
        alive = conv_barrier_all(ok, 5 + group);
        if (!alive) break;
        if (ctid == 0 && it * 64 < p.Kc) {
          tma_store_2d(&tm_codes, base + cbox_off, it * 32, m0);
          bulk_commit();
        }
        ++stored;
        if (lane == 0) mbar_arrive(ex_full(es));
      }
    }
    if (ctid == 0) bulk_wait<0>();
    if (track) {
      seen = __reduce_max_sync(0xFFFFFFFFu, seen);
      if (lane == 0) atomicMax(cta_max, seen);
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, LUQ_STATUS_TIMEOUT);
  if (track && threadIdx.x == 0) {
    // grid-wide maximum without a second launch: every CTA leaves its maximum in the scratch array
    // and takes a ticket; the one that draws the last ticket folds the array, writes the measured
    // maximum and the next estimate, and puts the ticket counter back to zero.  Nobody waits.
    __stcg(p.scratch + 2 + blockIdx.x, *cta_max);
    __threadfence();
    if (atomicAdd(p.scratch, 1u) == gridDim.x - 1) {
      __threadfence();
      uint32_t m = 0u;
      for (unsigned int b = 0; b < gridDim.x; ++b) m = max(m, __ldcg(p.scratch + 2 + b));
      *p.measured = m;   // Inf/NaN patterns win the maximum and raise the flag
      if (m >= 0x7F800000u) atomicOr(p.status, LUQ_STATUS_NONFINITE);
      *p.estimate = hindsight_next(m, given, p.eta);
      *p.scratch = 0u;
    }
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Sums the partial tiles of a split contraction in a fixed order, applies the
// scales and writes the output.  One thread per float4 of a tile.
__global__ void __launch_bounds__(256) split_reduce_kernel(const float* __restrict__ ws, void* __restrict__ out_any,
                                                           const float* __restrict__ scale_a,
                                                           const float* __restrict__ scale_b, float post_scale,
                                                           int tiles, int tiles_m, int splits, long long Mo,
                                                           long long No, int out_bf16) {
  pdl_wait();
  pdl_trigger();
  const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<long long>(tiles) * (kTileFloats / 4)) return;
  const int tile = static_cast<int>(idx / (kTileFloats / 4));
  const int rem = static_cast<int>(idx % (kTileFloats / 4));
  const int r = rem / (BN / 4), c4 = rem % (BN / 4);
  const float4* src = reinterpret_cast<const float4*>(ws) + (static_cast<size_t>(tile) * splits) * (kTileFloats / 4) + rem;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  int s = 0;
  for (; s + 8 <= splits; s += 8) {   // eight loads in flight, added in split order
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __ldcg(src + static_cast<size_t>(s + j) * (kTileFloats / 4));
#pragma unroll
    for (int j = 0; j < 8; ++j) { acc.x += v[j].x; acc.y += v[j].y; acc.z += v[j].z; acc.w += v[j].w; }
  }
  for (; s < splits; ++s) {
    const float4 v = __ldcg(src + static_cast<size_t>(s) * (kTileFloats / 4));
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  const long long row = static_cast<long long>(tile % tiles_m) * BM + r;
  const long long col = static_cast<long long>(tile / tiles_m) * BN + c4 * 4;
  if (row < Mo && col < No) {
    const float scale = (__ldg(scale_a) * __ldg(scale_b)) * post_scale;
    acc.x *= scale; acc.y *= scale; acc.z *= scale; acc.w *= scale;
    if (out_bf16)
      *reinterpret_cast<uint2*>(static_cast<uint16_t*>(out_any) + row * No + col) =
          make_uint2(pack_bf16x2(acc.x, acc.y), pack_bf16x2(acc.z, acc.w));
    else
      *reinterpret_cast<float4*>(static_cast<float*>(out_any) + row * No + col) = acc;
  }
}

// nibble -> operand byte tables.  kind 0: e4m3 (sign, 4-bit exponent bias 7, 3-bit
// mantissa); kind 1: two's-complement int8.  Every INT4 integer and every LUQ
// level 2^0..2^6 is exact in both.
uint8_t e4m3_of_int(int v) {
  static const uint8_t mag[16] = {0x00, 0x38, 0x40, 0x44, 0x48, 0x4A, 0x4C, 0x4E,
                                  0x50, 0x51, 0x52, 0x53, 0x54, 0x55, 0x56, 0x57};
  const int a = v < 0 ? -v : v;
  return static_cast<uint8_t>(mag[a] | (v < 0 ? 0x80 : 0));
}
uint4 make_lut(int mma_kind, int operand_kind) {
  uint8_t t[16];
  for (int n = 0; n < 16; ++n) {
    if (operand_kind == 0) {               // INT4 two's complement
      const int v = n < 8 ? n : n - 16;
      t[n] = mma_kind == 0 ? e4m3_of_int(v) : static_cast<uint8_t>(static_cast<int8_t>(v));
    } else if (operand_kind == 2) {        // unsigned INT4: the nibble is the value, 0..15
      t[n] = mma_kind == 0 ? e4m3_of_int(n) : static_cast<uint8_t>(n);
    } else {                               // LUQ: sign | c, value +-2^(c-1)
      const int c = n & 7, neg = n >> 3;
      if (c == 0) t[n] = 0;
      else if (mma_kind == 0) t[n] = static_cast<uint8_t>(((c + 6) << 3) | (neg << 7));
      else t[n] = static_cast<uint8_t>(static_cast<int8_t>(neg ? -(1 << (c - 1)) : (1 << (c - 1))));
    }
  }
  auto word = [&](int i) {
    return static_cast<uint32_t>(t[4 * i]) | (static_cast<uint32_t>(t[4 * i + 1]) << 8) |
           (static_cast<uint32_t>(t[4 * i + 2]) << 16) | (static_cast<uint32_t>(t[4 * i + 3]) << 24);
  };
  return make_uint4(word(0), word(1), word(2), word(3));
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// byte tensor `planes` x `rows` x `pitch` bytes.  Packed codes: box 1 x 128 rows x 64 bytes, no
// swizzle.  Operand planes: box 1 x 128 rows x 128 bytes, 128-byte swizzle (the tensor core's layout).
int encode_bytes_map(void* fn, CUtensorMap* map, const uint8_t* ptr, uint64_t pitch, uint64_t rows, uint64_t planes,
                     bool three_d, bool operand_plane) {
  const cuuint64_t dims[3] = {pitch, rows, planes};
  const cuuint64_t strides[2] = {pitch, pitch * rows};
  const cuuint32_t box[3] = {operand_plane ? 128u : 64u, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT8, three_d ? 3 : 2, const_cast<uint8_t*>(ptr), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, operand_plane ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}
// fp32 output (or workspace) tensor rows x cols, box = 32 rows x 32 columns, 128-byte swizzle in shared memory
// (bf16 output: the same box of 32 x 32 elements is 64 bytes wide, 64-byte swizzle)
int encode_out_map(void* fn, CUtensorMap* map, void* ptr, uint64_t rows, uint64_t cols, bool bf16) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * (bf16 ? 2 : 4)};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ptr, dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
      CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

// fp32 output as [rows][cols / 32][32]: a box is a strip of 32 rows x 8 chunks, whole 1 KB rows
int encode_out_rows_map(void* fn, CUtensorMap* map, void* ptr, uint64_t rows, uint64_t cols) {
  const cuuint64_t dims[3] = {32, cols / 32, rows};
  const cuuint64_t strides[2] = {128, cols * 4};
  const cuuint32_t box[3] = {32, BN / 32, 32};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

template <int KIND, bool A_MN, bool B_MN, bool A_LUQ>
int launch_rows(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to, const GemmParams& p, int grid,
                cudaStream_t st) {
  auto kernel = luq_gemm_kernel<KIND, A_MN, B_MN, A_LUQ, true, true, true>;
  constexpr int smem = Cfg<true, true, true>::smem_bytes;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return static_cast<int>(e);
  return static_cast<int>(luq_launch_kernel(kernel, grid, Cfg<true, true, true>::threads, smem, st, LUQ_LAUNCH_EARLY, 1, ta, tb, to, p));
}

template <int KIND, bool A_MN, bool B_MN, bool A_LUQ, bool A_PLANE, bool B_PLANE>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to, const GemmParams& p, int grid,
           cudaStream_t st) {
  auto kernel = luq_gemm_kernel<KIND, A_MN, B_MN, A_LUQ, A_PLANE, B_PLANE>;
  constexpr int smem = Cfg<A_PLANE, B_PLANE>::smem_bytes;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return static_cast<int>(e);
  return static_cast<int>(luq_launch_kernel(kernel, grid, Cfg<A_PLANE, B_PLANE>::threads, smem, st, LUQ_LAUNCH_EARLY, 1, ta, tb, to, p));
}

template <int KIND, bool A_MN, bool B_MN, bool A_LUQ>
int launch_planes(bool a_plane, bool b_plane, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                  const GemmParams& p, int grid, cudaStream_t st) {
  if (a_plane && b_plane) return launch<KIND, A_MN, B_MN, A_LUQ, true, true>(ta, tb, to, p, grid, st);
  if (a_plane) return launch<KIND, A_MN, B_MN, A_LUQ, true, false>(ta, tb, to, p, grid, st);
  if (b_plane) return launch<KIND, A_MN, B_MN, A_LUQ, false, true>(ta, tb, to, p, grid, st);
  return launch<KIND, A_MN, B_MN, A_LUQ, false, false>(ta, tb, to, p, grid, st);
}

template <int KIND, bool A_MN, bool B_MN>
int launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to, const GemmParams& p, int pairs,
                cudaStream_t st) {
  auto kernel = luq_gemm_pair_kernel<KIND, A_MN, B_MN>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem::smem_bytes);
  if (e != cudaSuccess) return static_cast<int>(e);
  e = luq_launch_kernel(kernel, 2 * pairs, kPairThreads, PairSmem::smem_bytes, st, LUQ_LAUNCH_EARLY, 2, ta, tb, to, p);
  return static_cast<int>(e);
}

template <int KIND>
int launch_expand(bool luq_codes, const uint8_t* codes, uint8_t* plane, size_t packed_bytes, const uint4& lut, int sms,
                  cudaStream_t st) {
  const size_t pieces = packed_bytes / 16;
  size_t blocks = (pieces + 255) / 256;
  const size_t cap = static_cast<size_t>(sms) * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  const uint4* src = reinterpret_cast<const uint4*>(codes);
  uint4* dst = reinterpret_cast<uint4*>(plane);
  const int grid = static_cast<int>(blocks);
  return static_cast<int>(luq_codes ? luq_launch_kernel(expand_plane_kernel<KIND, true>, grid, 256, 0, st, LUQ_LAUNCH_EARLY, 1, src, dst, pieces, lut)
                                    : luq_launch_kernel(expand_plane_kernel<KIND, false>, grid, 256, 0, st, LUQ_LAUNCH_EARLY, 1, src, dst, pieces, lut));
}

// Diagnostic: a bounded wait that is left to run out.  One thread initialises an mbarrier that
// nothing ever arrives on, polls it a fixed number of times, then reports the expiry the way the
// GEMM roles do (status bit, normal return).  The context stays usable.
__global__ void expire_wait_kernel(unsigned int* status, uint32_t polls) {
  __shared__ __align__(8) uint64_t bar;
  pdl_wait();
  pdl_trigger();
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    fence_barrier_init();
    bool arrived = false;
    for (uint32_t i = 0; i < polls && !arrived; ++i) arrived = mbar_test(smem_u32(&bar), 0);
    if (!arrived) atomicOr(status, LUQ_STATUS_TIMEOUT);
  }
}

constexpr size_t kSplitRegionBytes = 20u << 20;   // the first 20 MiB of a workspace hold split partial tiles

}  // namespace

static int luq_launch_gemm_impl(luq_ctx* ctx, const luq_gemm_args& a, cudaStream_t st) {
  GemmParams p{};
  p.scale_a = a.d_scale_a; p.scale_b = a.d_scale_b; p.status = ctx->d_status;
  p.Mo = a.Mo; p.No = a.No; p.Kc = a.Kc;
  // a summed plane (LUQ_OPT_SUM_SAMPLES) is one sample as far as the contraction goes; the division by
  // the sample count and the accumulator's range still follow a.n_samples
  const int ns = a.a_summed > 1 ? 1 : a.n_samples;
  if (a.a_summed > 1 && (a.a_summed != a.n_samples || a.a_kind != 1 || !a.a_operand)) return LUQ_ERR_ARG;
  p.n_samples = ns;
  p.out_bf16 = a.out_bf16;
  if (a.out_bf16 && a.No % 8 != 0) return LUQ_ERR_ARG;   // output rows must stay 16-byte aligned
  p.tiles_m = static_cast<int>((a.Mo + BM - 1) / BM);
  p.tiles_n = static_cast<int>((a.No + BN - 1) / BN);
  p.num_kb = static_cast<int>((a.Kc + BK - 1) / BK);
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
  const int total_iters = p.n_samples * p.num_kb;
  // the SMs this product may occupy (LUQ_OPT_SM_LIMIT): one persistent CTA each
  const int sms = (ctx->sm_limit > 0 && ctx->sm_limit < ctx->sm_count) ? ctx->sm_limit : ctx->sm_count;
  int splits = 1;
  if (a.allow_split) {
    if (ctx->forced_splits > 0) splits = ctx->forced_splits;
    else if (tiles * 2 <= sms) splits = static_cast<int>(sms / tiles);
    if (splits > total_iters / 4 && ctx->forced_splits <= 0) splits = total_iters / 4;
    if (splits > total_iters) splits = total_iters;
    if (splits < 1) splits = 1;
  }
  p.iters_per_split = (total_iters + splits - 1) / splits;
  p.splits = (total_iters + p.iters_per_split - 1) / p.iters_per_split;  // no empty split
  const size_t split_region = a.workspace_bytes < kSplitRegionBytes ? a.workspace_bytes : kSplitRegionBytes;
  if (p.splits > 1) {
    const size_t need = static_cast<size_t>(tiles * p.splits) * kTileFloats * sizeof(float);
    if (a.d_workspace == nullptr || need > split_region) {
      if (ctx->forced_splits > 0) return LUQ_ERR_WORKSPACE;
      p.splits = 1;
      p.iters_per_split = total_iters;
    }
  }
  const long long units = tiles * p.splits;

  // Operand type.  "Automatic" is int8: INT4 codes expand to it in three instructions per eight
  // codes, and it is the type of the operand bytes the quantizers can write themselves.
  // Where an int32 accumulator could wrap (a very long contraction) it is e4m3 with fp32 accumulators.
  auto worst = [](int kind) { return kind == 0 ? 7 * 16 : kind == 2 ? 15 : 64; };   // largest |operand byte|
  const long long worst_product = static_cast<long long>(worst(a.a_kind)) * worst(a.b_kind);
  const bool int32_safe = worst_product * a.Kc * a.n_samples < (1ll << 31);
  if (ctx->mma_kind == 2) ctx->mma_kind = int32_safe ? 1 : 0;
  if (ctx->mma_kind == 1 && !int32_safe) return LUQ_ERR_ARG;
  if (a.a_summed > 1 && ctx->mma_kind != 1) return LUQ_ERR_UNSUPPORTED;   // sums of levels are int8 values, not e4m3
  // Operand planes: an operand that at least two tiles re-read is fetched as bytes.  The caller's
  // bytes (written by the quantizer, int8) are taken as they are; otherwise the codes are expanded
  // once into the workspace behind the split region, if there is room.  A product with a short
  // contraction is bound by its output stream and hides the in-kernel expansion completely
  // (measured: the backward product of the ResNet shape, 2 blocks per tile), so it keeps the codes.
  const size_t a_plane_bytes = static_cast<size_t>(a.Mo) * a.Kc * ns;
  const size_t b_plane_bytes = static_cast<size_t>(a.No) * a.Kc;
  size_t plane_room = (a.d_workspace && a.workspace_bytes > kSplitRegionBytes) ? a.workspace_bytes - kSplitRegionBytes : 0;
  uint8_t* plane_ptr = a.d_workspace ? reinterpret_cast<uint8_t*>(a.d_workspace) + kSplitRegionBytes : nullptr;
  auto packed_ok = [](size_t bytes) { return bytes % 32 == 0; };   // whole 16-byte pieces of packed codes
  const uint8_t* a_given = ctx->mma_kind == 1 ? reinterpret_cast<const uint8_t*>(a.a_operand) : nullptr;
  const uint8_t* b_given = ctx->mma_kind == 1 ? reinterpret_cast<const uint8_t*>(a.b_operand) : nullptr;
  bool b_plane = false, a_plane = false, b_expand = false, a_expand = false;
  const bool long_contraction = total_iters >= 8;
  const uint8_t* b_plane_ptr = nullptr; const uint8_t* a_plane_ptr = nullptr;
  // Unsigned INT4 codes (kind 2) have no expansion inside the GEMM kernels: such an operand is
  // always fetched as bytes, the caller's or a plane expanded here.
  // The same holds for signed INT4 codes as the first operand of the backward / update products
  // (the uniform arm of the gradient ablation): those kernels expand LUQ codes there.
  const bool b_must = a.b_kind == 2, a_must = a.a_kind == 2 || (a.a_kind == 0 && (a.a_mn || a.b_mn)) || a.a_summed > 1;
  // (With bf16 outputs the output stream no longer hides the expansion: the caller's bytes are then
  // used for short contractions too - backward product of the ResNet shape 82 -> 65 us.)
  // A short contraction with fp32 output is bound by its output stream: with both operands' bytes at
  // hand it runs the whole-row epilogue (bare store kernels: 6.0 TB/s in 1 KB rows against 5.4 in boxes).
  const bool rows_epilogue = !a.out_bf16 && a_given && b_given && p.splits == 1 && total_iters <= 4 &&
                             a.No % 32 == 0 && ctx->use_pairs != 1;
  const bool use_given = a.out_bf16 != 0 || rows_epilogue;
  if (b_must || rows_epilogue || ((long_contraction || (use_given && b_given)) && p.tiles_m >= 2)) {
    if (b_given) {
      b_plane = true; b_plane_ptr = b_given;
    } else if (packed_ok(b_plane_bytes) && b_plane_bytes <= plane_room) {
      b_plane = b_expand = true; b_plane_ptr = plane_ptr;
      const size_t used = (b_plane_bytes + 1023) & ~static_cast<size_t>(1023);
      plane_ptr += used; plane_room -= used <= plane_room ? used : plane_room;
    } else if (b_must) {
      return LUQ_ERR_WORKSPACE;
    }
  }
  if (a_must || rows_epilogue || ((long_contraction || (use_given && a_given)) && p.tiles_n >= 2)) {
    if (a_given) {
      a_plane = true; a_plane_ptr = a_given;
    } else if (packed_ok(a_plane_bytes) && a_plane_bytes <= plane_room) {
      a_plane = a_expand = true; a_plane_ptr = plane_ptr;
    } else if (a_must) {
      return LUQ_ERR_WORKSPACE;
    }
  }
  p.lut_a = make_lut(ctx->mma_kind, a.a_kind);
  p.lut_b = make_lut(ctx->mma_kind, a.b_kind);
  // int8 operands carry INT4 integers as 16*q: undo with an exact power of two
  float pow2 = 1.0f;
  if (ctx->mma_kind == 1) {
    if (a.a_kind == 0) pow2 *= 1.0f / 16.0f;
    if (a.b_kind == 0) pow2 *= 1.0f / 16.0f;
  }
  p.post_scale = (1.0f / static_cast<float>(a.n_samples)) * pow2;

  int rc = 0;
  if (b_expand) {
    uint8_t* dst = const_cast<uint8_t*>(b_plane_ptr);   // workspace memory
    rc = ctx->mma_kind ? launch_expand<1>(a.b_kind != 0, a.b_codes, dst, b_plane_bytes / 2, p.lut_b, ctx->sm_count, st)
                       : launch_expand<0>(a.b_kind != 0, a.b_codes, dst, b_plane_bytes / 2, p.lut_b, ctx->sm_count, st);
    if (rc != 0) return rc;
    ctx->launches += 1;
  }
  if (a_expand) {
    uint8_t* dst = const_cast<uint8_t*>(a_plane_ptr);   // workspace memory
    rc = ctx->mma_kind ? launch_expand<1>(a.a_kind != 0, a.a_codes, dst, a_plane_bytes / 2, p.lut_a, ctx->sm_count, st)
                       : launch_expand<0>(a.a_kind != 0, a.a_codes, dst, a_plane_bytes / 2, p.lut_a, ctx->sm_count, st);
    if (rc != 0) return rc;
    ctx->launches += 1;
  }

  CUtensorMap ta, tb, to;
  int bad = 0;
  {
    const uint8_t* ptr = a_plane ? a_plane_ptr : a.a_codes;
    const uint64_t div = a_plane ? 1 : 2;   // bytes per row: elements (plane) or elements / 2 (codes)
    if (a.a_mn) bad |= encode_bytes_map(ctx->encode_tiled, &ta, ptr, a.Mo / div, a.Kc, ns, true, a_plane);
    else bad |= encode_bytes_map(ctx->encode_tiled, &ta, ptr, a.Kc / div, a.Mo, ns, true, a_plane);
  }
  {
    const uint8_t* ptr = b_plane ? b_plane_ptr : a.b_codes;
    const uint64_t div = b_plane ? 1 : 2;
    if (a.b_mn) bad |= encode_bytes_map(ctx->encode_tiled, &tb, ptr, a.No / div, a.Kc, 1, false, b_plane);
    else bad |= encode_bytes_map(ctx->encode_tiled, &tb, ptr, a.Kc / div, a.No, 1, false, b_plane);
  }
  if (p.splits > 1) bad |= encode_out_map(ctx->encode_tiled, &to, a.d_workspace, units * BM, BN, false);
  else if (rows_epilogue) bad |= encode_out_rows_map(ctx->encode_tiled, &to, a.d_out, a.Mo, a.No);
  else bad |= encode_out_map(ctx->encode_tiled, &to, a.d_out, a.Mo, a.No, a.out_bf16 != 0);
  if (bad) return LUQ_ERR_CUDA;

  // CTA pairs need both operands as planes (no expansion inside the kernel) and an unsplit contraction
  // CTA pairs: forced (1), or chosen here (2, the default) for the products they were measured faster on -
  // a long contraction with B stored contraction-major (backward and update products of a wide layer:
  // 35.2 -> 31.5 us and 33.1 -> 30.6 us on the Transformer shape; the forward product is 4 % slower on pairs)
  const bool pairs_wanted = ctx->use_pairs == 1 || (ctx->use_pairs == 2 && a.b_mn && total_iters >= 8);
  if (pairs_wanted && !rows_epilogue && a_plane && b_plane && p.splits == 1 && p.tiles_m >= 2 && !a.out_bf16) {
    const long long pair_tiles = static_cast<long long>((p.tiles_m + 1) / 2) * p.tiles_n;
    const int max_pairs = sms / 2 > 0 ? sms / 2 : 1;
    const int pairs = static_cast<int>(pair_tiles < max_pairs ? pair_tiles : max_pairs);
    const int sel2 = (ctx->mma_kind ? 4 : 0) | (a.a_mn ? 2 : 0) | (a.b_mn ? 1 : 0);
    switch (sel2) {
      case 0: rc = launch_pair<0, false, false>(ta, tb, to, p, pairs, st); break;
      case 1: rc = launch_pair<0, false, true>(ta, tb, to, p, pairs, st); break;
      case 3: rc = launch_pair<0, true, true>(ta, tb, to, p, pairs, st); break;
      case 4: rc = launch_pair<1, false, false>(ta, tb, to, p, pairs, st); break;
      case 5: rc = launch_pair<1, false, true>(ta, tb, to, p, pairs, st); break;
      case 7: rc = launch_pair<1, true, true>(ta, tb, to, p, pairs, st); break;
      default: return LUQ_ERR_UNSUPPORTED;
    }
    if (rc == 0) ctx->launches += 1;
    return rc;
  }

  const int grid = static_cast<int>(units < sms ? units : sms);
  const int sel = (ctx->mma_kind ? 4 : 0) | (a.a_mn ? 2 : 0) | (a.b_mn ? 1 : 0);
  // the kernels expand signed INT4 codes in B, and in A signed INT4 (forward) or LUQ codes (backward,
  // update); any other kind of operand must have arrived as bytes
  if ((a.b_kind != 0 && !b_plane) || (!a_plane && (a.a_kind == 1) != (sel & 3 ? true : false)) ||
      (a.a_kind == 2 && !a_plane))
    return LUQ_ERR_UNSUPPORTED;
  if (rows_epilogue) {
    switch (sel) {
      case 0: rc = launch_rows<0, false, false, false>(ta, tb, to, p, grid, st); break;
      case 1: rc = launch_rows<0, false, true, true>(ta, tb, to, p, grid, st); break;
      case 3: rc = launch_rows<0, true, true, true>(ta, tb, to, p, grid, st); break;
      case 4: rc = launch_rows<1, false, false, false>(ta, tb, to, p, grid, st); break;
      case 5: rc = launch_rows<1, false, true, true>(ta, tb, to, p, grid, st); break;
      case 7: rc = launch_rows<1, true, true, true>(ta, tb, to, p, grid, st); break;
      default: return LUQ_ERR_UNSUPPORTED;
    }
    if (rc == 0) ctx->launches += 1;
    return rc;
  }
  switch (sel) {
    case 0: rc = launch_planes<0, false, false, false>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    case 1: rc = launch_planes<0, false, true, true>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    case 3: rc = launch_planes<0, true, true, true>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    case 4: rc = launch_planes<1, false, false, false>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    case 5: rc = launch_planes<1, false, true, true>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    case 7: rc = launch_planes<1, true, true, true>(a_plane, b_plane, ta, tb, to, p, grid, st); break;
    default: return LUQ_ERR_UNSUPPORTED;
  }
  if (rc != 0) return rc;
  ctx->launches += 1;
  if (p.splits > 1) {
    const long long work = tiles * (kTileFloats / 4);
    rc = static_cast<int>(luq_launch_kernel(split_reduce_kernel, static_cast<int>((work + 255) / 256), 256, 0, st, LUQ_LAUNCH_EARLY, 1,
                                            a.d_workspace, a.d_out, a.d_scale_a, a.d_scale_b, p.post_scale,
                                            static_cast<int>(tiles), p.tiles_m, p.splits, a.Mo, a.No, a.out_bf16));
    if (rc == 0) ctx->launches += 1;
  }
  return rc;
}

// ---------------------------------------------------------------------------
// Forward product that quantizes its activations on the way in (luq_quant_int4_gemm_fwd).
// ---------------------------------------------------------------------------
namespace {

// high-precision activations [rows x cols]: box of 128 rows x 32 elements, swizzled like the box's row width
int encode_raw_map(void* fn, CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, bool bf16) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * (bf16 ? 2 : 4)};
  const cuuint32_t box[2] = {32, 128};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims,
      strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}
// packed codes [rows x cols/2 bytes] as the destination of 128-row x 32-byte boxes (32-byte swizzle in shared memory)
int encode_codes_store_map(void* fn, CUtensorMap* map, uint8_t* ptr, uint64_t rows, uint64_t pitch) {
  const cuuint64_t dims[2] = {pitch, rows};
  const cuuint64_t strides[1] = {pitch};
  const cuuint32_t box[2] = {32, 128};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

}  // namespace

// The fused kernel serves one column of output tiles with int8 operands and an fp32 output.
bool luq_quant_fwd_fusable(const luq_ctx* ctx, int64_t M, int64_t N, int64_t K, bool have_w_bytes) {
  if (M <= 0 || N <= 0 || K <= 0 || N > BN) return false;
  if (ctx->mma_kind == 0 || ctx->out_bf16 || ctx->unsigned_act) return false;
  if (112ll * 112ll * K >= (1ll << 31)) return false;                       // int32 accumulator
  if (!have_w_bytes) {
    const size_t bytes = static_cast<size_t>(N) * K;
    if (bytes % 32 != 0 || ctx->d_workspace == nullptr || ctx->workspace_bytes < kSplitRegionBytes + bytes) return false;
  }
  return true;
}

int luq_launch_quant_fwd(luq_ctx* ctx, const void* d_a, int dtype, const float* d_clip, uint8_t* d_a_codes,
                         float* d_sa, const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                         float* d_z, int64_t M, int64_t N, int64_t K, cudaStream_t st, float* d_estimate, float eta,
                         float* d_measured) {
  const bool bf16 = dtype == LUQ_BF16;
  const uint8_t* w_plane = reinterpret_cast<const uint8_t*>(d_w_operand);
  if (w_plane == nullptr) {   // widen W's codes once into the workspace (behind the split region)
    uint8_t* dst = reinterpret_cast<uint8_t*>(ctx->d_workspace) + kSplitRegionBytes;
    const int rc = launch_expand<1>(false, d_w_codes, dst, static_cast<size_t>(N) * K / 2, make_lut(1, 0), ctx->sm_count, st);
    if (rc != 0) return rc;
    ctx->launches += 1;
    w_plane = dst;
  }
  FusedParams p{};
  p.clip = d_estimate ? d_estimate : d_clip; p.scale_b = d_sw; p.scale_a_out = d_sa; p.status = ctx->d_status;
  p.estimate = d_estimate; p.measured = reinterpret_cast<unsigned int*>(d_measured); p.scratch = ctx->d_scratch; p.eta = eta;
  p.Mo = M; p.No = N; p.Kc = K;
  p.tiles_m = static_cast<int>((M + BM - 1) / BM);
  p.num_kb = static_cast<int>((K + BK - 1) / BK);
  CUtensorMap t_raw, t_b, t_codes, t_out;
  int bad = encode_raw_map(ctx->encode_tiled, &t_raw, d_a, M, K, bf16);
  bad |= encode_bytes_map(ctx->encode_tiled, &t_b, w_plane, K, N, 1, false, true);
  bad |= encode_codes_store_map(ctx->encode_tiled, &t_codes, d_a_codes, M, K / 2);
  bad |= encode_out_map(ctx->encode_tiled, &t_out, d_z, M, N, false);
  if (bad) return LUQ_ERR_CUDA;
  const int sms = (ctx->sm_limit > 0 && ctx->sm_limit < ctx->sm_count) ? ctx->sm_limit : ctx->sm_count;
  // As many CTAs as make whole rounds of tiles (392 tiles: 131 CTAs in three full rounds rather than 148 in
  // two and a round of 96): the last, partly filled round would run at what single SMs can pull, not at
  // what the memory system gives (107 -> 105 us on the ResNet shape).
  const int rounds = (p.tiles_m + sms - 1) / sms;
  const int grid = (p.tiles_m + rounds - 1) / rounds;
  cudaError_t e;
  if (bf16) {
    auto kernel = luq_quant_fwd_kernel<true>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedCfg<true>::smem_bytes);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = luq_launch_kernel(kernel, grid, FusedCfg<true>::threads, FusedCfg<true>::smem_bytes, st, LUQ_LAUNCH_EARLY, 1,
                          t_raw, t_b, t_codes, t_out, p);
  } else {
    auto kernel = luq_quant_fwd_kernel<false>;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedCfg<false>::smem_bytes);
    if (e != cudaSuccess) return static_cast<int>(e);
    e = luq_launch_kernel(kernel, grid, FusedCfg<false>::threads, FusedCfg<false>::smem_bytes, st, LUQ_LAUNCH_EARLY, 1,
                          t_raw, t_b, t_codes, t_out, p);
  }
  if (e == cudaSuccess) ctx->launches += 1;
  return static_cast<int>(e);
}

namespace {
// Diagnostic for the checking build: forms an address one byte beyond a 64-byte shared-memory region and
// asks the check about it.  Nothing is accessed.  With -DLUQ_DEBUG the check raises LUQ_STATUS_BOUNDS;
// in the normal build the check is compiled out and nothing happens.
__global__ void bounds_probe_kernel(unsigned int* status) {
  __shared__ __align__(16) uint8_t region[64];
  pdl_wait();
  pdl_trigger();
  if (threadIdx.x == 0) {
    const bool inside = smem_in(region + 16, region, 0, 64, 16, status);
    const bool beyond = smem_in(region + 49, region, 0, 64, 16, status);
    (void)inside; (void)beyond;
  }
}
}  // namespace

int luq_launch_bounds_probe(luq_ctx* ctx, cudaStream_t st) {
  const cudaError_t e = luq_launch_kernel(bounds_probe_kernel, 1, 32, 0, st, LUQ_LAUNCH_EARLY, 1, ctx->d_status);
  ctx->launches += 1;
  return static_cast<int>(e);
}

int luq_launch_expire_wait(luq_ctx* ctx, cudaStream_t st) {
  const cudaError_t e = luq_launch_kernel(expire_wait_kernel, 1, 32, 0, st, LUQ_LAUNCH_EARLY, 1, ctx->d_status, 1u << 16);
  ctx->launches += 1;
  return static_cast<int>(e);
}

int luq_launch_gemm(luq_ctx* ctx_in, const luq_gemm_args& a, cudaStream_t st) {
  if (a.Mo <= 0 || a.No <= 0) return 0;
  if (a.Kc <= 0) {  // an empty contraction (an empty batch in the update product): the sum is zero everywhere
    if (a.d_out == nullptr) return LUQ_ERR_ARG;
    return static_cast<int>(cudaMemsetAsync(a.d_out, 0, static_cast<size_t>(a.Mo) * a.No * (a.out_bf16 ? 2 : 4), st));
  }
  luq_ctx ctx_copy = *ctx_in;            // the operand type may be chosen per product below
  luq_ctx* ctx = &ctx_copy;
  const int rc_all = luq_launch_gemm_impl(ctx, a, st);
  ctx_in->launches = ctx->launches;
  return rc_all;
}


// ---------------------------------------------------------------------------
// Update GEMM for callers that must not allocate device memory.
//
// The split partial tiles normally live in the context's workspace, which
// luq_create obtains with cudaMalloc.  Here they live in a fixed array that is
// part of the library image: it exists on every GPU that loads the library, from
// load until the process ends, and is shared by every call of this entry point.
// ---------------------------------------------------------------------------
namespace {

constexpr int kStaticTiles = 152;                                  // partial tiles the array holds
constexpr size_t kStaticScratchBytes = static_cast<size_t>(kStaticTiles) * kTileFloats * sizeof(float);  // 19 MiB
constexpr int kMaxDevices = 64;

static __device__ __align__(256) float g_static_scratch[static_cast<size_t>(kStaticTiles) * kTileFloats];
static __device__ unsigned int g_static_status;

struct StaticSetup {
  bool ready = false;
  float* scratch = nullptr;        // device address of g_static_scratch on this device
  unsigned int* status = nullptr;  // device address of g_static_status on this device
  void* encode_tiled = nullptr;
  int sm_count = 0;
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current.  In host code the names of the two
// arrays are only handles: the addresses a kernel may use come from
// cudaGetSymbolAddress.
int static_setup(int device, StaticSetup** out) {
  if (device < 0 || device >= kMaxDevices) return LUQ_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSetup& s = g_static_setup[device];
  if (!s.ready) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return LUQ_ERR_CUDA;
    if (prop.major != 10) return LUQ_ERR_UNSUPPORTED;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return LUQ_ERR_CUDA;
    s.scratch = static_cast<float*>(p);
    p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_status) != cudaSuccess || p == nullptr) return LUQ_ERR_CUDA;
    s.status = static_cast<unsigned int*>(p);
    if (cudaMemset(s.status, 0, sizeof(unsigned int)) != cudaSuccess) return LUQ_ERR_CUDA;  // must start at zero
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &s.encode_tiled, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || s.encode_tiled == nullptr)
      return LUQ_ERR_CUDA;
    s.sm_count = prop.multiProcessorCount;
    s.ready = true;
  }
  *out = &s;
  return LUQ_OK;
}

}  // namespace

extern "C" int luq_gemm_wgrad_static(const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                                     const uint8_t* d_a_codes, const float* d_sa, float* d_dw,
                                     int64_t M, int64_t N, int64_t K, void* stream) {
  if (!d_alpha || !d_sa) return LUQ_ERR_ARG;
  if (M < 0 || N < 0 || K < 0 || M > (1ll << 31) || N > (1ll << 31) || K > (1ll << 31)) return LUQ_ERR_ARG;
  if (n_samples < 1 || n_samples > LUQ_MAX_SAMPLES) return LUQ_ERR_ARG;
  if (M && N && K && (!d_g_codes || !d_a_codes || !d_dw)) return LUQ_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(d_g_codes) | reinterpret_cast<uintptr_t>(d_a_codes) |
       reinterpret_cast<uintptr_t>(d_dw)) & 15u)
    return LUQ_ERR_ARG;
  if (N % 32 || K % 32) return LUQ_ERR_ARG;
  const long long tiles = ((N + BM - 1) / BM) * ((K + BN - 1) / BN);
  if (tiles > kStaticTiles) return LUQ_ERR_WORKSPACE;   // output larger than the fixed scratch serves

  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return LUQ_ERR_CUDA;
  StaticSetup* s = nullptr;
  int rc = static_setup(device, &s);
  if (rc != LUQ_OK) return rc;

  luq_ctx local{};               // a context on the stack: nothing in it is allocated
  local.device = device;
  local.sm_count = s->sm_count;
  local.d_status = s->status;
  local.d_workspace = s->scratch;
  local.workspace_bytes = kStaticScratchBytes;
  local.mma_kind = LUQ_DEFAULT_MMA_KIND;
  local.forced_splits = 0;
  local.use_pairs = 2;
  local.sm_limit = 0;
  local.grad_int4 = 0;
  local.kmax = LUQ_KMAX;
  local.unsigned_act = 0;
  local.out_bf16 = 0;
  local.launches = 0;
  local.encode_tiled = s->encode_tiled;

  luq_gemm_args a{};
  a.a_codes = d_g_codes; a.a_kind = 1; a.a_mn = 1; a.n_samples = n_samples;
  a.b_codes = d_a_codes; a.b_kind = 0; a.b_mn = 1;
  a.d_scale_a = d_alpha; a.d_scale_b = d_sa; a.d_out = d_dw; a.Mo = N; a.No = K; a.Kc = M;
  a.d_workspace = s->scratch; a.workspace_bytes = kStaticScratchBytes;
  a.allow_split = 1;
  rc = luq_launch_gemm(&local, a, reinterpret_cast<cudaStream_t>(stream));
  return rc == 0 ? LUQ_OK : (rc < 0 ? rc : LUQ_ERR_CUDA);
}
