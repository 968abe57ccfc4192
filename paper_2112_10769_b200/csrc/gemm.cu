// 4-bit training GEMMs on tcgen05 / tensor memory (sm_100a).
//
//   D[Mo x No] = scale * sum_s sum_k opA_s[mo, k] * opB[no, k]
//
// serves the three products of the path (forward, backward, update); the
// operands are packed 4-bit codes in global memory, stored either k-contiguous
// ("K-major": rows are mo / no) or contraction-major ("MN-major": rows are k).
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: packed 128-row x 64-byte slabs -> shared memory ring
//   warps 6-13  converters: nibble -> 8-bit operand (16-entry byte table through
//               PRMT), written in the 128-byte-swizzled layout the tensor core reads
//   warp 1      one thread issues tcgen05.mma (128 x 256 x 32 per instruction),
//               accumulators live in tensor memory, two buffers of 256 columns
//   warps 2-5   epilogue: tcgen05.ld -> scale -> global store (or split reduction)
// Every slab, in either orientation, is 128 rows x 64 packed bytes and expands to
// 128 rows x 128 bytes; only the matrix descriptor differs between orientations.
// All waits are bounded; on expiry the CTA flags LUQ_STATUS_TIMEOUT, drains its
// copies, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"

namespace {

using namespace luqdev;

constexpr int BM = 128;            // output rows per tile (tensor-memory lanes)
constexpr int BN = 256;            // output columns per tile
constexpr int BK = 128;            // contraction elements per pipeline stage
constexpr int kSlabRows = 128;
constexpr int kPackedSlab = kSlabRows * 64;      // bytes
constexpr int kExpandedSlab = kSlabRows * 128;   // bytes
constexpr int kSlabs = 1 + BN / 128;             // A, B0, B1
constexpr int kPackedStage = kSlabs * kPackedSlab;
constexpr int kExpandedStage = kSlabs * kExpandedSlab;
constexpr int kPackedStages = 4;
constexpr int kExpandedStages = 2;
constexpr int kConvWarps = 8;
constexpr int kFirstEpiWarp = 2;
constexpr int kFirstConvWarp = 6;
constexpr int kThreads = 32 * (kFirstConvWarp + kConvWarps);
constexpr int kTmemCols = 2 * BN;
constexpr int kTileFloats = BM * BN;

struct SmemLayout {
  static constexpr int expanded = 0;
  static constexpr int packed = expanded + kExpandedStages * kExpandedStage;
  static constexpr int barriers = packed + kPackedStages * kPackedStage;
  // barrier order: pk_full[PS] pk_empty[PS] ex_full[ES] ex_empty[ES] acc_full[2] acc_empty[2]
  static constexpr int num_barriers = 2 * kPackedStages + 2 * kExpandedStages + 4;
  static constexpr int tmem_slot = barriers + 8 * num_barriers;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int last_flag = abort_flag + 4;
  static constexpr int total = last_flag + 4;
};
constexpr int kSmemBytes = SmemLayout::total + 1024;  // slack to align the base to 1024 bytes

struct GemmParams {
  const float* scale_a;
  const float* scale_b;
  float* out;
  float* workspace;
  unsigned int* tickets;
  unsigned int* status;
  long long Mo, No, Kc;
  int n_samples;
  int tiles_m, tiles_n;
  int num_kb;          // contraction blocks per sample plane
  int splits;          // contraction splits per tile
  int iters_per_split;
  float inv_samples;
  uint4 lut_a, lut_b;  // nibble -> operand byte
};

// eight nibbles of `w` -> eight operand bytes
__device__ __forceinline__ void expand8(uint32_t w, const uint4& lut, uint32_t& lo, uint32_t& hi) {
  const uint32_t sel0 = w & 0x7777u;
  const uint32_t sel1 = (w >> 16) & 0x7777u;
  const uint32_t pick0 = 0x3210u | ((w >> 1) & 0x4444u);
  const uint32_t pick1 = 0x3210u | ((w >> 17) & 0x4444u);
  lo = __byte_perm(__byte_perm(lut.x, lut.y, sel0), __byte_perm(lut.z, lut.w, sel0), pick0);
  hi = __byte_perm(__byte_perm(lut.x, lut.y, sel1), __byte_perm(lut.z, lut.w, sel1), pick1);
}

template <int KIND, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
luq_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* const gen = smem_raw + (base - raw);

  const uint32_t bar0 = base + SmemLayout::barriers;
  auto pk_full = [&](int s) { return bar0 + 8u * s; };
  auto pk_empty = [&](int s) { return bar0 + 8u * (kPackedStages + s); };
  auto ex_full = [&](int s) { return bar0 + 8u * (2 * kPackedStages + s); };
  auto ex_empty = [&](int s) { return bar0 + 8u * (2 * kPackedStages + kExpandedStages + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kPackedStages + 2 * kExpandedStages + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kPackedStages + 2 * kExpandedStages + 2 + b); };
  volatile uint32_t* const tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + SmemLayout::tmem_slot);
  volatile uint32_t* const abort_flag = reinterpret_cast<volatile uint32_t*>(gen + SmemLayout::abort_flag);
  volatile uint32_t* const last_flag = reinterpret_cast<volatile uint32_t*>(gen + SmemLayout::last_flag);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPackedStages; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), kConvWarps); }
    for (int s = 0; s < kExpandedStages; ++s) { mbar_init(ex_full(s), kConvWarps); mbar_init(ex_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), 4); }
    *abort_flag = 0;
    *last_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tm_a); tma_prefetch_desc(&tm_b); }
  if (warp == 1) {  // this warp owns the tensor-memory allocation
    tmem_alloc(base + SmemLayout::tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int units = p.tiles_m * p.tiles_n * p.splits;
  const int total_iters = p.n_samples * p.num_kb;

  auto unit_range = [&](int u, int& tile, int& it_begin, int& it_end) {
    tile = u / p.splits;
    const int sp = u - tile * p.splits;
    it_begin = sp * p.iters_per_split;
    it_end = min(total_iters, it_begin + p.iters_per_split);
  };

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < units; u += gridDim.x) {
        int tile, it_begin, it_end;
        unit_range(u, tile, it_begin, it_end);
        const int m0 = (tile % p.tiles_m) * BM;
        const int n0 = (tile / p.tiles_m) * BN;
        for (int k_it = it_begin; k_it < it_end; ++k_it, ++it) {
          const int s = it % kPackedStages;
          const uint32_t ph = (it / kPackedStages) & 1u;
          if (!mbar_wait(pk_empty(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const int sample = k_it / p.num_kb;
          const int kb = k_it - sample * p.num_kb;
          const uint32_t dst = base + SmemLayout::packed + s * kPackedStage;
          mbar_arrive_expect_tx(pk_full(s), kPackedStage);
          if constexpr (A_MN) tma_load_3d(dst, &tm_a, pk_full(s), m0 / 2, kb * BK, sample);
          else tma_load_3d(dst, &tm_a, pk_full(s), kb * (BK / 2), m0, sample);
#pragma unroll
          for (int j = 0; j < BN / 128; ++j) {
            if constexpr (B_MN) tma_load_2d(dst + (1 + j) * kPackedSlab, &tm_b, pk_full(s), n0 / 2 + 64 * j, kb * BK);
            else tma_load_2d(dst + (1 + j) * kPackedSlab, &tm_b, pk_full(s), kb * (BK / 2), n0 + 128 * j);
          }
        }
      }
      // drain: every copy this thread issued must have landed before the CTA may exit
      const uint32_t issued = it;
      for (int s = 0; s < kPackedStages; ++s) {
        if (issued > static_cast<uint32_t>(s)) {
          const uint32_t last = ((issued - 1 - s) / kPackedStages);  // last fill index of stage s
          mbar_wait(pk_full(s), last & 1u, abort_flag);
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
      uint32_t it = 0, tile_it = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < units; u += gridDim.x, ++tile_it) {
        int tile, it_begin, it_end;
        unit_range(u, tile, it_begin, it_end);
        const uint32_t buf = tile_it & 1u;
        if (!mbar_wait(acc_empty(buf), ((tile_it >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        for (int k_it = it_begin; k_it < it_end; ++k_it, ++it) {
          const int s = it % kExpandedStages;
          if (!mbar_wait(ex_full(s), (it / kExpandedStages) & 1u, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_base = base + SmemLayout::expanded + s * kExpandedStage;
          const uint32_t b_base = a_base + kExpandedSlab;
#pragma unroll
          for (int kk = 0; kk < BK / 32; ++kk) {
            const uint64_t da = A_MN ? umma_desc_sw128(a_base + kk * 32 * 128, kExpandedSlab, 1024)
                                     : umma_desc_sw128(a_base + kk * 32, 16, 1024);
            const uint64_t db = B_MN ? umma_desc_sw128(b_base + kk * 32 * 128, kExpandedSlab, 1024)
                                     : umma_desc_sw128(b_base + kk * 32, 16, 1024);
            tc_mma<KIND>(tmem_d, da, db, idesc, (k_it > it_begin || kk > 0) ? 1u : 0u);
          }
          tc_commit(ex_empty(s));
        }
        if (ok) tc_commit(acc_full(buf));
      }
    }
  } else if (warp < kFirstConvWarp) {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;  // tensor-memory lanes this warp may read
    const int row_in_tile = quarter * 32 + lane;
    const float scale = (__ldg(p.scale_a) * __ldg(p.scale_b)) * p.inv_samples;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int u = blockIdx.x; ok && u < units; u += gridDim.x, ++tile_it) {
      int tile, it_begin, it_end;
      unit_range(u, tile, it_begin, it_end);
      const long long m0 = static_cast<long long>(tile % p.tiles_m) * BM;
      const long long n0 = static_cast<long long>(tile / p.tiles_m) * BN;
      const uint32_t buf = tile_it & 1u;
      const long long row = m0 + row_in_tile;
      float* const ws_row = p.workspace + static_cast<size_t>(tile) * kTileFloats + row_in_tile * BN;
      // a warp whose wait expired still takes part in the block barriers below
      const bool have = mbar_wait(acc_full(buf), (tile_it >> 1) & 1u, abort_flag);
      if (have) {
        tc_fence_after();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * BN;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32(taddr + c * 32, r);
          tmem_ld_wait();
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j)
            v[j] = KIND == 0 ? __uint_as_float(r[j]) : static_cast<float>(static_cast<int>(r[j]));
          const long long col = n0 + c * 32;
          if (p.splits == 1) {
            if (row < p.Mo && col < p.No) {
              float4* dst = reinterpret_cast<float4*>(p.out + row * p.No + col);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                dst[j] = make_float4(v[4 * j] * scale, v[4 * j + 1] * scale, v[4 * j + 2] * scale, v[4 * j + 3] * scale);
            }
          } else {
            // partial sums are integers below 2^24: float atomics add them exactly in any order
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              if (v[4 * j] != 0.0f || v[4 * j + 1] != 0.0f || v[4 * j + 2] != 0.0f || v[4 * j + 3] != 0.0f)
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(ws_row + c * 32 + 4 * j),
                             "f"(v[4 * j]), "f"(v[4 * j + 1]), "f"(v[4 * j + 2]), "f"(v[4 * j + 3]) : "memory");
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(buf));
      }

      if (p.splits > 1) {
        // the last CTA to finish a tile scales the sums and writes the result
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp == kFirstEpiWarp && lane == 0) {
          const unsigned int prev = atomicAdd(p.tickets + tile, 1u);
          *last_flag = (prev == static_cast<unsigned int>(p.splits - 1)) ? 1u : 0u;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const bool last = *last_flag != 0;
        const bool aborted = *abort_flag != 0;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (last) {
          __threadfence();
          for (int c = 0; c < BN / 4; ++c) {
            float4 v = __ldcg(reinterpret_cast<const float4*>(ws_row) + c);
            __stcg(reinterpret_cast<float4*>(ws_row) + c, make_float4(0.f, 0.f, 0.f, 0.f));
            const long long col = n0 + c * 4;
            if (row < p.Mo && col < p.No) {
              v.x *= scale; v.y *= scale; v.z *= scale; v.w *= scale;
              *reinterpret_cast<float4*>(p.out + row * p.No + col) = v;
            }
          }
          if (warp == kFirstEpiWarp && lane == 0) p.tickets[tile] = 0u;
        }
        if (aborted) ok = false;
      } else if (!have) {
        ok = false;
      }
    }
  } else {
    // -------------------------------------------------------------- converters
    const int ctid = threadIdx.x - kFirstConvWarp * 32;
    uint32_t it = 0;
    bool ok = true;
    for (int u = blockIdx.x; ok && u < units; u += gridDim.x) {
      int tile, it_begin, it_end;
      unit_range(u, tile, it_begin, it_end);
      for (int k_it = it_begin; k_it < it_end; ++k_it, ++it) {
        const int ps = it % kPackedStages;
        const int es = it % kExpandedStages;
        if (!mbar_wait(pk_full(ps), (it / kPackedStages) & 1u, abort_flag)) { ok = false; break; }
        if (!mbar_wait(ex_empty(es), ((it / kExpandedStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        const uint8_t* src = gen + SmemLayout::packed + ps * kPackedStage;
        uint8_t* dst = gen + SmemLayout::expanded + es * kExpandedStage;
#pragma unroll
        for (int j = 0; j < kSlabs * 512 / (kConvWarps * 32); ++j) {
          const int id = ctid + j * (kConvWarps * 32);
          const int slab = id >> 9;
          const int idx = id & 511;
          const int row = idx >> 2;
          const int q = idx & 3;
          const uint4 w = *reinterpret_cast<const uint4*>(src + slab * kPackedSlab + idx * 16);
          const uint4 lut = slab == 0 ? p.lut_a : p.lut_b;
          uint4 o0, o1;
          expand8(w.x, lut, o0.x, o0.y);
          expand8(w.y, lut, o0.z, o0.w);
          expand8(w.z, lut, o1.x, o1.y);
          expand8(w.w, lut, o1.z, o1.w);
          uint8_t* drow = dst + slab * kExpandedSlab + row * 128;
          const int sw = row & 7;
          *reinterpret_cast<uint4*>(drow + (((2 * q) ^ sw) << 4)) = o0;
          *reinterpret_cast<uint4*>(drow + (((2 * q + 1) ^ sw) << 4)) = o1;
        }
        fence_proxy_async();   // make the generic-proxy writes visible to the tensor core
        __syncwarp();
        if (lane == 0) { mbar_arrive(pk_empty(ps)); mbar_arrive(ex_full(es)); }
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

// nibble -> operand byte tables.  kind 0: e4m3 (sign, 4-bit exponent bias 7, 3-bit
// mantissa); kind 1: two's-complement int8.  Every INT4 integer and every LUQ
// level 2^0..2^6 is exact in both.
uint8_t e4m3_of_int(int v) {
  static const uint8_t mag[9] = {0x00, 0x38, 0x40, 0x44, 0x48, 0x4A, 0x4C, 0x4E, 0x50};
  const int a = v < 0 ? -v : v;
  return static_cast<uint8_t>(mag[a] | (v < 0 ? 0x80 : 0));
}
uint4 make_lut(int mma_kind, int operand_kind) {
  uint8_t t[16];
  for (int n = 0; n < 16; ++n) {
    if (operand_kind == 0) {               // INT4 two's complement
      const int v = n < 8 ? n : n - 16;
      t[n] = mma_kind == 0 ? e4m3_of_int(v) : static_cast<uint8_t>(static_cast<int8_t>(v));
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

// packed-code tensor: `planes` x `rows` x `pitch` bytes, box = 1 x 128 rows x 64 bytes
int encode_map(void* fn, CUtensorMap* map, const uint8_t* ptr, uint64_t pitch, uint64_t rows, uint64_t planes,
               bool three_d) {
  const cuuint64_t dims[3] = {pitch, rows, planes};
  const cuuint64_t strides[2] = {pitch, pitch * rows};
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      map, CU_TENSOR_MAP_DATA_TYPE_UINT8, three_d ? 3 : 2, const_cast<uint8_t*>(ptr), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? 0 : 1;
}

template <int KIND, bool A_MN, bool B_MN>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, int grid, cudaStream_t st) {
  auto kernel = luq_gemm_kernel<KIND, A_MN, B_MN>;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return static_cast<int>(e);
  kernel<<<grid, kThreads, kSmemBytes, st>>>(ta, tb, p);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace

int luq_launch_gemm(luq_ctx* ctx, const luq_gemm_args& a, cudaStream_t st) {
  if (a.Mo <= 0 || a.No <= 0 || a.Kc <= 0) return 0;
  GemmParams p{};
  p.scale_a = a.d_scale_a; p.scale_b = a.d_scale_b; p.out = a.d_out;
  p.workspace = a.d_workspace; p.tickets = a.d_tickets; p.status = ctx->d_status;
  p.Mo = a.Mo; p.No = a.No; p.Kc = a.Kc;
  p.n_samples = a.n_samples;
  p.tiles_m = static_cast<int>((a.Mo + BM - 1) / BM);
  p.tiles_n = static_cast<int>((a.No + BN - 1) / BN);
  p.num_kb = static_cast<int>((a.Kc + BK - 1) / BK);
  p.inv_samples = 1.0f / static_cast<float>(a.n_samples);
  p.lut_a = make_lut(ctx->mma_kind, a.a_kind);
  p.lut_b = make_lut(ctx->mma_kind, a.b_kind);

  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n;
  const int total_iters = p.n_samples * p.num_kb;
  int splits = 1;
  if (a.allow_split) {
    if (ctx->forced_splits > 0) splits = ctx->forced_splits;
    else if (tiles * 2 <= ctx->sm_count) splits = static_cast<int>(ctx->sm_count / tiles);
    if (splits > total_iters / 4 && ctx->forced_splits <= 0) splits = total_iters / 4;
    if (splits > total_iters) splits = total_iters;
    if (splits < 1) splits = 1;
  }
  if (splits > 1) {
    const size_t need = static_cast<size_t>(tiles) * kTileFloats * sizeof(float);
    if (a.d_workspace == nullptr || need > a.workspace_bytes || tiles > a.max_tickets) {
      if (ctx->forced_splits > 0) return LUQ_ERR_WORKSPACE;
      splits = 1;
    }
  }
  p.iters_per_split = (total_iters + splits - 1) / splits;
  p.splits = (total_iters + p.iters_per_split - 1) / p.iters_per_split;  // no empty split

  CUtensorMap ta, tb;
  int bad = 0;
  if (a.a_mn) bad |= encode_map(ctx->encode_tiled, &ta, a.a_codes, a.Mo / 2, a.Kc, a.n_samples, true);
  else bad |= encode_map(ctx->encode_tiled, &ta, a.a_codes, a.Kc / 2, a.Mo, a.n_samples, true);
  if (a.b_mn) bad |= encode_map(ctx->encode_tiled, &tb, a.b_codes, a.No / 2, a.Kc, 1, false);
  else bad |= encode_map(ctx->encode_tiled, &tb, a.b_codes, a.Kc / 2, a.No, 1, false);
  if (bad) return LUQ_ERR_CUDA;

  const long long units = tiles * p.splits;
  const int grid = static_cast<int>(units < ctx->sm_count ? units : ctx->sm_count);
  int rc;
  const int sel = (ctx->mma_kind ? 4 : 0) | (a.a_mn ? 2 : 0) | (a.b_mn ? 1 : 0);
  switch (sel) {
    case 0: rc = launch<0, false, false>(ta, tb, p, grid, st); break;
    case 1: rc = launch<0, false, true>(ta, tb, p, grid, st); break;
    case 3: rc = launch<0, true, true>(ta, tb, p, grid, st); break;
    case 4: rc = launch<1, false, false>(ta, tb, p, grid, st); break;
    case 5: rc = launch<1, false, true>(ta, tb, p, grid, st); break;
    case 7: rc = launch<1, true, true>(ta, tb, p, grid, st); break;
    default: return LUQ_ERR_UNSUPPORTED;
  }
  if (rc == 0) ctx->launches += 1;
  return rc;
}
