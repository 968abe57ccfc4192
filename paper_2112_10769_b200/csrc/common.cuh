// Shared declarations of the sm_100a library: context, status word, PTX wrappers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "luq.h"

#define LUQ_KMAX 4  // default level count: alpha = max / 2^LUQ_KMAX (Eq. alpha with b = 3)
#define LUQ_DEFAULT_MMA_KIND 2  // automatic: int8, the type of the operand bytes the quantizers can emit

struct luq_ctx {
  int device;
  int sm_count;
  unsigned int* d_status;   // device status word (LUQ_STATUS_* bits)
  unsigned int* d_scratch;  // grid-wide maximum: ticket counter (zero between kernels) + one word per block
  float* d_workspace;       // split-contraction partial tiles
  size_t workspace_bytes;
  int mma_kind;             // 0 f8f6f4/e4m3, 1 i8, 2 chosen per product
  int forced_splits;        // 0 = automatic
  int use_pairs;            // CTA-pair kernel for products whose operands are both planes
  int out_bf16;             // the GEMMs write bf16 outputs
  int unsigned_act;         // activation codes handed to the forward / update GEMMs are unsigned INT4
  int grad_int4;            // gradient codes handed to the backward / update GEMMs are INT4 (the ablation's uniform arm)
  int sm_limit;             // GEMM grids use at most this many SMs (0 = all)
  int sum_samples;          // the LUQ quantizers' operand bytes are one plane: the sum over the samples
  int kmax;                 // LUQ levels alpha * 2^0 .. alpha * 2^kmax (1..6, default LUQ_KMAX)
  int64_t launches;
  void* encode_tiled;       // cuTensorMapEncodeTiled, resolved at create
};

// internal launchers (defined in quant.cu / gemm.cu); return a cudaError_t as int
int luq_launch_amax(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_amax, cudaStream_t st);
// d_operand (may be null): int8 operand bytes, one per element (and per sample), written with the codes
// d_amax_out (may be null): fused - the kernel reduces the tensor's maximum itself, uses it as clip, writes it there
// is_unsigned: the grid 0..15 with scale clip/15 instead of -7..7 with clip/7 (not with d_amax_out)
int luq_launch_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t n, const float* d_clip,
                          uint8_t* d_codes, int8_t* d_operand, float* d_scale, float* d_amax_out, bool is_unsigned,
                          cudaStream_t st);

// in-hindsight INT4: d_estimate is the clip (values beyond it saturate); the tensor's own max|x| goes to
// d_measured and d_estimate is replaced by (1 - eta) * measured + eta * estimate, all in one kernel
int luq_launch_quant_int4_hindsight(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_estimate, float eta,
                                    uint8_t* d_codes, int8_t* d_operand, float* d_scale, float* d_measured,
                                    cudaStream_t st);
// flags: bit 0 = power-of-two scale; bit 1 = in-hindsight (d_amax is the running estimate: the tensor's own
// max|x| goes to d_measured and d_estimate (= d_amax) is replaced by (1 - eta) * measured + eta * estimate);
// bit 2 = deterministic rounding; bit 3 = d_operand is one plane, the sum of the samples' bytes
int luq_launch_quant_grad_ex(luq_ctx* ctx, const void* d_g, int dtype, size_t n, const float* d_amax, uint64_t seed,
                             int n_samples, uint8_t* d_codes, int8_t* d_operand, float* d_alpha, int flags,
                             float* d_measured, float* d_estimate, float eta, float* d_amax_out, cudaStream_t st);
// scheme: bit 0 = stochastic rounding inside the range, bit 1 = stochastic underflow, on the LUQ grid
// (the other region rounds to the nearest level; d_scale gets alpha); 4 = the uniform grid -7..7 with
// stochastic rounding (INT4 codes, d_scale gets max/7)
int luq_launch_quant_grad_ablation(luq_ctx* ctx, const void* d_g, int dtype, size_t n, const float* d_amax,
                                   uint64_t seed, int n_samples, int scheme, uint8_t* d_codes, int8_t* d_operand,
                                   float* d_scale, cudaStream_t st);
// Scratch words for grid-wide maxima.  Words 0 .. LUQ_SCRATCH_SINGLE-1: the one-tensor kernels (two
// counters + one word per block).  Then LUQ_SCRATCH_MULTI regions of LUQ_SCRATCH_REGION words, one per
// tensor of a several-tensor launch.  Grids of the reducing kernels stay below the region sizes.
#define LUQ_SCRATCH_SINGLE 4096
#define LUQ_SCRATCH_REGION 2048
#define LUQ_SCRATCH_MULTI 4
#define LUQ_SCRATCH_WORDS (LUQ_SCRATCH_SINGLE + LUQ_SCRATCH_MULTI * LUQ_SCRATCH_REGION)
// several tensors of one element type in one launch (count <= LUQ_SCRATCH_MULTI); host arrays
int luq_launch_amax_multi(luq_ctx* ctx, int count, const void* const* d_x, const size_t* n, float* const* d_amax,
                          int dtype, cudaStream_t st);
int luq_launch_quant_int4_multi(luq_ctx* ctx, int count, const void* const* d_x, const size_t* n,
                                const float* const* d_clip, uint8_t* const* d_codes, float* const* d_scale,
                                int8_t* const* d_operand, int dtype, cudaStream_t st);
int luq_launch_debug_quotient(luq_ctx* ctx, const float* d_x, size_t n, const float* d_amax, float* d_t,
                              cudaStream_t st);

// One GEMM  D[Mo x No] = scale * sum_s sum_k opA_s[mo,k] * opB[no,k].
//   a_mn / b_mn: operand is stored contraction-major (rows = k) instead of
//   k-contiguous (rows = mo / no).  a_kind / b_kind: 0 INT4 codes, 1 LUQ codes, 2 unsigned INT4 codes.
struct luq_gemm_args {
  const uint8_t* a_codes; int a_kind; int a_mn; int n_samples;
  const uint8_t* b_codes; int b_kind; int b_mn;
  const int8_t* a_operand; const int8_t* b_operand;   // int8 operand bytes from the quantizer, or null
  int a_summed;   // > 1: a_operand is ONE plane, the sum of that many samples' bytes (n_samples equals it)
  const float* d_scale_a; const float* d_scale_b;
  void* d_out; int out_bf16;   // fp32 [Mo x No], or bf16 when out_bf16
  int64_t Mo, No, Kc;
  float* d_workspace; size_t workspace_bytes;   // split partial tiles (caller-chosen memory)
  int allow_split;
};
int luq_launch_gemm(luq_ctx* ctx, const luq_gemm_args& a, cudaStream_t st);
int luq_launch_expire_wait(luq_ctx* ctx, cudaStream_t st);
int luq_launch_bounds_probe(luq_ctx* ctx, cudaStream_t st);
// Forward product that quantizes its activations itself (one column of output tiles): writes the INT4
// codes of A, its scale and Z = Q(A) . Q(W)^T.  d_w_operand may be null (W's codes are then widened
// into the workspace).  Call only when luq_quant_fwd_fusable() says yes.
bool luq_quant_fwd_fusable(const luq_ctx* ctx, int64_t M, int64_t N, int64_t K, bool have_w_bytes);
// In-hindsight form (d_estimate != null; d_clip is then ignored): A is quantized with *d_estimate, its own
// max|a| goes to *d_measured and *d_estimate is replaced by (1 - eta) * measured + eta * estimate.
int luq_launch_quant_fwd(luq_ctx* ctx, const void* d_a, int dtype, const float* d_clip, uint8_t* d_a_codes,
                         float* d_sa, const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                         float* d_z, int64_t M, int64_t N, int64_t K, cudaStream_t st, float* d_estimate = nullptr,
                         float eta = 0.0f, float* d_measured = nullptr);

#ifdef __CUDACC__

// Launch helper.  LUQ_LAUNCH_COOPERATIVE: all blocks of the grid are resident at once (the kernel
// has a grid barrier inside).  LUQ_LAUNCH_EARLY = programmatic dependent launch: the kernel may
// become resident and set up (barriers, tensor memory, descriptor prefetch) while its predecessor
// in the stream drains, and waits in pdl_wait() until that predecessor has completed and its writes
// are visible.  Every kernel of the library calls pdl_wait() before its first access to global
// memory, and all but the cooperative ones are launched this way.  One trap, measured: a small
// streaming block that becomes resident beside a running GEMM block sits on an SM carved for
// maximum shared memory and keeps that small L1 after the GEMM has gone (the 462 MB max reduction:
// 68 -> 96 us).  The streaming kernels therefore state a preference for the largest L1 carve-out,
// which keeps their blocks off such an SM until it is free.
#define LUQ_LAUNCH_NORMAL 0
#define LUQ_LAUNCH_EARLY 1
#define LUQ_LAUNCH_COOPERATIVE 2
template <typename... KArgs, typename... Args>
cudaError_t luq_launch_kernel(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                              int mode, unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
  cfg.blockDim = dim3(static_cast<unsigned>(block), 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (mode == LUQ_LAUNCH_EARLY) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  } else if (mode == LUQ_LAUNCH_COOPERATIVE) {
    attr[n].id = cudaLaunchAttributeCooperative;
    attr[n].val.cooperative = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Checking build (-DLUQ_DEBUG): LUQ_IN_BOUNDS(cond, status) is `cond`, and a false one raises
// LUQ_STATUS_BOUNDS in the status word; callers skip the access.  In the normal build it is `true`
// and costs nothing.
#ifdef LUQ_DEBUG
#define LUQ_IN_BOUNDS(cond, status) ((cond) ? true : (atomicOr((status), LUQ_STATUS_BOUNDS), false))
#else
#define LUQ_IN_BOUNDS(cond, status) (true)
#endif

namespace luqdev {

// is [p, p + bytes) inside the region [lo, hi) of the CTA's shared-memory block starting at `base`?
// (always true, and free, outside the checking build)
__device__ __forceinline__ bool smem_in(const void* p, const void* base, int lo, int hi, int bytes, unsigned int* status) {
  const long long off = static_cast<const unsigned char*>(p) - static_cast<const unsigned char*>(base);
  (void)off; (void)lo; (void)hi; (void)bytes; (void)status;
  return LUQ_IN_BOUNDS(off >= lo && off + bytes <= hi, status);
}
// do the 32 accumulator columns read at `taddr` lie inside the `cols` columns allocated at `tmem_base`?
__device__ __forceinline__ bool tmem_in(unsigned int taddr, unsigned int tmem_base, int cols, unsigned int* status) {
  const int col = static_cast<int>(taddr & 0xFFFFu) - static_cast<int>(tmem_base & 0xFFFFu);
  const int lane = static_cast<int>(taddr >> 16) - static_cast<int>(tmem_base >> 16);
  (void)col; (void)lane; (void)cols; (void)status;
  return LUQ_IN_BOUNDS(col >= 0 && col + 32 <= cols && lane >= 0 && lane + 32 <= 128, status);
}

// waits until the preceding kernel of the stream has completed and its memory is visible
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// lets the next kernel of the stream become resident (it still waits for this one to complete)
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- mbarrier ---------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// Bounded wait: gives up after about two seconds and reports it.  The first probe is
// inlined (the single-thread producer and MMA loops run it every stage); the spin is not.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
    if (mbar_test(bar, parity)) return true;
    if (spin > 1024) {
      if (*abort_flag) return false;
      __nanosleep(spin > 65536 ? 512 : 32);
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag);
}
// The same bounded wait for roles that wait by the dozen of warps (the converters of the fused forward
// kernel): it sleeps between probes from the start, so that waiting warps leave the issue slots to the
// working ones.
static __device__ __noinline__ bool mbar_wait_idle_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
    if (mbar_test(bar, parity)) return true;
    if ((spin & 255u) == 255u && *abort_flag) return false;
    __nanosleep(spin > 4096 ? 512 : 48);
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test(bar, parity)) return true;
  return mbar_wait_idle_slow(bar, parity, abort_flag);
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- TMA --------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// store of a shared-memory box to global memory through a tensor map (clipped at the tensor's edges)
__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const void* tmap, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until at most N of this thread's bulk groups still read their shared-memory source
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N> __device__ __forceinline__ void bulk_wait() {
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// ---- tcgen05 / tensor memory ---------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// arrives on an mbarrier once all tcgen05.mma issued so far by this thread are done
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <int KIND>
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                       uint32_t accumulate) {
  if constexpr (KIND == 0) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// 32 lanes x 32 columns of 32-bit accumulators: thread t gets row (lane base + t)
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// ---- CTA pairs (cluster of two, tcgen05 cta_group::2) -----------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// wait whose acquire covers arrivals made by the peer CTA
__device__ __forceinline__ bool mbar_test_cluster(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 P, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
static __device__ __noinline__ bool mbar_wait_cluster_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t spin = 0; spin < (1u << 22); ++spin) {
    if (mbar_test_cluster(bar, parity)) return true;
    if (spin > 1024) {
      if (*abort_flag) return false;
      __nanosleep(spin > 65536 ? 512 : 32);
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_test_cluster(bar, parity)) return true;
  return mbar_wait_cluster_slow(bar, parity, abort_flag);
}
// TMA load issued inside a CTA pair: data lands in this CTA, the transaction bytes are
// counted on the mbarrier `bar_cluster` (a shared::cluster address, here the leader's)
__device__ __forceinline__ void tma_pair_load_2d(uint32_t dst, const void* tmap, uint32_t bar_cluster, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_3d(uint32_t dst, const void* tmap, uint32_t bar_cluster, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// arrives, in both CTAs of the pair, on the mbarrier at this shared-memory offset once all
// tcgen05.mma issued so far by this thread are done
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}
template <int KIND>
__device__ __forceinline__ void tc_mma_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  if constexpr (KIND == 0) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

// Shared-memory matrix descriptor for tcgen05.mma, 128-byte swizzle.
//   bits  0..13 start address >> 4, 16..29 leading byte offset >> 4,
//   32..45 stride byte offset >> 4, 46..47 version (1 on sm_100), 61..63 layout (2 = 128B swizzle)
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

}  // namespace luqdev
#endif  // __CUDACC__
