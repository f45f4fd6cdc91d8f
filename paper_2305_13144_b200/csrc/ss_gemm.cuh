// Weight-streaming GEMM for sm_100a:  D[n_out, tok] = W[n_out, K] . X[tok, K]^T   (bf16 in, fp32 accumulate)
//
// The weight matrix is the tcgen05 "A" operand (128 rows per tile), the activations are "B"
// (16..256 tokens per tile), so a decode step with a handful of rows still fills the 128-lane
// tensor-memory accumulator while every weight byte crosses HBM exactly once.  Both operands
// arrive by TMA (128-byte swizzle) into a multi-stage shared-memory ring; one elected thread
// issues tcgen05.mma; four warps drain the accumulator from tensor memory.
//
// Work decomposition: the (tile, k-block) iteration space is cut into gridDim.y equal
// contiguous ranges.  A range that ends inside a tile produces a partial sum; in kGemmPartial
// mode all segments are written as fp32 partials which the consumer kernel adds in CTA order.
//
// Programmatic dependent launch: weights never depend on the previous kernel, so the producer
// fills the ring with weight tiles BEFORE griddepcontrol.wait and only then loads activations.
// Every wait on an mbarrier is bounded; on expiry the kernel records a status word and leaves.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ss_internal.h"

namespace ss {

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after ~2 s of SM clock, records `code` and returns false.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t* status, uint32_t code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (clock64() - t0 > 4000000000LL) {
      atomicCAS(status, 0u, code);
      return false;
    }
  }
}

__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                            uint64_t hint) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      :
      : "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y), "l"(hint)
      : "memory");
}
// Linear bulk copy global -> shared (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t hint) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      :
      : "r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar), "l"(hint)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], bf16 x bf16 -> fp32, M = 128, N from the instruction descriptor, K = 16.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      :
      : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 8 consecutive fp32 columns: thread i of the warp gets lane (base + i), columns c..c+7.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
               : "r"(taddr)
               : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  v[0] = __uint_as_float(r0); v[1] = __uint_as_float(r1); v[2] = __uint_as_float(r2); v[3] = __uint_as_float(r3);
  v[4] = __uint_as_float(r4); v[5] = __uint_as_float(r5); v[6] = __uint_as_float(r6); v[7] = __uint_as_float(r7);
}
// 32 lanes x 32 consecutive fp32 columns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
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
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// 32 lanes x 64 consecutive fp32 columns in one load.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&r)[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 {"
      "%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];\n"
      "tcgen05.wait::ld.sync.aligned;"
      :
        "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]),
        "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]),
        "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]),
        "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]),
        "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
      : "r"(taddr)
      : "memory");
}

// ---- forms for a pair of CTAs on neighbouring SMs working on one accumulator tile (cta_group::2) ---------------
// TMA tile load whose bytes are counted on the mbarrier of the pair's first CTA (the one that issues the MMAs):
// both CTAs execute it with the address of their own copy of the barrier; clearing the CTA-rank bit of the
// shared-window address makes it the first CTA's.  Every CTA loads only its own operand halves.
constexpr uint32_t kPairLeaderMask = 0xFEFFFFFFu;
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y,
                                                 uint64_t hint) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4}], [%2], %5;"
      :
      : "r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar & kPairLeaderMask), "r"(x), "r"(y), "l"(hint)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B with M = 256 (128 rows from each CTA's shared memory), N from the descriptor
// (half of the B rows from each CTA), K = 16.  Issued by one thread of the pair's first CTA.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      :
      : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z)
      : "memory");
}
// Arrives on the same-named mbarrier of both CTAs of the pair once every MMA issued so far has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);          // start address
  d |= (uint64_t)1 << 16;                          // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                          // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                          // layout: SWIZZLE_128B
  return d;
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = m (128 or 64), N = n.
// Accumulator row i of an M = 128 instruction is tensor-memory lane i; of an M = 64 instruction it is lane
// (i % 16) + 32 * (i / 16), i.e. the first 16 lanes of each warp's lane quarter.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int n, int m = 128) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------ split bookkeeping
__host__ __device__ __forceinline__ long long split_begin(const SplitInfo& s, int c) {
  return (long long)c * s.total / s.gridx;
}
// CTA whose range holds iteration x.
__host__ __device__ __forceinline__ int split_owner(const SplitInfo& s, long long x) {
  int c = (int)(x * s.gridx / s.total);
  while (c + 1 < s.gridx && split_begin(s, c + 1) <= x) ++c;
  return c;
}
// Sum of the fp32 partials of output row n (of n_out) for token `tok`, in CTA order; the tile's
// segments are derived from the split arithmetic on the fly (several 64-bit divisions).
__device__ __forceinline__ float sum_partials_derived(const float* __restrict__ partial, const SplitInfo& s, int n, int tok) {
  const int tile = n >> 7, row = n & 127;
  const long long x0 = (long long)tile * s.kb;
  const int c0 = split_owner(s, x0), c1 = split_owner(s, x0 + s.kb - 1);
  float acc = 0.f;
  for (int c = c0; c <= c1; ++c) {
    const int seg = tile - (int)(split_begin(s, c) / s.kb);
    const size_t slot = (size_t)c * s.max_seg + seg;
    acc += partial[(slot * s.NT + tok) * 128 + row];
  }
  return acc;
}
// The same sum with the tile's segments read from the precomputed table (same order, same bits).
__device__ __forceinline__ float sum_partials(const float* __restrict__ partial, const SplitInfo& s, int n, int tok) {
  const int4 t = __ldg(reinterpret_cast<const int4*>(s.tiles) + (n >> 7));
  const size_t slot_stride = (size_t)s.NT * 128;
  const size_t off = (size_t)tok * 128 + (n & 127);
  float acc = partial[(size_t)t.x * slot_stride + off];
  const size_t cta_stride = slot_stride * s.max_seg;
  for (int c = t.y; c <= t.z; ++c) acc += partial[(size_t)c * cta_stride + off];
  return acc;
}

// ------------------------------------------------------------------------------------ the kernel
constexpr int kGemmThreads = 192;   // warp 0: TMA producer, warp 1: MMA issuer, warps 2..5: epilogue
constexpr int kGemmMaxStages = 16;

struct GemmSmemHeader {
  uint64_t full[kGemmMaxStages];
  uint64_t empty[kGemmMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  uint32_t pad;
};

// internal linkage: the header is compiled into more than one translation unit
static __global__ void __launch_bounds__(kGemmThreads, 1)
gemm_wx_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const GemmPlan& p = a.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.y, tok_tile = blockIdx.x;

  // carve shared memory: header, then 1024-byte aligned stages
  GemmSmemHeader* hdr = reinterpret_cast<GemmSmemHeader*>(smem_raw);
  const uint32_t smem_base = smem_u32(smem_raw);
  const uint32_t stage0 = (smem_base + (uint32_t)sizeof(GemmSmemHeader) + 1023u) & ~1023u;
  const uint32_t a_bytes = kTileM * kTileK * 2;               // 16 KiB
  const uint32_t b_bytes = (uint32_t)p.NT * kTileK * 2;
  const uint32_t stage_bytes = a_bytes + b_bytes;

  const long long total = (long long)p.n_tiles * p.kb;
  const long long it0 = (long long)cta * total / p.gridx;
  const long long it1 = (long long)(cta + 1) * total / p.gridx;
  const int n_it = (int)(it1 - it0);

  if (threadIdx.x == 0) {
    pdl_launch_dependents();
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&hdr->acc_full[b]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[b]), 4);
    }
    fence_barrier_init();
    if (!a.w_tiled) tma_prefetch_desc(&map_w);
    tma_prefetch_desc(&map_x);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&hdr->tmem_base), (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = hdr->tmem_base;

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      // weights are streamed once: evict-first; activations are shared by all CTAs: evict-last
      uint64_t hint_w, hint_x;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(hint_w));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(hint_x));
      const int pre = n_it < p.stages ? n_it : p.stages;
      // Repacked weights: the 128-row tile `tile` at k-block `kblk` is one half of the 32 KiB block
      // (tile / 2, kblk), already in the swizzled shared-memory image.
      const uint8_t* w_tiled = reinterpret_cast<const uint8_t*>(a.w_tiled);
      auto w_block = [&](int tile, int kblk) {
        return w_tiled + ((size_t)(tile >> 1) * p.kb + kblk) * (size_t)kBlockBytes + (size_t)(tile & 1) * a_bytes;
      };
      // phase 1: weight tiles of the first ring fill, before the dependency resolves
      for (int i = 0; i < pre; ++i) {
        const long long it = it0 + i;
        const int tile = (int)(it / p.kb), kblk = (int)(it % p.kb);
        const uint32_t full = smem_u32(&hdr->full[i]);
        mbar_expect_tx(full, stage_bytes);
        if (w_tiled) bulk_load(stage0 + i * stage_bytes, w_block(tile, kblk), a_bytes, full, hint_w);
        else tma_load_2d(stage0 + i * stage_bytes, &map_w, full, kblk * kTileK, tile * kTileM, hint_w);
      }
      pdl_wait();
      for (int i = 0; i < pre; ++i) {
        const long long it = it0 + i;
        const int kblk = (int)(it % p.kb);
        tma_load_2d(stage0 + i * stage_bytes + a_bytes, &map_x, smem_u32(&hdr->full[i]), kblk * kTileK,
                    tok_tile * p.NT, hint_x);
      }
      // phase 2: steady state (second and later passes over the ring)
      int stage = 0, issued = pre;
      uint32_t phase = 1u;
      for (int i = pre; i < n_it; ++i) {
        const long long it = it0 + i;
        const int tile = (int)(it / p.kb), kblk = (int)(it % p.kb);
        if (!mbar_wait(smem_u32(&hdr->empty[stage]), phase ^ 1u, a.status, kStatusProducerTimeout)) break;
        const uint32_t full = smem_u32(&hdr->full[stage]);
        mbar_expect_tx(full, stage_bytes);
        if (w_tiled) bulk_load(stage0 + stage * stage_bytes, w_block(tile, kblk), a_bytes, full, hint_w);
        else tma_load_2d(stage0 + stage * stage_bytes, &map_w, full, kblk * kTileK, tile * kTileM, hint_w);
        tma_load_2d(stage0 + stage * stage_bytes + a_bytes, &map_x, full, kblk * kTileK, tok_tile * p.NT, hint_x);
        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        ++issued;
      }
      if (issued < n_it) {
        // a wait ran out and the kernel is leaving: the copies still in flight (at most one ring) get a bounded
        // time to land before the CTA's shared memory is given up
        for (int s2 = 0; s2 < p.stages; ++s2) {
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&hdr->full[s2]), 0u) && !mbar_try_wait(smem_u32(&hdr->full[s2]), 1u) &&
                 clock64() - t0 < 2000000LL) { }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      pdl_wait();
      const uint32_t idesc = umma_idesc_bf16(p.NT);
      int stage = 0;
      uint32_t phase = 0;
      int seg = 0;
      bool ok = true;
      long long it = it0;
      while (it < it1 && ok) {
        const int tile = (int)(it / p.kb);
        long long seg_end = (long long)(tile + 1) * p.kb;
        if (seg_end > it1) seg_end = it1;
        const int buf = seg & 1;
        const uint32_t use = (uint32_t)(seg >> 1);
        // wait until the epilogue has drained this accumulator buffer (first use passes at once)
        ok = mbar_wait(smem_u32(&hdr->acc_empty[buf]), (use & 1u) ^ 1u, a.status, kStatusMmaTimeout);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.NT);
        bool first = true;
        for (; it < seg_end; ++it) {
          ok = mbar_wait(smem_u32(&hdr->full[stage]), phase, a.status, kStatusMmaTimeout);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = stage0 + stage * stage_bytes;
          const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
          for (int k = 0; k < kTileK / 16; ++k) {
            // +32 bytes per 16-element K step inside the 128-byte swizzled row
            umma_bf16(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (first && k == 0) ? 0u : 1u);
          }
          first = false;
          umma_commit(smem_u32(&hdr->empty[stage]));      // frees the stage when these MMAs retire
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&hdr->acc_full[buf]));
        ++seg;
      }
    }
  } else {
    // ===================== epilogue (4 warps, one TMEM lane quarter each) =====================
    pdl_wait();
    const int quarter = warp & 3;                 // warps 2,3,4,5 -> lane quarters 2,3,0,1
    const int row = quarter * 32 + lane;          // row inside the 128-row tile
    int seg = 0;
    long long it = it0;
    const int tok0 = tok_tile * p.NT;
    int n_valid = a.n_tok - tok0;
    if (n_valid > p.NT) n_valid = p.NT;
    while (it < it1) {
      const int tile = (int)(it / p.kb);
      long long seg_end = (long long)(tile + 1) * p.kb;
      if (seg_end > it1) seg_end = it1;
      const int buf = seg & 1;
      const uint32_t use = (uint32_t)(seg >> 1);
      bool ok = mbar_wait(smem_u32(&hdr->acc_full[buf]), use & 1u, a.status, kStatusEpilogueTimeout);
      ok = __all_sync(0xffffffffu, ok);           // warp-uniform, and reconverges the warp
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.NT);
      const int n = tile * kTileM + row;            // output feature
      if (a.mode == kGemmPartial) {
        const size_t slot = (size_t)cta * p.max_seg + seg;
        float* dst = a.partial + slot * p.NT * 128 + row;
        for (int c = 0; c < p.NT; c += 8) {
          float v[8];
          tmem_ld8(taddr + c, v);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (c + j < n_valid) dst[(size_t)(c + j) * 128] = v[j];
        }
      } else if (a.mode == kGemmDirectBf16) {
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out_bf16);
        for (int c = 0; c < p.NT; c += 8) {
          float v[8];
          tmem_ld8(taddr + c, v);
          if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (c + j < n_valid) out[(size_t)(tok0 + c + j) * a.ld_out + n] = __float2bfloat16_rn(v[j]);
          }
        }
      } else if (a.mode == kGemmDirectF32) {
        // plain fp32 store: the consumer (RoPE, SwiGLU) rounds once, after its own arithmetic
        for (int c = 0; c < p.NT; c += 8) {
          float v[8];
          tmem_ld8(taddr + c, v);
          if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (c + j < n_valid) a.out_f32[(size_t)(tok0 + c + j) * a.ld_out + n] = v[j];
          }
        }
      } else if (p.NT % 32 == 0) {
        // read-modify-write of the fp32 residual: 32 tokens' loads in flight per round trip
        for (int c = 0; c < p.NT; c += 32) {
          float v[32], h[32];
          tmem_ld32(taddr + c, v);
          if (n < p.n_out) {
            float* o = a.out_f32 + (size_t)(tok0 + c) * a.ld_out + n;
#pragma unroll
            for (int j = 0; j < 32; ++j) h[j] = (c + j < n_valid) ? __ldcg(o + (size_t)j * a.ld_out) : 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c + j < n_valid) o[(size_t)j * a.ld_out] = h[j] + v[j];
          }
        }
      } else {
        for (int c = 0; c < p.NT; c += 8) {
          float v[8];
          tmem_ld8(taddr + c, v);
          if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (c + j < n_valid) a.out_f32[(size_t)(tok0 + c + j) * a.ld_out + n] += v[j];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&hdr->acc_empty[buf]));
      it = seg_end;
      ++seg;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// ------------------------------------------------------------------------------------ the paired kernel
// The prompt-pass GEMM on pairs of CTAs (a cluster of two neighbouring SMs, tcgen05 cta_group::2): the pair
// computes a 256-row x 256-token tile, CTA r of the pair holding weight rows 128 r .. 128 r + 127 (its half of a
// 32 KiB block of the tiled layout) and tokens 128 r .. 128 r + 127 of the token tile in its shared memory, and
// rows 128 r .. of the accumulator in its tensor memory.  One thread of the first CTA issues the MMAs for both.
// Why: with one CTA per tile, 48 KiB written into shared memory and 48 KiB read out of it by the tensor core per
// k-block exceed what the shared memory of one SM moves in the 512 cycles the four MMAs take; in the pair every
// CTA stages 32 KiB per k-block for the same arithmetic.
constexpr int kPairStageBytes = 2 * kTileM * kTileK * 2;        // 16 KiB of weights + 16 KiB of activations
constexpr int kPairTokens = 256;                                 // token tile of the pair (128 per CTA)

// Remote arrival on the first CTA's copy of a barrier (used by the partner's epilogue warps).
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar & kPairLeaderMask) : "memory");
}

// Persistent: gridDim.x / 2 pairs walk the (pair of weight tiles, token tile) units pair, pair + P, pair + 2 P, ...
// with the token tile as the fast index (pairs that run side by side read the same weight block: it crosses HBM
// once).  Two accumulator buffers of 256 columns: the drain of one unit overlaps the MMAs of the next.
static __global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_wx_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const GemmPlan& p = a.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();          // 0: issues the MMAs; 1: its partner
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int tok_tiles = p.gridy;                     // token tiles of 256
  const int n_units = (p.n_tiles >> 1) * tok_tiles;
  GemmSmemHeader* hdr = reinterpret_cast<GemmSmemHeader*>(smem_raw);
  const uint32_t stage0 = (smem_u32(smem_raw) + (uint32_t)sizeof(GemmSmemHeader) + 1023u) & ~1023u;
  const uint32_t a_bytes = kTileM * kTileK * 2;
  const int kb = p.kb;

  if (threadIdx.x == 0) {
    pdl_launch_dependents();
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(smem_u32(&hdr->full[s]), 1);
      mbar_init(smem_u32(&hdr->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&hdr->acc_full[b]), 1);
      mbar_init(smem_u32(&hdr->acc_empty[b]), 8);    // four epilogue warps of each CTA (used in the first CTA only)
    }
    fence_barrier_init();
    tma_prefetch_desc(&map_w);
    tma_prefetch_desc(&map_x);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&hdr->tmem_base), 2u * kPairTokens);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // both CTAs' barriers exist before either signals the other's
  tc_fence_after();
  const uint32_t tmem_base = hdr->tmem_base;

  if (warp == 0) {
    // ===================== TMA producer (one per CTA) =====================
    if (lane == 0) {
      uint64_t hint_w, hint_x;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(hint_w));
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(hint_x));
      pdl_wait();
      int stage = 0, gi = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair; u < n_units && ok; u += n_pairs) {
        const int wt = u / tok_tiles, tt = u - wt * tok_tiles;
        // the tiled weights seen as lines of 128 bytes: this CTA's half of block (wt, k) starts at line
        // (wt * kb + k) * 256 + rank * 128 and is 128 lines long
        const int line0 = wt * kb * kTileN + (int)rank * kTileM;
        const int tok0 = tt * kPairTokens + (int)rank * (kPairTokens / 2);
        for (int i = 0; i < kb; ++i, ++gi) {
          if (gi >= p.stages && !(ok = mbar_wait(smem_u32(&hdr->empty[stage]), phase ^ 1u, a.status, kStatusProducerTimeout))) break;
          const uint32_t full = smem_u32(&hdr->full[stage]);
          // the first CTA's barrier counts the bytes of all four loads of the stage (two per CTA)
          if (rank == 0) mbar_expect_tx(full, 2u * kPairStageBytes);
          const uint32_t dst = stage0 + (uint32_t)stage * kPairStageBytes;
          tma_load_2d_pair(dst, &map_w, full, 0, line0 + i * kTileN, hint_w);
          tma_load_2d_pair(dst + a_bytes, &map_x, full, i * kTileK, tok0, hint_x);
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // a wait ran out: give the copies in flight a bounded time to land before the shared memory is given up
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (first CTA of the pair only) =====================
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_bf16(kPairTokens, 256);
      int stage = 0, r = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair; u < n_units && ok; u += n_pairs, ++r) {
        const int buf = r & 1;
        // both CTAs' epilogues have drained this buffer (its first use passes at once)
        ok = mbar_wait(smem_u32(&hdr->acc_empty[buf]), ((uint32_t)(r >> 1) & 1u) ^ 1u, a.status, kStatusMmaTimeout);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kPairTokens);
        for (int i = 0; i < kb; ++i) {
          ok = mbar_wait(smem_u32(&hdr->full[stage]), phase, a.status, kStatusMmaTimeout);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = stage0 + (uint32_t)stage * kPairStageBytes;
          const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + a_bytes);
#pragma unroll
          for (int k = 0; k < kTileK / 16; ++k)
            umma_bf16_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, (i == 0 && k == 0) ? 0u : 1u);
          umma_commit_pair(smem_u32(&hdr->empty[stage]));    // frees the stage in both CTAs when these MMAs retire
          if (++stage == p.stages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(smem_u32(&hdr->acc_full[buf]));
      }
    }
  } else {
    // ===================== epilogue (4 warps, one TMEM lane quarter each): this CTA's 128 rows x 256 tokens ====
    pdl_wait();
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    int r = 0;
    for (int u = pair; u < n_units; u += n_pairs, ++r) {
      const int wt = u / tok_tiles, tt = u - wt * tok_tiles;
      const int buf = r & 1;
      const int tok0 = tt * kPairTokens;
      int n_valid = a.n_tok - tok0;
      if (n_valid > kPairTokens) n_valid = kPairTokens;
      bool ok = mbar_wait(smem_u32(&hdr->acc_full[buf]), (uint32_t)(r >> 1) & 1u, a.status, kStatusEpilogueTimeout);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kPairTokens);
      const int n = (2 * wt + (int)rank) * kTileM + row;
      if (a.mode == kGemmDirectF32) {
        for (int c = 0; c < kPairTokens; c += 32) {
          float v[32];
          tmem_ld32(taddr + c, v);
          if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c + j < n_valid) a.out_f32[(size_t)(tok0 + c + j) * a.ld_out + n] = v[j];
          }
        }
      } else if (a.mode == kGemmDirectBf16) {
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out_bf16);
        for (int c = 0; c < kPairTokens; c += 32) {
          float v[32];
          tmem_ld32(taddr + c, v);
          if (n < p.n_out) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c + j < n_valid) out[(size_t)(tok0 + c + j) * a.ld_out + n] = __float2bfloat16_rn(v[j]);
          }
        }
      } else {
        // read-modify-write of the fp32 residual: 32 tokens' loads in flight per round trip
        for (int c = 0; c < kPairTokens; c += 32) {
          float v[32], h[32];
          tmem_ld32(taddr + c, v);
          if (n < p.n_out) {
            float* o = a.out_f32 + (size_t)(tok0 + c) * a.ld_out + n;
#pragma unroll
            for (int j = 0; j < 32; ++j) h[j] = (c + j < n_valid) ? __ldcg(o + (size_t)j * a.ld_out) : 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c + j < n_valid) o[(size_t)j * a.ld_out] = h[j] + v[j];
          }
        }
      }
      // the buffer may be overwritten once all eight epilogue warps of the pair have read it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(smem_u32(&hdr->acc_empty[buf]));
        else mbar_arrive_leader(smem_u32(&hdr->acc_empty[buf]));
      }
    }
  }

  // neither CTA may give up its shared or tensor memory while the other's MMAs or copies can still touch it
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 2u * kPairTokens);
  }
}

}  // namespace ss
