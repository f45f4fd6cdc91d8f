// One decode step as ONE persistent cooperative kernel (one CTA per SM).
//
// Why: a decode step at small batch is a chain of ~130 weight-streaming projections separated by
// tiny dependent stages.  As separate kernels every projection pays several microseconds of
// launch, ramp-up and drain during which HBM idles.  Here a dedicated producer warp streams the
// tiled weights of ALL projections of the step, in order, through one shared-memory ring; it
// never waits for activations, so while the other warps sit in a grid barrier or run a small
// stage, the ring keeps filling with the next projection's weights.
//
// Warp roles (352 threads):
//   warp 0      weight producer: linear bulk copies of 32 KiB (256-row tile, k-block) images into the ring
//   warp 1      MMA issuer: tcgen05.mma, accumulators in tensor memory (two buffers)
//   warp 2      activation loader: TMA loads of the [tokens x 64] activation block of each ring stage,
//               issued once the stage that produced the activations has passed its grid barrier
//   warps 3-10  workers: drain accumulators to fp32 partials, then run the stage between two
//               projections (partial sums in CTA order, RoPE, cache append, attention, residual,
//               SwiGLU, arg-max, bookkeeping), separated by grid barriers
//
// Operand roles: one tcgen05.mma costs about the same issue time whatever its shape, so the decode
// projections put the WEIGHTS on the wide side: D[token, row] += X[token, 16] . W[row, 16]^T with
// M = 64 or 128 token lanes and N = 256 weight rows (8 KiB of weights per instruction).  Token lanes
// beyond the batch compute on whatever shared memory follows the activation block; rows of D are
// independent, and those lanes are never read.
//
// RMSNorm is applied lazily: the residual stage writes x' = bf16(h * g) and per-slice sums of
// squares; since a projection is linear, the consumer of its partial sums multiplies by
// rsqrt(mean h^2 + eps).  This lets a row be split over many CTAs without a cross-CTA reduction.
//
// Every wait (mbarrier, grid barrier, flag) is bounded; on expiry the kernel records a status word,
// raises a CTA-wide abort flag and all roles leave.
#pragma once

#include "ss_kernels.cuh"

namespace ss {

constexpr int kMegaThreads = 352;
constexpr int kMegaWorkers = 256;          // warps 3..10
constexpr int kMegaMaxStages = 8;          // ring depth bound (shared memory holds 5 at batch 16)
constexpr int kSegTabEntries = 256;        // tile-table entries kept in shared memory (the four per-layer projections)
constexpr int kRowSlice = 128;             // elements of a row handled by one residual work item (one warp, 4 per lane)
constexpr int kMaxSlices = 64;             // d_model <= 8192

enum : uint32_t { kStatusGridBarrierTimeout = 5, kStatusFlagTimeout = 6 };

struct MegaGemmShape {
  int n_tiles, kb, max_seg;
  int gsplit;              // CTAs that share the iteration space (the others idle through this projection)
  long long total;
  const TileSeg* tiles;
  int smem_off;            // first entry of this projection's table in MegaSmem::seg_tab, or -1 (read it from `tiles`)
};

// Range of the (tile, k-block) iteration space owned by a CTA.
__device__ __forceinline__ void mega_range(const MegaGemmShape& gs, int cta, long long& it0, long long& it1) {
  if (cta < gs.gsplit) {
    it0 = (long long)cta * gs.total / gs.gsplit;
    it1 = (long long)(cta + 1) * gs.total / gs.gsplit;
  } else {
    it0 = it1 = 0;
  }
}

struct MegaArgs {
  // model
  int n_layers, d, H, Dh, F, V, eos_id;
  float eps;
  const uint8_t* const* wptr;      // [4*L + 1] tiled weights in execution order (qkv, o, gate/up, down)*L, lm head
  const bf16* const* norm_ptr;     // [2*L + 1] gains: attn_norm(l), ffn_norm(l) ..., final
  const bf16* embed;
  const float* inv_freq;
  MegaGemmShape shape[5];          // qkv, o, gate/up, down, lm head
  // batch
  int B, NT, stages;
  int m_tiles;                     // 128-token accumulator tiles (1, or 2 above 128 rows)
  int x_rows;                      // activation rows per TMA load (the tensor map's box height)
  RowState st;
  KvLayout kv;
  // activations (decode buffers)
  float* h;                        // [B][d] residual stream
  bf16 *x, *o, *act;               // GEMM operands: x' [B][d], attention out [B][d], SwiGLU out [B][F]
  float* rowss;                    // [B][kMaxSlices] sums of squares of h per slice
  float* partial;
  float* tile_val;
  int32_t* tile_idx;
  int n_tiles_lm;
  // options
  const int32_t* forced;
  int32_t* next_tokens;
  float *dump_logits, *dump_hidden;
  int32_t* dump_choice;
  SampleCfg sample;
  // sync
  unsigned long long* grid_ctr;    // monotone arrival counter
  unsigned long long grid_base;    // its value when this launch starts
  uint32_t* status;
  unsigned long long* trace;       // [2 + 4 * projections] global-timer stamps of CTA 0 (stage boundaries)
  long long wait_limit;            // SM cycles after which any wait inside the kernel gives up
};

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

struct MegaSmem {
  uint64_t full[kMegaMaxStages];
  uint64_t empty[kMegaMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  volatile int w_issued;           // ring iterations armed by the weight producer
  volatile int act_epoch;          // projections whose activation operand is complete
  volatile int abort;
  int prefix[kMaxBatch + 1];
  float inv_s[kMaxBatch];          // 1/rms of every row for the running stage
  __align__(16) float q_s[8][128]; // attention: per worker warp, rotated query (then the new token's value); read as float4
  __align__(16) float att_s[8][9][132];   // attention: [pair of the pass][partial: 8 warps + new token][acc[Dh], max, sum]
  int pair_id[8], pair_ustart[9], pair_n, pair_next, pair_lo, pair_hi;
  // per-step attention set-up that does not change from layer to layer (valid when att_single)
  int att_single;                  // the CTA's pairs fit one pass: the lists above are built once per step
  int att_warp_pairs;              // the CTA's run has many pairs: every warp takes whole pairs (attention_warp_pairs)
  int pair_pos[8], pair_pgnew[8];  // per pass: new token's position and page
  int unit_pg[8][8];               // per pass: ids of the first 8 pages of each warp's slice of the scan
  float rope_c[8][128], rope_sn[8][128];   // cos / sin of the new position per pair, cooperative lane layout
  int4 seg_tab[kSegTabEntries];    // tile tables of the per-layer projections (when they fit)
  uint8_t active_s[kMaxBatch];     // rows active in this step
};
static_assert(sizeof(float) * 8 * 9 * 132 >= 2 * (2 * 4 * 64 * 4), "arg-max scratch aliases att_s");
static_assert(sizeof(float) * 8 * 9 * 132 >= 8 * 32 * 36 * sizeof(float), "the drain's transposition scratch aliases att_s");

__device__ __forceinline__ void named_bar_workers() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// mbarrier wait that also gives up when the CTA aborts.
__device__ __forceinline__ bool mega_wait(uint32_t bar, uint32_t parity, MegaSmem* sm, uint32_t* status, uint32_t code,
                                          long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (sm->abort) return false;
    if (clock64() - t0 > limit) {
      atomicCAS(status, 0u, code);
      sm->abort = 1;
      return false;
    }
    __nanosleep(40);                 // a spinning role must not starve the warps that share its scheduler
  }
}

// Arrival on a grid-wide counter and the bounded poll for `target` arrivals, as one thread of a CTA does them.
// Returns false when the limit ran out (or the CTA's abort flag went up) before the counter got there.
__device__ __forceinline__ bool arrive_and_poll(unsigned long long* ctr, unsigned long long target, long long limit,
                                                const volatile int* abort_flag) {
  // arrive: release-add without waiting for the old value (the writes of the whole CTA, made visible to this
  // thread by the bar.sync in front, are ordered before it); then poll with acquire loads
  asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(ctr), "l"(1ULL) : "memory");
  const long long t0 = clock64();
  while (ld_acquire_u64(ctr) < target) {
    if (abort_flag && *abort_flag) return false;
    if (clock64() - t0 > limit) return false;
  }
  return true;
}

// Workers only.  Returns false if the CTA aborted.  `wrote_operand`: this CTA wrote activations that other
// CTAs read with TMA after the barrier, so its global writes are ordered before the async proxy's reads.
// The barrier after a projection publishes only fp32 partials, which are read with ordinary loads: there the
// proxy fence is left out (with bulk copies of the weight ring in flight it took about 2 us per barrier).
__device__ __forceinline__ bool grid_barrier(const MegaArgs& a, MegaSmem* sm, unsigned long long& epoch, int wtid,
                                             bool wrote_operand) {
  if (wrote_operand) fence_proxy_async_global();
  named_bar_workers();
  ++epoch;
  if (wtid == 0) {
    const unsigned long long target = a.grid_base + epoch * gridDim.x;
    if (!arrive_and_poll(a.grid_ctr, target, a.wait_limit, &sm->abort) && !sm->abort) {
      atomicCAS(a.status, 0u, (uint32_t)kStatusGridBarrierTimeout);
      sm->abort = 1;
    }
  }
  named_bar_workers();
  return sm->abort == 0;
}

// The stages between projections are chains of dependent L2 round trips (~0.7 us each), not bandwidth: the
// helpers below put independent loads in flight together and keep only true dependencies serial.

// An L2 load that the compiler may not move (a plain __ldcg can sink to its first use, which puts its
// round trip back in series with the loads issued in between).
__device__ __forceinline__ float ldcg_now(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}

template <int N>
__device__ __forceinline__ void ldcg_vec(const float* p, float (&x)[N]) {
  static_assert(N == 2 || N == 4 || N == 8, "N");
  if constexpr (N == 2) {
    asm volatile("ld.global.cg.v2.f32 {%0, %1}, [%2];" : "=f"(x[0]), "=f"(x[1]) : "l"(p));
  } else {
#pragma unroll
    for (int i = 0; i < N; i += 4)
      asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];"
                   : "=f"(x[i]), "=f"(x[i + 1]), "=f"(x[i + 2]), "=f"(x[i + 3])
                   : "l"(p + i));
  }
}

// Partial sums of the N consecutive outputs n0.. (inside one tile) for token tok, read past L1: the tile's
// first segment, then segment 0 of CTAs c_next..c_last (additions in CTA order, so the sum does not depend
// on timing).  Split in three so that a stage can put the loads of several sums in flight before it waits:
//   tile_seg()       the tile's table entry (one load);
//   partials_issue() the first segment and the next BATCH segments (loads only, unconditional so that they
//                    stay in registers: past the last segment the last one is read again and dropped);
//   partials_sum()   the additions, and any segments beyond the first batch.
__device__ __forceinline__ int4 tile_seg(const MegaSmem* sm, const MegaGemmShape& s, int n0) {
  const int tile = n0 / kTileN;
  if (s.smem_off >= 0) return sm->seg_tab[s.smem_off + tile];
  return __ldg(reinterpret_cast<const int4*>(s.tiles) + tile);
}
template <int N, int BATCH>
struct PartialLoads {
  float x[N];
  float u[BATCH][N];
};
template <int N, int BATCH>
__device__ __forceinline__ void partials_issue(const float* __restrict__ partial, const MegaGemmShape& s, int NT, const int4 t,
                                               int n0, int tok, PartialLoads<N, BATCH>& q) {
  const size_t slot_stride = (size_t)NT * kTileN, cta_stride = slot_stride * s.max_seg;
  const size_t off = (size_t)tok * kTileN + (n0 % kTileN);
  ldcg_vec<N>(partial + (size_t)t.x * slot_stride + off, q.x);
#pragma unroll
  for (int j = 0; j < BATCH; ++j) ldcg_vec<N>(partial + (size_t)min(t.y + j, t.z) * cta_stride + off, q.u[j]);
}
template <int N, int BATCH>
__device__ __forceinline__ void partials_sum(const float* __restrict__ partial, const MegaGemmShape& s, int NT, const int4 t,
                                             int n0, int tok, const PartialLoads<N, BATCH>& q, float (&x)[N]) {
#pragma unroll
  for (int i = 0; i < N; ++i) x[i] = q.x[i];
  if (t.y > t.z) return;
#pragma unroll
  for (int j = 0; j < BATCH; ++j) {
    const bool on = t.y + j <= t.z;
#pragma unroll
    for (int i = 0; i < N; ++i) x[i] += on ? q.u[j][i] : 0.f;
  }
  const size_t cta_stride = (size_t)NT * kTileN * s.max_seg;
  const size_t off = (size_t)tok * kTileN + (n0 % kTileN);
  for (int c = t.y + BATCH; c <= t.z; c += BATCH) {
    float u[BATCH][N];
#pragma unroll
    for (int j = 0; j < BATCH; ++j) ldcg_vec<N>(partial + (size_t)min(c + j, t.z) * cta_stride + off, u[j]);
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      const bool on = c + j <= t.z;
#pragma unroll
      for (int i = 0; i < N; ++i) x[i] += on ? u[j][i] : 0.f;
    }
  }
}
// One sum on its own.
template <int N, int BATCH>
__device__ __forceinline__ void sum_partials_cg(const MegaSmem* sm, const float* __restrict__ partial, const MegaGemmShape& s,
                                                int NT, int n0, int tok, float (&x)[N]) {
  const int4 t = tile_seg(sm, s, n0);
  PartialLoads<N, BATCH> q;
  partials_issue<N, BATCH>(partial, s, NT, t, n0, tok, q);
  partials_sum<N, BATCH>(partial, s, NT, t, n0, tok, q, x);
}

// 1/rms of row r; warp-collective (every lane returns it).  Lane i reads slices i, i+32.
__device__ __forceinline__ float warp_row_inv_rms(const MegaArgs& a, int r, int lane) {
  const int ns = (a.d + kRowSlice - 1) / kRowSlice;        // <= 64
  const float* p = a.rowss + (size_t)r * kMaxSlices;
  const float v0 = lane < ns ? ldcg_now(p + lane) : 0.f;
  const float v1 = lane + 32 < ns ? ldcg_now(p + lane + 32) : 0.f;
  return rsqrtf(warp_sum(v0 + v1) / a.d + a.eps);
}

// ---- stage: embedding (or residual add) + lazy RMSNorm operand -------------------------------------
// Work unit = (row, slice of 128 columns) per warp, 4 columns per lane; units are dealt round-robin over
// the CTAs first, so the whole stage is one pass with a few warps busy in every CTA.
// mode 0: h = E[cur_tok]; mode 1: h += projection (partials of shape `gs`).
__device__ void stage_residual(const MegaArgs& a, const MegaSmem* sm, int wtid, int mode, const MegaGemmShape* gs,
                               const bf16* __restrict__ gain, bool dump) {
  const int ns = (a.d + kRowSlice - 1) / kRowSlice;
  const int n_units = a.B * ns;
  const int lane = wtid & 31, wid = wtid >> 5;
  for (int u = wid * gridDim.x + blockIdx.x; u < n_units; u += 8 * gridDim.x) {
    const int r = u / ns, sl = u - r * ns;
    if (!sm->active_s[r]) continue;
    const int c = sl * kRowSlice + lane * 4;
    float ss = 0.f;
    if (c < a.d) {
      float v[4];
      if (mode == 0) {
        int tok = a.st.cur_tok[r];
        if (tok < 0 || tok >= a.V) tok = 0;
        const uint2 e = __ldg(reinterpret_cast<const uint2*>(a.embed + (size_t)tok * a.d + c));
        const float2 e0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.x));
        const float2 e1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&e.y));
        v[0] = e0.x; v[1] = e0.y; v[2] = e1.x; v[3] = e1.y;
      } else {
        const float4 h4 = __ldcg(reinterpret_cast<const float4*>(a.h + (size_t)r * a.d + c));
        sum_partials_cg<4, 12>(sm, a.partial, *gs, a.NT, c, r, v);
        v[0] += h4.x; v[1] += h4.y; v[2] += h4.z; v[3] += h4.w;
      }
      const uint2 gb = __ldg(reinterpret_cast<const uint2*>(gain + c));
      const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gb.x));
      const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gb.y));
      *reinterpret_cast<float4*>(a.h + (size_t)r * a.d + c) = make_float4(v[0], v[1], v[2], v[3]);
      if (dump && a.dump_hidden)
        *reinterpret_cast<float4*>(a.dump_hidden + (size_t)r * a.d + c) = make_float4(v[0], v[1], v[2], v[3]);
      __align__(8) bf16 xb[4];
      xb[0] = __float2bfloat16_rn(v[0] * g0.x); xb[1] = __float2bfloat16_rn(v[1] * g0.y);
      xb[2] = __float2bfloat16_rn(v[2] * g1.x); xb[3] = __float2bfloat16_rn(v[3] * g1.y);
      *reinterpret_cast<uint2*>(a.x + (size_t)r * a.d + c) = *reinterpret_cast<const uint2*>(xb);
      ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
    }
    ss = warp_sum(ss);
    if (lane == 0) a.rowss[(size_t)r * kMaxSlices + sl] = ss;
  }
}

// ---- helpers shared by the stages ----------------------------------------------------------------------
// 1/rms of every active row into shared memory: warp w takes rows w, w+8, ... (four rows' loads in flight).
// Split in two so that a stage can put its own loads in flight between the halves.
struct InvRmsLoads { float v[4][2]; };
__device__ __forceinline__ InvRmsLoads inv_rms_issue(const MegaArgs& a, const MegaSmem* sm, int r0, int lane) {
  const int ns = (a.d + kRowSlice - 1) / kRowSlice;        // <= 64: two slices per lane
  InvRmsLoads q;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int r = r0 + 8 * k;
    const bool on = r < a.B && sm->active_s[r];
    const float* p = a.rowss + (size_t)(on ? r : 0) * kMaxSlices;
    q.v[k][0] = (on && lane < ns) ? ldcg_now(p + lane) : 0.f;
    q.v[k][1] = (on && lane + 32 < ns) ? ldcg_now(p + lane + 32) : 0.f;
  }
  return q;
}
__device__ __forceinline__ void inv_rms_finish(const MegaArgs& a, MegaSmem* sm, const InvRmsLoads& q, int r0, int lane) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int r = r0 + 8 * k;
    const float t = warp_sum(q.v[k][0] + q.v[k][1]);
    if (r < a.B && lane == 0) sm->inv_s[r] = sm->active_s[r] ? rsqrtf(t / a.d + a.eps) : 0.f;
  }
}
__device__ __forceinline__ void stage_inv_rms(const MegaArgs& a, MegaSmem* sm, int wtid) {
  const int lane = wtid & 31, wid = wtid >> 5;
  for (int r0 = wid; r0 < a.B; r0 += 32) {
    const InvRmsLoads q = inv_rms_issue(a, sm, r0, lane);
    inv_rms_finish(a, sm, q, r0, lane);
  }
  named_bar_workers();
}

__device__ __forceinline__ void group_bar(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// ---- stage: q,k,v from partials + RoPE + cache append + paged attention ----------------------------------
// Work is dealt in units of (row, head, one batch of loads = kAttnU load steps of cached tokens: 16 tokens
// at head size 128, i.e. half a page).  Every CTA owns a contiguous run of (row, head) pairs holding
// about 1/gridDim of all units (pairs are not split across CTAs, so their partial results meet in shared
// memory).  A CTA works through its pairs in passes of up to 8:
//   A  warp j builds pair j's rotated query (shared memory) and the new token's k,v: appended to the
//      page, and entered as the pair's ninth partial (score, 1, v);
//   B  the pass's units are cut into 8 equal contiguous slices, one per warp; a warp scans its units
//      and leaves one (max, sum, acc) partial per pair it touched;
//   C  warp j merges pair j's partials and writes the bf16 output.
// Scan layout: a key row is Dh/8 chunks of 16 bytes; lane (g, gl) of the warp handles key g of the
// load step and chunks gl, gl+GROUP, gl+2*GROUP, gl+3*GROUP, so each warp-wide load reads 64
// contiguous bytes per key (full sectors).
constexpr int kAttnPass = 8;               // pairs per pass (= worker warps)
constexpr int kAttnU = 2;                  // load steps per work unit of the cache scan (one batch of loads in flight)
constexpr int kAttnSlots = 9;              // partials per pair: one per warp + the new token
constexpr int kAttnWarpPairsMin = 24;      // pairs in a CTA's run from which every warp takes whole pairs (at most 1/3 idle)

// Tables of the pass whose pair list is in shared memory: the new tokens' positions and pages, the ids of the first
// pages of every warp's slice of the scan (all requested together, so that the scan itself starts no chain of
// dependent look-ups), and -- with_rope, for a CTA whose pairs fit one pass: once per step -- the rotations.
template <int DH>
__device__ __forceinline__ void attention_pass_tables(const MegaArgs& a, MegaSmem* sm, int wtid, bool with_rope) {
  constexpr int EPL = DH / 32;
  constexpr int UT = kAttnU * (32 / (DH / 32));
  constexpr int UPP = kPageTokens / UT;
  const int lane = wtid & 31, wid = wtid >> 5;
  const int H = a.H;
  const int np = sm->pair_n, U = sm->pair_ustart[np];
  if (wid < np) {
    const int p = sm->pair_id[wid];
    const int r = p / H;
    const int pos = a.st.ctx_len[r];
    if (with_rope) {
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        float sn, cs;
        sincosf((float)pos * a.inv_freq[(lane & 15) * EPL + j], &sn, &cs);
        sm->rope_c[wid][lane * EPL + j] = cs;
        sm->rope_sn[wid][lane * EPL + j] = sn;
      }
    }
    if (lane == 0) {
      sm->pair_pos[wid] = pos;
      sm->pair_pgnew[wid] = a.st.block_table[(size_t)r * a.st.max_pages + pos / kPageTokens];
    }
  }
  // page ids of the first (up to 8) distinct pages of this warp's slice, in scan order
  const int u0 = (int)((long long)wid * U / 8), u1 = (int)((long long)(wid + 1) * U / 8);
  const int u = u0 + lane;
  int j = 0, ui = 0;
  bool newpage = false;
  if (u < u1) {
    while (j + 1 < np && sm->pair_ustart[j + 1] <= u) ++j;
    ui = u - sm->pair_ustart[j];
    newpage = lane == 0 || ui % UPP == 0;
  }
  const unsigned int starts = __ballot_sync(0xffffffffu, newpage);
  const int ord = __popc(starts & (0xffffffffu >> (31 - lane))) - 1;
  if (newpage && ord < 8)
    sm->unit_pg[wid][ord] = a.st.block_table[(size_t)(sm->pair_id[j] / H) * a.st.max_pages + ui / UPP];
}

// Once per step (the lengths do not change between layers): units per row, this CTA's run of pairs, and --
// when the run fits one pass -- the pass list, the new tokens' positions/pages/rotations and the ids of
// the first pages of every warp's slice.
template <int DH, bool WIDE>
__device__ void attention_setup(const MegaArgs& a, MegaSmem* sm, int wtid) {
  constexpr int UT = kAttnU * (32 / (DH / 32));   // cached tokens per work unit (16 at Dh 128, 32 at Dh 64)
  const int lane = wtid & 31, wid = wtid >> 5;
  const int H = a.H, B = a.B;
  // ---- per-step copies in shared memory: which rows are active, and the per-layer tile tables
  for (int r = wtid; r < kMaxBatch; r += kMegaWorkers) sm->active_s[r] = (r < B && a.st.active[r]) ? 1 : 0;
  for (int t = 0; t < 4; ++t) {
    const MegaGemmShape& gs = a.shape[t];
    if (gs.smem_off < 0) continue;
    for (int i = wtid; i < gs.n_tiles; i += kMegaWorkers)
      sm->seg_tab[gs.smem_off + i] = __ldg(reinterpret_cast<const int4*>(gs.tiles) + i);
  }
  // ---- pages per row (exclusive prefix, active rows only) and this CTA's run of pairs
  if (wid == 0) {
    int cnt[8], loc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int r = lane * 8 + j;
      int c = 0;
      if (r < B && a.st.active[r]) c = (a.st.ctx_len[r] + UT - 1) / UT;
      cnt[j] = c;
      loc += c;
    }
    int inc = loc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += t;
    }
    int run = inc - loc;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      sm->prefix[lane * 8 + j] = run;
      run += cnt[j];
    }
    if (lane == 31) sm->prefix[kMaxBatch] = inc;
    if (lane == 0) { sm->pair_lo = 0x7fffffff; sm->pair_hi = -1; }
  }
  named_bar_workers();
  {
    const long long T = (long long)sm->prefix[kMaxBatch] * H;        // all units
    const long long lo = (long long)blockIdx.x * T / gridDim.x, hi = (long long)(blockIdx.x + 1) * T / gridDim.x;
    int mylo = 0x7fffffff, myhi = -1;
    for (int p = wtid; p < B * H; p += kMegaWorkers) {
      const int r = p / H, hd = p - r * H;
      const int npr = sm->prefix[r + 1] - sm->prefix[r];     // pages of this row (0 if inactive)
      if (npr <= 0) continue;
      const long long cum = (long long)sm->prefix[r] * H + (long long)hd * npr;   // units before this pair
      if (cum >= lo && cum < hi) { mylo = min(mylo, p); myhi = max(myhi, p); }
    }
    if (mylo <= myhi) { atomicMin(&sm->pair_lo, mylo); atomicMax(&sm->pair_hi, myhi); }
  }
  named_bar_workers();
  const int p_begin = sm->pair_lo, p_end = sm->pair_hi + 1;
  if (wid == 0) {
    int n = 0, p = p_begin, ustart = 0;
    while (p < p_end && n < kAttnPass) {
      const int r = p / H;
      const int npr = sm->prefix[r + 1] - sm->prefix[r];
      if (npr <= 0) { p = (r + 1) * H; continue; }
      if (lane == 0) { sm->pair_id[n] = p; sm->pair_ustart[n] = ustart; }
      ustart += npr;
      ++n;
      ++p;
    }
    // any pair with work left beyond the first eight?
    bool more = false;
    for (int q = p; q < p_end && !more; ) {
      const int r = q / H;
      if (sm->prefix[r + 1] - sm->prefix[r] > 0) more = true; else q = (r + 1) * H;
    }
    if (lane == 0) { sm->pair_n = n; sm->pair_next = p; sm->pair_ustart[n] = ustart; sm->att_single = more ? 0 : 1; }
    if constexpr (WIDE) {
      // pairs with work in the whole run
      int cnt = 0;
      for (int q = p_begin; q < p_end; ) {
        const int r = q / H;
        const int e = min(p_end, (r + 1) * H);
        if (sm->prefix[r + 1] - sm->prefix[r] > 0) cnt += e - q;
        q = e;
      }
      if (lane == 0) sm->att_warp_pairs = cnt >= kAttnWarpPairsMin ? 1 : 0;
    }
  }
  named_bar_workers();
  if (sm->att_single) attention_pass_tables<DH>(a, sm, wtid, true);
  named_bar_workers();
}

// ---- pieces of the attention stage, each run by one warp, as attention_warp_pairs puts them together ----------
// (stage_attention below has the same steps written out in place: it is the path of the small batches, and its
// register allocation is what the whole kernel's speed hangs on)
template <int DH> struct AttnLayout {
  static constexpr int GROUP = DH / 32;           // lanes per key in the cache scan
  static constexpr int KPW = 32 / GROUP;          // keys per warp-wide load step
  static constexpr int EPL = DH / 32;             // cooperative layout: consecutive dimensions per lane
  static constexpr int U = kAttnU;                // load steps per work unit: one batch of loads
  static constexpr int UPP = kPageTokens / (U * KPW);   // units per page (2 at Dh 128, 1 at Dh 64)
};

// A: the pair's rotated, scaled query into qs[DH]; the new token's k, v appended to page pg at position pos and
// entered as the partial ns[DH + 2] = (v, score, 1).  cs / sn: the rotation of this lane's dimensions.
template <int DH>
__device__ __forceinline__ void attn_prepare_pair(const MegaArgs& a, const MegaSmem* sm, int layer, int lane, int r, int hd, int pos,
                                                  int pg, const float (&cs)[DH / 32], const float (&sn)[DH / 32], float* qs, float* ns) {
  constexpr int EPL = AttnLayout<DH>::EPL;
  const int H = a.H, d = a.d;
  const MegaGemmShape& gs = a.shape[0];
  const float qscale = rsqrtf((float)DH) * 1.4426950408889634f;
  const size_t v_off = (size_t)H * kPageTokens * DH;
  const float inv = warp_row_inv_rms(a, r, lane);
  const int e0 = lane * EPL;
  float qx[EPL], kx[EPL], vx[EPL];
  {
    const int nq = hd * DH + e0, nk = d + nq, nv = 2 * d + nq;
    const int4 tq = tile_seg(sm, gs, nq), tk = tile_seg(sm, gs, nk), tv = tile_seg(sm, gs, nv);
    PartialLoads<EPL, 4> lq, lk, lv;
    partials_issue<EPL, 4>(a.partial, gs, a.NT, tq, nq, r, lq);
    partials_issue<EPL, 4>(a.partial, gs, a.NT, tk, nk, r, lk);
    partials_issue<EPL, 4>(a.partial, gs, a.NT, tv, nv, r, lv);
    partials_sum<EPL, 4>(a.partial, gs, a.NT, tq, nq, r, lq, qx);
    partials_sum<EPL, 4>(a.partial, gs, a.NT, tk, nk, r, lk, kx);
    partials_sum<EPL, 4>(a.partial, gs, a.NT, tv, nv, r, lv, vx);
  }
  if (pg < 0 || pg >= a.kv.n_pages) { atomicCAS(a.status, 0u, (uint32_t)kStatusBadPage); pg = -1; }
  bf16* kdst = a.kv.pool + (size_t)layer * a.kv.layer_stride + (size_t)(pg < 0 ? 0 : pg) * a.kv.page_elems +
               ((size_t)hd * kPageTokens + (pos % kPageTokens)) * DH + e0;
  float dot = 0.f;
#pragma unroll
  for (int j = 0; j < EPL; ++j) {
    const float xq = qx[j] * inv, xk = kx[j] * inv;
    const float pq = __shfl_xor_sync(0xffffffffu, xq, 16), pk = __shfl_xor_sync(0xffffffffu, xk, 16);
    const float oq = (lane < 16) ? xq * cs[j] - pq * sn[j] : xq * cs[j] + pq * sn[j];
    const float ok = (lane < 16) ? xk * cs[j] - pk * sn[j] : xk * cs[j] + pk * sn[j];
    const float qf = oq * qscale;                     // the query is only ever an ALU operand: it stays fp32
    const bf16 kb16 = __float2bfloat16_rn(ok), vb16 = __float2bfloat16_rn(vx[j] * inv);
    if (pg >= 0) { kdst[j] = kb16; kdst[v_off + j] = vb16; }
    qs[e0 + j] = qf;
    ns[e0 + j] = __bfloat162float(vb16);
    dot += qf * __bfloat162float(kb16);
  }
  dot = warp_sum(dot);
  if (lane == 0) { ns[DH] = dot; ns[DH + 1] = 1.f; }
}

// B: one unit (U load steps of KPW keys; kb = first key of the page's head, s0 = first load step, tcount = the
// page's tokens) folded into the running (m, l, acc) of the lane's key slot.
template <int DH>
__device__ __forceinline__ void attn_scan_unit(const bf16* __restrict__ kb, size_t v_off, int s0, int tcount, const float* qs, int g, int gl,
                                               float& m, float& l, float (&acc)[32]) {
  constexpr int GROUP = AttnLayout<DH>::GROUP, KPW = AttnLayout<DH>::KPW, U = AttnLayout<DH>::U;
  uint4 kk[U][4], vv[U][4];
#pragma unroll
  for (int uu = 0; uu < U; ++uu) {
    const int t = (s0 + uu) * KPW + g;
    if (t < tcount) {
      const uint4* kp = reinterpret_cast<const uint4*>(kb + (size_t)t * DH);
      const uint4* vp = reinterpret_cast<const uint4*>(kb + (size_t)t * DH + v_off);
#pragma unroll
      for (int c = 0; c < 4; ++c) { kk[uu][c] = __ldg(kp + c * GROUP + gl); vv[uu][c] = __ldg(vp + c * GROUP + gl); }
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c) { kk[uu][c] = make_uint4(0, 0, 0, 0); vv[uu][c] = kk[uu][c]; }
    }
  }
  float sc_[U];
#pragma unroll
  for (int uu = 0; uu < U; ++uu) {
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float kf[8];
      unpack8(kk[uu][c], kf);
      const float4 qa = *reinterpret_cast<const float4*>(qs + (c * GROUP + gl) * 8);
      const float4 qb = *reinterpret_cast<const float4*>(qs + (c * GROUP + gl) * 8 + 4);
      dot += qa.x * kf[0] + qa.y * kf[1] + qa.z * kf[2] + qa.w * kf[3] + qb.x * kf[4] + qb.y * kf[5] +
             qb.z * kf[6] + qb.w * kf[7];
    }
#pragma unroll
    for (int o = GROUP / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    sc_[uu] = ((s0 + uu) * KPW + g < tcount) ? dot : -CUDART_INF_F;
  }
  float mn = m;
#pragma unroll
  for (int uu = 0; uu < U; ++uu) mn = fmaxf(mn, sc_[uu]);
  if (mn != -CUDART_INF_F) {
    if (mn != m) {
      const float sc = exp2f(m - mn);
      l *= sc;
#pragma unroll
      for (int e = 0; e < 32; ++e) acc[e] *= sc;
      m = mn;
    }
#pragma unroll
    for (int uu = 0; uu < U; ++uu) {
      if (sc_[uu] != -CUDART_INF_F) {
        const float pw = exp2f(sc_[uu] - mn);
        l += pw;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float vf[8];
          unpack8(vv[uu][c], vf);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[c * 8 + e] += pw * vf[e];
        }
      }
    }
  }
}

// The warp's KPW key slots merged, the result stored as the partial slot[DH + 2] = (acc, m, l); (m, l, acc) reset.
template <int DH>
__device__ __forceinline__ void attn_flush(float* slot, int g, int gl, float& m, float& l, float (&acc)[32]) {
  constexpr int GROUP = AttnLayout<DH>::GROUP;
#pragma unroll
  for (int o = GROUP; o < 32; o <<= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const float ol = __shfl_xor_sync(0xffffffffu, l, o);
    const float mn = fmaxf(m, om);
    const float w0 = (m == -CUDART_INF_F) ? 0.f : exp2f(m - mn);
    const float w1 = (om == -CUDART_INF_F) ? 0.f : exp2f(om - mn);
    l = l * w0 + ol * w1;
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const float oa = __shfl_xor_sync(0xffffffffu, acc[e], o);
      acc[e] = acc[e] * w0 + oa * w1;
    }
    m = mn;
  }
  if (g == 0) {
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int e = 0; e < 8; ++e) slot[(c * GROUP + gl) * 8 + e] = acc[c * 8 + e];
    if (gl == 0) { slot[DH] = m; slot[DH + 1] = l; }
  }
  m = -CUDART_INF_F;
  l = 0.f;
#pragma unroll
  for (int e = 0; e < 32; ++e) acc[e] = 0.f;
}

// C: the pair's partials slots[0 .. kAttnSlots) merged and written as bf16 output of (row r, head hd).
template <int DH>
__device__ __forceinline__ void attn_merge_pair(const MegaArgs& a, const float (*slots)[132], int lane, int r, int hd) {
  constexpr int EPL = AttnLayout<DH>::EPL;
  const int e0 = lane * EPL;
  float M = -CUDART_INF_F;
  for (int k = 0; k < kAttnSlots; ++k) M = fmaxf(M, slots[k][DH]);
  float L = 0.f, A[EPL];
#pragma unroll
  for (int j = 0; j < EPL; ++j) A[j] = 0.f;
  for (int k = 0; k < kAttnSlots; ++k) {
    const float mk = slots[k][DH];
    if (mk == -CUDART_INF_F) continue;
    const float wt = exp2f(mk - M);
    L += slots[k][DH + 1] * wt;
#pragma unroll
    for (int j = 0; j < EPL; ++j) A[j] += slots[k][e0 + j] * wt;
  }
  const float il = 1.f / L;
#pragma unroll
  for (int j = 0; j < EPL; ++j) a.o[(size_t)r * a.d + hd * DH + e0 + j] = __float2bfloat16_rn(A[j] * il);
}

// Wide batches, where a CTA's run has many pairs: every warp takes whole pairs (the run's pairs with work, in turn)
// and does all three steps for them by itself, so nothing is shared between the warps and nothing holds them in
// step: while one warp builds a query, the others' loads are in flight.  The pair's page ids are looked up by the
// lanes together (lane i: pages i and i + 32) and handed out by shuffle.
template <int DH>
__device__ void attention_warp_pairs(const MegaArgs& a, MegaSmem* sm, int wtid, int layer) {
  using L = AttnLayout<DH>;
  constexpr int GROUP = L::GROUP, EPL = L::EPL, U = L::U, UPP = L::UPP;
  const int lane = wtid & 31, wid = wtid >> 5;
  const int gl = lane % GROUP, g = lane / GROUP;
  const int H = a.H;
  const bf16* kv_layer = a.kv.pool + (size_t)layer * a.kv.layer_stride;
  const size_t v_off = (size_t)H * kPageTokens * DH;
  const int p_begin = sm->pair_lo, p_end = sm->pair_hi + 1;
  float (*slots)[132] = sm->att_s[wid];
  float* qs = sm->q_s[wid];
  int n = 0;
  for (int p = p_begin; p < p_end; ) {
    const int r = p / H;
    const int npr = sm->prefix[r + 1] - sm->prefix[r];
    if (npr <= 0) { p = (r + 1) * H; continue; }
    if ((n++ & 7) != wid) { ++p; continue; }
    const int hd = p - r * H;
    const int pos = a.st.ctx_len[r];
    const int last_page = pos / kPageTokens;            // the new token's page
    const int32_t* bt = a.st.block_table + (size_t)r * a.st.max_pages;
    const int pgs0 = lane <= last_page ? bt[lane] : 0;
    const int pgs1 = lane + 32 <= last_page ? bt[lane + 32] : 0;
    if (lane < kAttnSlots) slots[lane][DH] = -CUDART_INF_F;
    float sn[EPL], cs[EPL];
#pragma unroll
    for (int j = 0; j < EPL; ++j) sincosf((float)pos * a.inv_freq[(lane & 15) * EPL + j], &sn[j], &cs[j]);
    const int pg_new = last_page < 32 ? __shfl_sync(0xffffffffu, pgs0, last_page)
                                      : (last_page < 64 ? __shfl_sync(0xffffffffu, pgs1, last_page - 32) : bt[last_page]);
    __syncwarp();
    attn_prepare_pair<DH>(a, sm, layer, lane, r, hd, pos, pg_new, cs, sn, qs, slots[kAttnSlots - 1]);
    __syncwarp();
    float m = -CUDART_INF_F, l = 0.f, acc[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) acc[e] = 0.f;
    int pg = 0;
    for (int ui = 0; ui < npr; ++ui) {
      const int pi = ui / UPP;
      if (ui % UPP == 0) {
        pg = pi < 32 ? __shfl_sync(0xffffffffu, pgs0, pi) : (pi < 64 ? __shfl_sync(0xffffffffu, pgs1, pi - 32) : bt[pi]);
        if (pg < 0 || pg >= a.kv.n_pages) { atomicCAS(a.status, 0u, (uint32_t)kStatusBadPage); pg = 0; }
      }
      const int tcount = min(kPageTokens, pos - pi * kPageTokens);
      const bf16* kb = kv_layer + (size_t)pg * a.kv.page_elems + (size_t)hd * kPageTokens * DH;
      attn_scan_unit<DH>(kb, v_off, (ui % UPP) * U, tcount, qs, g, gl, m, l, acc);
    }
    attn_flush<DH>(slots[0], g, gl, m, l, acc);
    __syncwarp();
    attn_merge_pair<DH>(a, slots, lane, r, hd);
    __syncwarp();
    ++p;
  }
}

template <int DH>
__device__ void stage_attention(const MegaArgs& a, MegaSmem* sm, int wtid, int layer) {
  constexpr int GROUP = DH / 32;           // lanes per key in the cache scan
  constexpr int KPW = 32 / GROUP;          // keys per warp-wide load step
  constexpr int EPL = DH / 32;             // cooperative layout: consecutive dimensions per lane
  constexpr int U = kAttnU;                // load steps per work unit: one batch of loads
  constexpr int UPP = kPageTokens / (U * KPW);   // units per page (2 at Dh 128, 1 at Dh 64)
  const int lane = wtid & 31, wid = wtid >> 5;
  const int gl = lane % GROUP, g = lane / GROUP;
  const int H = a.H, d = a.d;
  const MegaGemmShape& gs = a.shape[0];
  const float qscale = rsqrtf((float)DH) * 1.4426950408889634f;
  const bf16* kv_layer = a.kv.pool + (size_t)layer * a.kv.layer_stride;
  const size_t v_off = (size_t)H * kPageTokens * DH;

  const int p_begin = sm->pair_lo, p_end = sm->pair_hi + 1;          // empty run: lo > hi
  const bool single = sm->att_single != 0;

  for (int pass0 = p_begin; pass0 < p_end; ) {
    // ---- the pass: next (up to 8) pairs with work; pair_id / pair_pages / pair_ustart in shared memory
    if (wid == 0 && !single) {
      int n = 0, p = pass0, ustart = 0;
      // lanes walk the pairs together (few iterations: rows without work are skipped by whole rows)
      while (p < p_end && n < kAttnPass) {
        const int r = p / H;
        const int npr = sm->prefix[r + 1] - sm->prefix[r];
        if (npr <= 0) { p = (r + 1) * H; continue; }
        if (lane == 0) { sm->pair_id[n] = p; sm->pair_ustart[n] = ustart; }
        ustart += npr;
        ++n;
        ++p;
      }
      if (lane == 0) { sm->pair_n = n; sm->pair_next = p; sm->pair_ustart[n] = ustart; }
    }
    for (int i = wtid; i < kAttnPass * kAttnSlots; i += kMegaWorkers) sm->att_s[i / kAttnSlots][i % kAttnSlots][DH] = -CUDART_INF_F;
    named_bar_workers();
    if (!single) {
      // positions and page ids of this pass, looked up together (a CTA with one pass did this once per step)
      attention_pass_tables<DH>(a, sm, wtid, false);
      named_bar_workers();
    }
    const int np_pass = sm->pair_n;
    const int U_pass = sm->pair_ustart[np_pass];

    // ---- A: warp j prepares pair j
    if (wid < np_pass) {
      const int p = sm->pair_id[wid];
      const int r = p / H, hd = p - r * H;
      const int pos = sm->pair_pos[wid];
      const float inv = warp_row_inv_rms(a, r, lane);
      const int e0 = lane * EPL;
      float sn[EPL], cs[EPL];
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        if (single) { cs[j] = sm->rope_c[wid][e0 + j]; sn[j] = sm->rope_sn[wid][e0 + j]; }
        else sincosf((float)pos * a.inv_freq[(lane & 15) * EPL + j], &sn[j], &cs[j]);
      }
      float qx[EPL], kx[EPL], vx[EPL];
      {
        const int nq = hd * DH + e0, nk = d + nq, nv = 2 * d + nq;
        const int4 tq = tile_seg(sm, gs, nq), tk = tile_seg(sm, gs, nk), tv = tile_seg(sm, gs, nv);
        PartialLoads<EPL, 4> lq, lk, lv;
        partials_issue<EPL, 4>(a.partial, gs, a.NT, tq, nq, r, lq);
        partials_issue<EPL, 4>(a.partial, gs, a.NT, tk, nk, r, lk);
        partials_issue<EPL, 4>(a.partial, gs, a.NT, tv, nv, r, lv);
        partials_sum<EPL, 4>(a.partial, gs, a.NT, tq, nq, r, lq, qx);
        partials_sum<EPL, 4>(a.partial, gs, a.NT, tk, nk, r, lk, kx);
        partials_sum<EPL, 4>(a.partial, gs, a.NT, tv, nv, r, lv, vx);
      }
      int pg = sm->pair_pgnew[wid];
      if (pg < 0 || pg >= a.kv.n_pages) { atomicCAS(a.status, 0u, (uint32_t)kStatusBadPage); pg = -1; }
      bf16* kdst = a.kv.pool + (size_t)layer * a.kv.layer_stride + (size_t)(pg < 0 ? 0 : pg) * a.kv.page_elems +
                   ((size_t)hd * kPageTokens + (pos % kPageTokens)) * DH + e0;
      float dot = 0.f;
      float* qs = sm->q_s[wid];
      float* ns = sm->att_s[wid][kAttnSlots - 1];
#pragma unroll
      for (int j = 0; j < EPL; ++j) {
        const float xq = qx[j] * inv, xk = kx[j] * inv;
        const float pq = __shfl_xor_sync(0xffffffffu, xq, 16), pk = __shfl_xor_sync(0xffffffffu, xk, 16);
        const float oq = (lane < 16) ? xq * cs[j] - pq * sn[j] : xq * cs[j] + pq * sn[j];
        const float ok = (lane < 16) ? xk * cs[j] - pk * sn[j] : xk * cs[j] + pk * sn[j];
        const float qf = oq * qscale;                     // the query is only ever an ALU operand: it stays fp32
        const bf16 kb16 = __float2bfloat16_rn(ok), vb16 = __float2bfloat16_rn(vx[j] * inv);
        if (pg >= 0) { kdst[j] = kb16; kdst[v_off + j] = vb16; }
        qs[e0 + j] = qf;
        ns[e0 + j] = __bfloat162float(vb16);
        dot += qf * __bfloat162float(kb16);
      }
      dot = warp_sum(dot);
      if (lane == 0) { ns[DH] = dot; ns[DH + 1] = 1.f; }
    }
    named_bar_workers();

    // ---- B: this warp's slice of the pass's units
    {
      const int u0 = (int)((long long)wid * U_pass / 8), u1 = (int)((long long)(wid + 1) * U_pass / 8);
      int j = 0;
      while (j + 1 < np_pass && sm->pair_ustart[j + 1] <= u0) ++j;
      float m = -CUDART_INF_F, l = 0.f, acc[32];
#pragma unroll
      for (int e = 0; e < 32; ++e) acc[e] = 0.f;
      auto flush = [&](int jj) {
        // merge the KPW key slots of the warp, then lanes of key slot 0 store the partial
#pragma unroll
        for (int o = GROUP; o < 32; o <<= 1) {
          const float om = __shfl_xor_sync(0xffffffffu, m, o);
          const float ol = __shfl_xor_sync(0xffffffffu, l, o);
          const float mn = fmaxf(m, om);
          const float w0 = (m == -CUDART_INF_F) ? 0.f : exp2f(m - mn);
          const float w1 = (om == -CUDART_INF_F) ? 0.f : exp2f(om - mn);
          l = l * w0 + ol * w1;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float oa = __shfl_xor_sync(0xffffffffu, acc[e], o);
            acc[e] = acc[e] * w0 + oa * w1;
          }
          m = mn;
        }
        float* slot = sm->att_s[jj][wid];
        if (g == 0) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 8; ++e) slot[(c * GROUP + gl) * 8 + e] = acc[c * 8 + e];
          if (gl == 0) { slot[DH] = m; slot[DH + 1] = l; }
        }
        m = -CUDART_INF_F;
        l = 0.f;
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
      };
      int kpage = -1, pg = 0;                            // ordinal of the current page in this slice, its id
      for (int u = u0; u < u1; ++u) {
        if (u >= sm->pair_ustart[j + 1]) { flush(j); ++j; }
        const int p = sm->pair_id[j];
        const int r = p / H, hd = p - r * H;
        const int ui = u - sm->pair_ustart[j];           // unit of the pair: page ui / UPP, batch ui % UPP of it
        const int pi = ui / UPP;
        const int pos = sm->pair_pos[j];
        if (u == u0 || ui % UPP == 0) {
          ++kpage;
          pg = kpage < 8 ? sm->unit_pg[wid][kpage] : a.st.block_table[(size_t)r * a.st.max_pages + pi];
          if (pg < 0 || pg >= a.kv.n_pages) { atomicCAS(a.status, 0u, (uint32_t)kStatusBadPage); pg = 0; }
        }
        const int tcount = min(kPageTokens, pos - pi * kPageTokens);
        const bf16* kb = kv_layer + (size_t)pg * a.kv.page_elems + (size_t)hd * kPageTokens * DH;
        const float* qs = sm->q_s[j];
        {
          const int s0 = (ui % UPP) * U;
          uint4 kk[U][4], vv[U][4];
#pragma unroll
          for (int uu = 0; uu < U; ++uu) {
            const int t = (s0 + uu) * KPW + g;
            if (t < tcount) {
              const uint4* kp = reinterpret_cast<const uint4*>(kb + (size_t)t * DH);
              const uint4* vp = reinterpret_cast<const uint4*>(kb + (size_t)t * DH + v_off);
#pragma unroll
              for (int c = 0; c < 4; ++c) { kk[uu][c] = __ldg(kp + c * GROUP + gl); vv[uu][c] = __ldg(vp + c * GROUP + gl); }
            } else {
#pragma unroll
              for (int c = 0; c < 4; ++c) { kk[uu][c] = make_uint4(0, 0, 0, 0); vv[uu][c] = kk[uu][c]; }
            }
          }
          float sc_[U];
#pragma unroll
          for (int uu = 0; uu < U; ++uu) {
            float dot = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              float kf[8];
              unpack8(kk[uu][c], kf);
              const float4 qa = *reinterpret_cast<const float4*>(qs + (c * GROUP + gl) * 8);
              const float4 qb = *reinterpret_cast<const float4*>(qs + (c * GROUP + gl) * 8 + 4);
              dot += qa.x * kf[0] + qa.y * kf[1] + qa.z * kf[2] + qa.w * kf[3] + qb.x * kf[4] + qb.y * kf[5] +
                     qb.z * kf[6] + qb.w * kf[7];
            }
#pragma unroll
            for (int o = GROUP / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            sc_[uu] = ((s0 + uu) * KPW + g < tcount) ? dot : -CUDART_INF_F;
          }
          float mn = m;
#pragma unroll
          for (int uu = 0; uu < U; ++uu) mn = fmaxf(mn, sc_[uu]);
          if (mn != -CUDART_INF_F) {
            if (mn != m) {
              const float sc = exp2f(m - mn);
              l *= sc;
#pragma unroll
              for (int e = 0; e < 32; ++e) acc[e] *= sc;
              m = mn;
            }
#pragma unroll
            for (int uu = 0; uu < U; ++uu) {
              if (sc_[uu] != -CUDART_INF_F) {
                const float pw = exp2f(sc_[uu] - mn);
                l += pw;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                  float vf[8];
                  unpack8(vv[uu][c], vf);
#pragma unroll
                  for (int e = 0; e < 8; ++e) acc[c * 8 + e] += pw * vf[e];
                }
              }
            }
          }
        }
      }
      if (u1 > u0) flush(j);
    }
    named_bar_workers();

    // ---- C: warp j merges pair j
    if (wid < np_pass) {
      const int p = sm->pair_id[wid];
      const int r = p / H, hd = p - r * H;
      const int e0 = lane * EPL;
      float M = -CUDART_INF_F;
      for (int k = 0; k < kAttnSlots; ++k) M = fmaxf(M, sm->att_s[wid][k][DH]);
      float L = 0.f, A[EPL];
#pragma unroll
      for (int j = 0; j < EPL; ++j) A[j] = 0.f;
      for (int k = 0; k < kAttnSlots; ++k) {
        const float mk = sm->att_s[wid][k][DH];
        if (mk == -CUDART_INF_F) continue;
        const float wt = exp2f(mk - M);
        L += sm->att_s[wid][k][DH + 1] * wt;
#pragma unroll
        for (int j = 0; j < EPL; ++j) A[j] += sm->att_s[wid][k][e0 + j] * wt;
      }
      const float il = 1.f / L;
#pragma unroll
      for (int j = 0; j < EPL; ++j) a.o[(size_t)r * d + hd * DH + e0 + j] = __float2bfloat16_rn(A[j] * il);
    }
    pass0 = single ? p_end : sm->pair_next;       // a single pass covers the whole run
    named_bar_workers();
  }
}

// ---- stage: SwiGLU ----------------------------------------------------------------------------------
// 8 consecutive features per thread (two 128-bit loads per partial segment, one 128-bit store).  The loads
// for 1/rms and the first unit's partials are in flight together.
__device__ __forceinline__ void gate_up_sums(const MegaArgs& a, const MegaSmem* sm, const MegaGemmShape& gs, int f0, int r, float (&gt)[8],
                                             float (&up)[8]) {
  const int4 tg = tile_seg(sm, gs, f0), tu = tile_seg(sm, gs, a.F + f0);
  PartialLoads<8, 2> qg, qu;
  partials_issue<8, 2>(a.partial, gs, a.NT, tg, f0, r, qg);
  partials_issue<8, 2>(a.partial, gs, a.NT, tu, a.F + f0, r, qu);
  partials_sum<8, 2>(a.partial, gs, a.NT, tg, f0, r, qg, gt);
  partials_sum<8, 2>(a.partial, gs, a.NT, tu, a.F + f0, r, qu, up);
}

__device__ void stage_swiglu(const MegaArgs& a, MegaSmem* sm, int wtid) {
  const MegaGemmShape& gs = a.shape[2];
  const int lane = wtid & 31, wid = wtid >> 5;
  const int F8 = a.F >> 3;
  const long long n = (long long)a.B * F8, stride = (long long)gridDim.x * kMegaWorkers;
  long long e = (long long)blockIdx.x * kMegaWorkers + wtid;
  const InvRmsLoads q = inv_rms_issue(a, sm, wid, lane);
  float gt[8], up[8];
  int r = 0, f0 = 0;
  bool have = false;
  if (e < n) {
    r = (int)(e / F8);
    f0 = (int)(e - (long long)r * F8) << 3;
    have = sm->active_s[r] != 0;
    if (have) gate_up_sums(a, sm, gs, f0, r, gt, up);
  }
  inv_rms_finish(a, sm, q, wid, lane);
  for (int r0 = wid + 32; r0 < a.B; r0 += 32) {
    const InvRmsLoads q2 = inv_rms_issue(a, sm, r0, lane);
    inv_rms_finish(a, sm, q2, r0, lane);
  }
  named_bar_workers();
  for (;;) {
    if (have) {
      const float inv = sm->inv_s[r];
      __align__(16) bf16 ob[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float gv = gt[j] * inv;
        ob[j] = __float2bfloat16_rn(__fdividef(gv, 1.f + __expf(-gv)) * (up[j] * inv));
      }
      *reinterpret_cast<uint4*>(a.act + (size_t)r * a.F + f0) = *reinterpret_cast<const uint4*>(ob);
    }
    e += stride;
    if (e >= n) break;
    r = (int)(e / F8);
    f0 = (int)(e - (long long)r * F8) << 3;
    have = sm->active_s[r] != 0;
    if (have) gate_up_sums(a, sm, gs, f0, r, gt, up);
  }
}

// ---- stage: per-tile arg-max of the logits --------------------------------------------------------------
// One vocabulary tile per half of the workers (128 threads = the tile's rows).
__device__ void stage_tile_argmax(const MegaArgs& a, MegaSmem* sm, int wtid) {
  const MegaGemmShape& gs = a.shape[4];
  const int half_id = wtid >> 7, t128 = wtid & 127, lane = wtid & 31, w4 = t128 >> 5;
  // scratch [tile half][4 warps][64 batch rows] of keys, then of ids, in the attention partials' space
  uint32_t* s_key = reinterpret_cast<uint32_t*>(&sm->att_s[0][0][0]) + half_id * 256;
  int* s_id = reinterpret_cast<int*>(&sm->att_s[0][0][0]) + 512 + half_id * 256;
  stage_inv_rms(a, sm, wtid);
  const size_t slot_stride = (size_t)a.NT * kTileN, cta_stride = slot_stride * gs.max_seg;
  for (int tile0 = blockIdx.x * 2; tile0 < a.n_tiles_lm; tile0 += gridDim.x * 2) {
    const int tile = tile0 + half_id;                   // 128 vocabulary rows: one half of a 256-row GEMM tile
    const bool tile_ok = tile < a.n_tiles_lm;
    const int v = tile * 128 + t128;
    int4 ts = make_int4(0, 1, 0, 0);
    if (tile_ok) ts = tile_seg(sm, gs, v);
    for (int rb = 0; rb < a.B; rb += 64) {              // 64 batch rows at a time (scratch holds 4 x 64 per half)
      const int rend = min(a.B, rb + 64);
      for (int r0 = rb; r0 < rend; r0 += 8) {           // 8 rows' partial loads in flight together
        float x0[8], x1[8], x2[8];
        const size_t col = (size_t)(v % kTileN);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = r0 + j;
          const bool on = tile_ok && r < rend && sm->active_s[r] && v < a.V;
          const size_t off = (size_t)(on ? r : 0) * kTileN + col;
          x0[j] = on ? __ldcg(a.partial + (size_t)ts.x * slot_stride + off) : 0.f;
          x1[j] = (on && ts.y <= ts.z) ? __ldcg(a.partial + (size_t)ts.y * cta_stride + off) : 0.f;
          x2[j] = (on && ts.y + 1 <= ts.z) ? __ldcg(a.partial + (size_t)(ts.y + 1) * cta_stride + off) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = r0 + j;
          if (r >= rend) break;                           // uniform over the CTA
          uint32_t key = 0;
          if (tile_ok && sm->active_s[r] && v < a.V) {
            float lg = x0[j] + x1[j] + x2[j];             // CTA order: slot0, c_next, c_next + 1, ...
            const size_t off = (size_t)r * kTileN + col;
            for (int c = ts.y + 2; c <= ts.z; ++c) lg += __ldcg(a.partial + (size_t)c * cta_stride + off);
            lg *= sm->inv_s[r];
            if (a.dump_logits) a.dump_logits[(size_t)r * a.V + v] = lg;
            if (!(a.st.eos_at[r] > 0 && v == a.eos_id))
              key = float_order_key(decision_value(lg, a.sample, v, a.st.gen[r] + 1, a.st.row_key[r]));
          }
          const uint32_t best = __reduce_max_sync(0xffffffffu, key);
          const uint32_t who = __ballot_sync(0xffffffffu, key == best);
          if (lane == 0) {
            s_key[w4 * 64 + (r - rb)] = best;
            s_id[w4 * 64 + (r - rb)] = tile * 128 + w4 * 32 + (__ffs(who) - 1);
          }
        }
      }
      named_bar_workers();
      if (tile_ok) {
        for (int r = rb + t128; r < rend; r += 128) {
          if (!sm->active_s[r]) continue;
          uint32_t bk = s_key[r - rb];
          int bi = s_id[r - rb];
#pragma unroll
          for (int w = 1; w < 4; ++w)
            if (s_key[w * 64 + (r - rb)] > bk) { bk = s_key[w * 64 + (r - rb)]; bi = s_id[w * 64 + (r - rb)]; }
          a.tile_val[(size_t)r * a.n_tiles_lm + tile] = __uint_as_float(bk);
          a.tile_idx[(size_t)r * a.n_tiles_lm + tile] = bi;
        }
      }
      named_bar_workers();
    }
  }
}

// ---- stage: final arg-max over tiles + row bookkeeping (one warp per row) -------------------------------
__device__ void stage_final(const MegaArgs& a, int wtid) {
  const int lane = wtid & 31, wid = wtid >> 5;
  for (int r = blockIdx.x * 8 + wid; r < a.B; r += gridDim.x * 8) {
    int tok = a.eos_id;
    if (a.st.active[r]) {
      uint32_t bk = 0;
      int bi = 0x7fffffff;
      for (int t = lane; t < a.n_tiles_lm; t += 32) {
        const uint32_t k = __float_as_uint(__ldcg(a.tile_val + (size_t)r * a.n_tiles_lm + t));
        const int id = __ldcg(a.tile_idx + (size_t)r * a.n_tiles_lm + t);
        if (k > bk || (k == bk && id < bi)) { bk = k; bi = id; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const uint32_t ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ok > bk || (ok == bk && oi < bi)) { bk = ok; bi = oi; }
      }
      if (lane == 0) {
        a.st.ctx_len[r] += 1;
        const int cap = a.st.scalars[0];
        const int gidx = a.st.gen[r] + 1;
        tok = (bi == 0x7fffffff) ? 0 : bi;
        if (a.dump_choice) a.dump_choice[r] = tok;
        if (a.st.eos_at[r] > 0 && gidx == a.st.eos_at[r]) tok = a.eos_id;
        if (a.forced) tok = a.forced[r];
        a.st.out_tokens[(size_t)r * a.st.max_new + (gidx - 1)] = tok;
        a.st.gen[r] = gidx;
        a.st.cur_tok[r] = tok;
        if (tok == a.eos_id) { a.st.finished[r] = 1; a.st.active[r] = 0; }
        else if (gidx >= cap) { a.st.active[r] = 0; }
        else atomicAdd(a.st.scalars + 1, 1);
      }
    }
    if (lane == 0 && a.next_tokens) a.next_tokens[r] = tok;
  }
}

// ------------------------------------------------------------------------------------ the kernel
// WIDE: the variant for batches of more than 64 rows, which adds attention_warp_pairs.  It is an instantiation of
// its own because the batches up to 64 rows live on this kernel's register allocation: the same code with the
// extra path compiled in ran the 16-row step 2.5 % slower.
// TRACE: with the stage-boundary time stamps of CTA 0 (ss_set_trace); the timed paths run the variant without them.
template <int DH, bool WIDE, bool TRACE>
__global__ void __launch_bounds__(kMegaThreads, 1)
decode_step_mega_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_o,
                        const __grid_constant__ CUtensorMap map_act, const __grid_constant__ MegaArgs a) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  MegaSmem* sm = reinterpret_cast<MegaSmem*>(smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const uint32_t stage0 = (smem_u32(smem_raw) + (uint32_t)sizeof(MegaSmem) + 1023u) & ~1023u;
  // ring: S activation blocks first, then S weight blocks.  A token tile shorter than 128 rows is read
  // by the tensor core as 128 rows anyway; the surplus rows fall on the blocks that follow.
  // the batches up to 64 rows always have one token tile, computed with the 64-lane instruction
  const int m_tiles = WIDE ? a.m_tiles : 1;
  const uint32_t x_tile_bytes = (uint32_t)a.x_rows * kTileK * 2;
  const uint32_t x_bytes = (uint32_t)m_tiles * x_tile_bytes;
  const uint32_t stage_tx = (uint32_t)kBlockBytes + x_bytes;
  const int S = a.stages;
  const uint32_t x0 = stage0, w0 = stage0 + (uint32_t)S * x_bytes;
  const int acc_bufs = m_tiles == 1 ? 2 : 1;         // 512 columns: two buffers of 256, or one of 2 x 256
  constexpr uint32_t kTmemCols = 512;
  const int n_gemm = 4 * a.n_layers + 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(&sm->full[s]), 1);
      mbar_init(smem_u32(&sm->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sm->acc_full[b]), 1);
      mbar_init(smem_u32(&sm->acc_empty[b]), 8);
    }
    sm->w_issued = 0;
    sm->act_epoch = 0;
    sm->abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_o);
    tma_prefetch_desc(&map_act);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sm->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sm->tmem_base;

  if (warp == 0) {
    // ===================== weight producer =====================
    if (lane == 0) {
      uint64_t hint_w;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(hint_w));
      int gi = 0;
      bool ok = true;
      for (int gm = 0; gm < n_gemm && ok; ++gm) {
        const MegaGemmShape& gs = a.shape[gm == n_gemm - 1 ? 4 : (gm & 3)];
        const uint8_t* w = a.wptr[gm];
        long long it0, it1;
        mega_range(gs, cta, it0, it1);
        for (long long it = it0; it < it1; ++it, ++gi) {
          const int stage = gi % S;
          if (gi >= S) {
            ok = mega_wait(smem_u32(&sm->empty[stage]), (uint32_t)(((gi / S) & 1) ^ 1), sm, a.status, kStatusProducerTimeout, a.wait_limit);
            if (!ok) break;
          }
          const uint32_t full = smem_u32(&sm->full[stage]);
          mbar_expect_tx(full, stage_tx);
          bulk_load(w0 + (uint32_t)stage * kBlockBytes, w + (size_t)it * kBlockBytes, kBlockBytes, full, hint_w);
          __threadfence_block();
          sm->w_issued = gi + 1;
        }
      }
      if (!ok || sm->abort) {
        // The step was abandoned.  Before this CTA gives its shared memory up, the bulk copies it still has in
        // flight (at most the last S ring stages) are given time to land: a bounded look at each stage's barrier,
        // which flips once the stage's bytes are in (a stage whose activation block was never requested does not
        // flip; its weight block has landed long before the limit, a thousand times a copy's latency, runs out).
        for (int j = gi > S ? gi - S : 0; j < gi; ++j) {
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&sm->full[j % S]), (uint32_t)((j / S) & 1)) && clock64() - t0 < 2000000LL) __nanosleep(100);
        }
      }
    }
  } else if (warp == 2) {
    // ===================== activation loader =====================
    if (lane == 0) {
      uint64_t hint_x;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(hint_x));
      int gi = 0;
      bool ok = true;
      for (int gm = 0; gm < n_gemm && ok; ++gm) {
        const int type = gm == n_gemm - 1 ? 4 : (gm & 3);
        const MegaGemmShape& gs = a.shape[type];
        const CUtensorMap* mp = (type == 1) ? &map_o : (type == 3) ? &map_act : &map_x;
        long long it0, it1;
        mega_range(gs, cta, it0, it1);
        if (it0 == it1) continue;
        // the operand is complete once the workers have passed the grid barrier before this projection
        {
          const long long t0 = clock64();
          while (sm->act_epoch <= gm) {
            __nanosleep(20);
            if (sm->abort) { ok = false; break; }
            if (clock64() - t0 > a.wait_limit) {
              atomicCAS(a.status, 0u, (uint32_t)kStatusFlagTimeout);
              sm->abort = 1;
              ok = false;
              break;
            }
          }
          if (!ok) break;
          // the worker that set the flag had acquired the grid barrier at gpu scope and released the flag at CTA
          // scope; a CTA-scope fence here completes the chain (a gpu-scope fence costs a round trip to L2)
          __threadfence_block();
          fence_proxy_async_global();          // global only: the full fence stalls ~2 us while ring copies are in flight
        }
        for (long long it = it0; it < it1; ++it, ++gi) {
          const long long t0 = clock64();
          while (sm->w_issued <= gi) {
            __nanosleep(40);
            if (sm->abort) { ok = false; break; }
            if (clock64() - t0 > a.wait_limit) {
              atomicCAS(a.status, 0u, (uint32_t)kStatusFlagTimeout);
              sm->abort = 1;
              ok = false;
              break;
            }
          }
          if (!ok) break;
          const int stage = gi % S;
          for (int mt = 0; mt < m_tiles; ++mt)
            tma_load_2d(x0 + (uint32_t)stage * x_bytes + (uint32_t)mt * x_tile_bytes, mp, smem_u32(&sm->full[stage]),
                        (int)(it % gs.kb) * kTileK, mt * 128, hint_x);
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      // M = token lanes (64 up to 64 rows: half the tensor-core work on unused lanes), N = 256 weight rows
      const uint32_t idesc = umma_idesc_bf16(kTileN, WIDE ? 128 : 64);
      int gi = 0, seg = 0;
      bool ok = true;
      for (int gm = 0; gm < n_gemm && ok; ++gm) {
        const MegaGemmShape& gs = a.shape[gm == n_gemm - 1 ? 4 : (gm & 3)];
        long long it0, it1;
        mega_range(gs, cta, it0, it1);
        long long it = it0;
        while (it < it1 && ok) {
          const int tile = (int)(it / gs.kb);
          long long seg_end = (long long)(tile + 1) * gs.kb;
          if (seg_end > it1) seg_end = it1;
          const int buf = seg % acc_bufs;
          ok = mega_wait(smem_u32(&sm->acc_empty[buf]), (uint32_t)(((seg / acc_bufs) & 1) ^ 1), sm, a.status,
                         kStatusMmaTimeout, a.wait_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kTileN);
          bool first = true;
          for (; it < seg_end; ++it, ++gi) {
            const int stage = gi % S;
            ok = mega_wait(smem_u32(&sm->full[stage]), (uint32_t)((gi / S) & 1), sm, a.status, kStatusMmaTimeout, a.wait_limit);
            if (!ok) break;
            tc_fence_after();
            const uint64_t dw = smem_desc_sw128(w0 + (uint32_t)stage * kBlockBytes);
            for (int mt = 0; mt < m_tiles; ++mt) {
              const uint64_t dx = smem_desc_sw128(x0 + (uint32_t)stage * x_bytes + (uint32_t)mt * x_tile_bytes);
#pragma unroll
              for (int k = 0; k < kTileK / 16; ++k)
                umma_bf16(d_tmem + (uint32_t)(mt * kTileN), dx + (uint64_t)(k * 2), dw + (uint64_t)(k * 2), idesc,
                          (first && k == 0) ? 0u : 1u);
            }
            first = false;
            umma_commit(smem_u32(&sm->empty[stage]));
          }
          if (!ok) break;
          umma_commit(smem_u32(&sm->acc_full[buf]));
          ++seg;
        }
      }
    }
  } else if (warp >= 3) {
    // ===================== workers =====================
    const int wtid = threadIdx.x - 96;
    const int wid = wtid >> 5;
    const int quarter = warp & 3;                   // tensor-memory lane quarter this warp may read
    const int colhalf = wid >> 2;                   // warps 3-6 take the first 128 weight rows of a tile
    unsigned long long epoch = 0;
    int seg = 0;
    bool ok = true;

    const bool tracer = TRACE && cta == 0 && wtid == 0 && a.trace != nullptr;
    int tr = 0;
    if (tracer) a.trace[tr++] = global_timer_ns();
    if (cta == 0 && wtid == 0) a.st.scalars[1] = 0;   // rows still active after this step (counted in the last stage)
    attention_setup<DH, WIDE>(a, sm, wtid);
    stage_residual(a, sm, wtid, 0, nullptr, a.norm_ptr[0], a.n_layers == 0);
    ok = grid_barrier(a, sm, epoch, wtid, true);
    if (ok && wtid == 0) { __threadfence_block(); sm->act_epoch = 1; }
    if (tracer) a.trace[tr++] = global_timer_ns();

    for (int gm = 0; gm < n_gemm && ok; ++gm) {
      const int type = gm == n_gemm - 1 ? 4 : (gm & 3);
      const int layer = gm >> 2;
      const MegaGemmShape& gs = a.shape[type];
      // ---- drain this CTA's segments of projection gm into fp32 partials
      long long it0, it1;
        mega_range(gs, cta, it0, it1);
      long long it = it0;
      int seg_local = 0;
      while (it < it1 && ok) {
        const int tile = (int)(it / gs.kb);
        long long seg_end = (long long)(tile + 1) * gs.kb;
        if (seg_end > it1) seg_end = it1;
        const int buf = seg % acc_bufs;
        ok = mega_wait(smem_u32(&sm->acc_full[buf]), (uint32_t)((seg / acc_bufs) & 1), sm, a.status,
                       kStatusEpilogueTimeout, a.wait_limit);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const size_t slot = (size_t)cta * gs.max_seg + seg_local;
        for (int mt = 0; mt < m_tiles; ++mt) {
          // batch row held by this thread's lane: 32 per lane quarter, or 16 with the 64-row instruction
          constexpr int per_q = WIDE ? 32 : 16;
          if (mt * 128 + quarter * per_q >= a.B) continue;     // no batch row in this warp's lanes (warp-uniform)
          const int tok = lane < per_q ? mt * 128 + quarter * per_q + lane : a.B;
          const uint32_t taddr =
              tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((buf + mt) * kTileN + colhalf * 128);
          float* dst = a.partial + (slot * a.NT + tok) * kTileN + colhalf * 128;
          // 64 columns per TMEM load: the last segment's drain is the serial tail of every projection
#pragma unroll 1
          for (int c = 0; c < 128; c += 64) {
            uint32_t v[64];
            tmem_ld64(taddr + c, v);
            if (a.NT <= 16) {
              // one MMA's worth of rows or fewer: the tail is a chain of latencies, direct stores are the shortest one
              if (tok < a.B) {
#pragma unroll
                for (int j = 0; j < 64; j += 4)
                  *reinterpret_cast<uint4*>(dst + c + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
              }
            } else {
              // many rows: a lane holds one token's outputs, so direct 128-bit stores put every lane's 16 bytes
              // into a sector of its own, 1 KiB apart, and the drain is bound by the sectors it writes.  The
              // warp turns 32 outputs at a time through shared memory (rows padded to 36 floats: both
              // directions free of bank conflicts) and stores whole 128-byte lines, four tokens per instruction.
              float* tr = &sm->att_s[0][0][0] + wid * (32 * 36);
              const int t_hi = lane >> 3, cg = lane & 7;
#pragma unroll
              for (int sub = 0; sub < 2; ++sub) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                  *reinterpret_cast<uint4*>(tr + lane * 36 + j) =
                      make_uint4(v[sub * 32 + j], v[sub * 32 + j + 1], v[sub * 32 + j + 2], v[sub * 32 + j + 3]);
                __syncwarp();
                for (int i = 0; i < per_q / 4; ++i) {
                  const int tl = 4 * i + t_hi;
                  const int tg = mt * 128 + quarter * per_q + tl;
                  if (tg < a.B)
                    *reinterpret_cast<uint4*>(a.partial + (slot * a.NT + tg) * kTileN + colhalf * 128 + c + sub * 32 + 4 * cg) =
                        *reinterpret_cast<const uint4*>(tr + tl * 36 + 4 * cg);
                }
                __syncwarp();
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm->acc_empty[buf]));
        it = seg_end;
        ++seg;
        ++seg_local;
      }
      if (!ok) break;
      if (tracer) a.trace[tr++] = global_timer_ns();       // this CTA's accumulators drained
      ok = grid_barrier(a, sm, epoch, wtid, false);
      if (!ok) break;
      if (tracer) a.trace[tr++] = global_timer_ns();       // every CTA's partials visible
      // ---- the stage that consumes the projection
      if (type == 0) {
        if constexpr (WIDE) {
          if (sm->att_warp_pairs) attention_warp_pairs<DH>(a, sm, wtid, layer);
          else stage_attention<DH>(a, sm, wtid, layer);
        } else {
          stage_attention<DH>(a, sm, wtid, layer);
        }
      } else if (type == 1) {
        stage_residual(a, sm, wtid, 1, &a.shape[1], a.norm_ptr[2 * layer + 1], false);
      } else if (type == 2) {
        stage_swiglu(a, sm, wtid);
      } else if (type == 3) {
        stage_residual(a, sm, wtid, 1, &a.shape[3], a.norm_ptr[2 * layer + 2], layer + 1 == a.n_layers);
      } else {
        stage_tile_argmax(a, sm, wtid);
      }
      if (tracer) a.trace[tr++] = global_timer_ns();       // this CTA's share of the stage done
      ok = grid_barrier(a, sm, epoch, wtid, true);
      if (!ok) break;
      if (tracer) a.trace[tr++] = global_timer_ns();       // stage complete everywhere
      if (type == 4) stage_final(a, wtid);
      else if (wtid == 0) { __threadfence_block(); sm->act_epoch = gm + 2; }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Self-test of the bounded grid-wide wait, with nothing else in flight (no bulk copies, no tensor-core work): every
// CTA arrives on the counter and then waits for one arrival more than the grid can deliver.  The wait must run out
// after `limit` cycles, record kStatusGridBarrierTimeout and let the kernel end normally.
__global__ void __launch_bounds__(32)
grid_wait_selftest_kernel(unsigned long long* ctr, unsigned long long base, long long limit, uint32_t* status) {
  if (threadIdx.x == 0) {
    const unsigned long long target = base + (unsigned long long)gridDim.x + 1ULL;
    if (!arrive_and_poll(ctr, target, limit, nullptr)) atomicCAS(status, 0u, (uint32_t)kStatusGridBarrierTimeout);
  }
}

}  // namespace ss
