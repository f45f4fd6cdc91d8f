// Memory-bound kernels of the decode step and the prompt pass (sm_100a).
//
// Decode (one token per active row):
//   embed_rmsnorm -> [ qkv GEMM -> rope_append_decode -> attn_decode -> attn_combine -> o GEMM ->
//   residual_rmsnorm -> gate/up GEMM -> swiglu -> down GEMM -> residual_rmsnorm ] x layers ->
//   lm_head GEMM -> lmhead_argmax -> bookkeeping
// The GEMMs leave fp32 partial sums (split along K); the kernel that consumes a projection adds
// the partials in a fixed order and applies what follows the projection in the model.
//
// Every kernel starts with griddepcontrol.launch_dependents / griddepcontrol.wait so that the
// next kernel's prologue (for a GEMM: its first weight tiles) overlaps this kernel's body.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "ss_gemm.cuh"

namespace ss {

using bf16 = __nv_bfloat16;

// Per-batch device state (arrays of max_batch entries unless noted).
struct RowState {
  int32_t* ctx_len;      // tokens whose keys/values are cached
  int32_t* cur_tok;      // last emitted token, fed by the next step
  int32_t* gen;          // tokens generated so far
  int32_t* active;       // 1 while the row is generating
  int32_t* finished;     // 1 once EOS was emitted
  int32_t* eos_at;       // 0 = natural EOS, t >= 1 = forced EOS at generated index t
  int32_t* choice;       // argmax of the current step
  int32_t* out_tokens;   // [max_batch][max_new]
  int32_t* block_table;  // [max_batch][max_pages]
  int32_t* scalars;      // [0] = cap, [1] = n_active
  int max_pages, max_new;
};

struct KvLayout {
  bf16* pool;            // [layer][page][K|V][head][page_tok][Dh]
  size_t layer_stride;   // elements between layers
  size_t page_elems;     // elements per page: 2*H*page_tok*Dh
  int n_pages, H, Dh;
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Sum over the block; every thread gets the result.  `red` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < nw) ? red[lane] : 0.f;
  t = warp_sum(t);
  return t;
}

// ------------------------------------------------------------------------------------ weight repacking
// Row-major [rows, K] bf16 -> the GEMM's streaming layout: 16 KiB blocks in (tile, k-block) order, each
// the exact shared-memory image of a 128-row x 64-column tile under the 128-byte swizzle (row r at
// r*128 bytes, its 16-byte chunk c stored at chunk position c ^ (r & 7)).  One thread per 16-byte chunk.
// row_off places the source at a row offset of the destination matrix (q,k,v and gate,up are stacked).
__global__ void __launch_bounds__(256)
repack_weights_kernel(const uint4* __restrict__ src, long long rows, int K, uint8_t* __restrict__ dst, int row_off,
                      int kb) {
  const int chunks_per_row = K >> 3;
  const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (id >= rows * chunks_per_row) return;
  const long long sr = id / chunks_per_row;
  const int cc = (int)(id - sr * chunks_per_row);
  const long long n = row_off + sr;
  const long long tile = n >> 7;
  const int r = (int)(n & 127), k = cc >> 3, c = cc & 7;
  uint8_t* blk = dst + ((size_t)tile * kb + k) * (size_t)(kTileM * kTileK * 2);
  *reinterpret_cast<uint4*>(blk + r * 128 + ((c ^ (r & 7)) << 4)) = src[id];
}

// ------------------------------------------------------------------------------------ embedding + first norm
// h[row] = E[token]; x[row] = RMSNorm(h[row]) * g   (rows: decode B rows or T prompt tokens)
__global__ void __launch_bounds__(256)
embed_rmsnorm_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ active,
                     const bf16* __restrict__ E, const bf16* __restrict__ g, float* __restrict__ h,
                     bf16* __restrict__ x, int d, float eps, int vocab) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  if (active && !active[r]) return;
  int tok = tokens[r];
  if (tok < 0 || tok >= vocab) tok = 0;
  const bf16* e = E + (size_t)tok * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = __bfloat162float(e[i]);
    h[(size_t)r * d + i] = v;
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = __bfloat162float(e[i]);
    x[(size_t)r * d + i] = __float2bfloat16_rn(v * inv * __bfloat162float(g[i]));
  }
}

// ------------------------------------------------------------------------------------ RoPE + KV append (decode)
// grid (H, B), block Dh.  q,k,v come as fp32 partials of the [3d] projection; thread i owns element
// i of the head.  Pair (i, i+Dh/2) of q and k is rotated by pos * inv_freq[i]; k,v go to the row's page.
__global__ void __launch_bounds__(128)
rope_append_decode_kernel(const float* __restrict__ partial, SplitInfo sp, RowState st, KvLayout kv, int layer,
                          const float* __restrict__ inv_freq, bf16* __restrict__ qbuf, int d, uint32_t* status) {
  __shared__ float s_q[128], s_k[128];
  pdl_launch_dependents();
  pdl_wait();
  const int hd = blockIdx.x, r = blockIdx.y, i = threadIdx.x;
  if (!st.active[r]) return;
  const int Dh = kv.Dh, half = Dh >> 1;
  const int pos = st.ctx_len[r];
  const int n = hd * Dh + i;
  const float qv = sum_partials(partial, sp, n, r);
  const float kvv = sum_partials(partial, sp, d + n, r);
  const float vv = sum_partials(partial, sp, 2 * d + n, r);
  s_q[i] = qv;
  s_k[i] = kvv;
  __syncthreads();
  const int j = i < half ? i : i - half;          // frequency index
  float sn, cs;
  sincosf((float)pos * inv_freq[j], &sn, &cs);
  // first half: x_i cos - x_{i+half} sin; second half: x_i cos + x_{i-half} sin
  const float qo = i < half ? qv * cs - s_q[i + half] * sn : qv * cs + s_q[i - half] * sn;
  const float ko = i < half ? kvv * cs - s_k[i + half] * sn : kvv * cs + s_k[i - half] * sn;
  qbuf[(size_t)r * d + n] = __float2bfloat16_rn(qo);
  const int page = st.block_table[(size_t)r * st.max_pages + pos / kPageTokens];
  if (page < 0 || page >= kv.n_pages) {
    atomicCAS(status, 0u, (uint32_t)kStatusBadPage);
    return;
  }
  bf16* kbase = kv.pool + (size_t)layer * kv.layer_stride + (size_t)page * kv.page_elems +
                ((size_t)hd * kPageTokens + (pos % kPageTokens)) * Dh;
  bf16* vbase = kbase + (size_t)kv.H * kPageTokens * Dh;
  kbase[i] = __float2bfloat16_rn(ko);
  vbase[i] = __float2bfloat16_rn(vv);
}

// ------------------------------------------------------------------------------------ decode attention (paged)
// Work item = (row, head, chunk of kAttnChunk cached tokens); items are dealt round-robin to a
// fixed grid, so the launch does not depend on the lengths (which live on the device).
// A group of Dh/8 lanes owns one key: each lane loads 8 bf16 (128 bits) of K and of V, the group
// reduces q.k with shuffles and keeps a running (max, sum, acc) triple; groups are merged in
// shared memory and the item's triple goes to the partial buffer.
struct AttnArgs {
  RowState st;
  KvLayout kv;
  const bf16* q;         // [B][d]
  float* part_ml;        // [B][H][max_chunks][2]
  float* part_acc;       // [B][H][max_chunks][Dh]
  bf16* out;             // [B][d]
  int B, d, layer, max_chunks;
  uint32_t* status;
};

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 t = __bfloat1622float2(p[j]);
    f[2 * j] = t.x;
    f[2 * j + 1] = t.y;
  }
}

template <int DH>
__global__ void __launch_bounds__(128) attn_decode_kernel(AttnArgs a) {
  constexpr int GROUP = DH / 8;          // lanes per key
  constexpr int KPW = 32 / GROUP;        // keys per warp
  constexpr int NG = 4 * KPW;            // groups per CTA
  constexpr int PPC = kAttnChunk / kPageTokens;
  __shared__ int s_prefix[kMaxBatch + 1];
  __shared__ float s_m[NG], s_l[NG];
  __shared__ float s_acc[NG][DH];
  __shared__ int s_pages[PPC];

  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = a.B, H = a.kv.H;

  // exclusive prefix of chunk counts over rows (warp 0: 8 rows per lane)
  if (warp == 0) {
    int cnt[8], loc = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int r = lane * 8 + j;
      int c = 0;
      if (r < B && a.st.active[r]) c = (a.st.ctx_len[r] + 1 + kAttnChunk - 1) / kAttnChunk;
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
      s_prefix[lane * 8 + j] = run;
      run += cnt[j];
    }
    if (lane == 31) s_prefix[kMaxBatch] = inc;
  }
  __syncthreads();
  const int total_chunks = s_prefix[kMaxBatch];
  const int n_items = total_chunks * H;
  const int g = warp * KPW + lane / GROUP, gl = lane % GROUP;
  const float qscale = rsqrtf((float)DH) * 1.4426950408889634f;   // 1/sqrt(Dh) * log2(e)
  const bf16* kv_layer = a.kv.pool + (size_t)a.layer * a.kv.layer_stride;
  const size_t v_off = (size_t)H * kPageTokens * DH;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int cidx = item / H, hd = item - cidx * H;
    int lo = 0, hi = B - 1;                       // largest r with prefix[r] <= cidx
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (s_prefix[mid] <= cidx) lo = mid; else hi = mid - 1;
    }
    const int r = lo, chunk = cidx - s_prefix[r];
    const int n_keys = a.st.ctx_len[r] + 1;
    const int t0 = chunk * kAttnChunk;
    const int t1 = min(t0 + kAttnChunk, n_keys);
    if (tid < PPC) {
      const int pi = t0 / kPageTokens + tid;
      int pg = 0;
      if (pi * kPageTokens < t1) {
        pg = a.st.block_table[(size_t)r * a.st.max_pages + pi];
        if (pg < 0 || pg >= a.kv.n_pages) { atomicCAS(a.status, 0u, (uint32_t)kStatusBadPage); pg = 0; }
      }
      s_pages[tid] = pg;
    }
    float q[8];
    {
      const uint4 u = *reinterpret_cast<const uint4*>(a.q + (size_t)r * a.d + hd * DH + gl * 8);
      unpack8(u, q);
#pragma unroll
      for (int j = 0; j < 8; ++j) q[j] *= qscale;
    }
    __syncthreads();

    float m = -CUDART_INF_F, l = 0.f, acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;

    constexpr int U = 4;
    // the trip count is the same for every lane of the warp (the shuffles below need all of them)
    for (int base = t0; base < t1; base += NG * U) {
      const int tb = base + g;
      uint4 kk[U], vv[U];
      bool valid[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int t = tb + u * NG;
        valid[u] = t < t1;
        kk[u] = make_uint4(0, 0, 0, 0);
        vv[u] = kk[u];
        if (valid[u]) {
          const int pg = s_pages[(t - t0) / kPageTokens];
          const bf16* kp = kv_layer + (size_t)pg * a.kv.page_elems +
                           ((size_t)hd * kPageTokens + (t % kPageTokens)) * DH + gl * 8;
          kk[u] = __ldg(reinterpret_cast<const uint4*>(kp));
          vv[u] = __ldg(reinterpret_cast<const uint4*>(kp + v_off));
        }
      }
      float s[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float kf[8], dot = 0.f;
        unpack8(kk[u], kf);
#pragma unroll
        for (int j = 0; j < 8; ++j) dot += q[j] * kf[j];
#pragma unroll
        for (int o = GROUP / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        s[u] = valid[u] ? dot : -CUDART_INF_F;
      }
      float mn = m;
#pragma unroll
      for (int u = 0; u < U; ++u) mn = fmaxf(mn, s[u]);
      // a group that has seen no key yet keeps (m, l, acc) = (-inf, 0, 0): exp2(-inf - -inf) would be NaN
      const float sc = (mn == -CUDART_INF_F) ? 1.f : exp2f(m - mn);
      l *= sc;
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] *= sc;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        if (valid[u]) {
          const float pw = exp2f(s[u] - mn);
          float vf[8];
          unpack8(vv[u], vf);
          l += pw;
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[j] += pw * vf[j];
        }
      }
      m = mn;
    }
    if (gl == 0) { s_m[g] = m; s_l[g] = l; }
#pragma unroll
    for (int j = 0; j < 8; ++j) s_acc[g][gl * 8 + j] = acc[j];
    __syncthreads();
    if (tid < DH) {
      float M = -CUDART_INF_F;
#pragma unroll
      for (int x = 0; x < NG; ++x) M = fmaxf(M, s_m[x]);
      float L = 0.f, A = 0.f;
#pragma unroll
      for (int x = 0; x < NG; ++x) {
        const float w = (s_m[x] == -CUDART_INF_F) ? 0.f : exp2f(s_m[x] - M);
        L += s_l[x] * w;
        A += s_acc[x][tid] * w;
      }
      const size_t slot = ((size_t)r * H + hd) * a.max_chunks + chunk;
      a.part_acc[slot * DH + tid] = A;
      if (tid == 0) { a.part_ml[slot * 2] = M; a.part_ml[slot * 2 + 1] = L; }
    }
    __syncthreads();
  }
}

// grid (H, B), block DH: merge the chunks of one (row, head); out = acc / sum in bf16.
template <int DH>
__global__ void __launch_bounds__(DH) attn_combine_kernel(AttnArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  const int hd = blockIdx.x, r = blockIdx.y, i = threadIdx.x;
  if (!a.st.active[r]) return;
  const int n_keys = a.st.ctx_len[r] + 1;
  const int nch = (n_keys + kAttnChunk - 1) / kAttnChunk;
  const size_t base = ((size_t)r * a.kv.H + hd) * a.max_chunks;
  float M = -CUDART_INF_F;
  for (int c = 0; c < nch; ++c) M = fmaxf(M, a.part_ml[(base + c) * 2]);
  float L = 0.f, A = 0.f;
  for (int c = 0; c < nch; ++c) {
    const float w = exp2f(a.part_ml[(base + c) * 2] - M);
    L += a.part_ml[(base + c) * 2 + 1] * w;
    A += a.part_acc[(base + c) * DH + i] * w;
  }
  a.out[(size_t)r * a.d + hd * DH + i] = __float2bfloat16_rn(A / L);
}

// ------------------------------------------------------------------------------------ residual + RMSNorm (decode)
// h[r] += projection (from partials); x[r] = RMSNorm(h[r]) * g.  grid B, block 1024 (d <= 8192).
__global__ void __launch_bounds__(1024)
residual_rmsnorm_partial_kernel(const float* __restrict__ partial, SplitInfo sp, const int32_t* __restrict__ active,
                                float* __restrict__ h, const bf16* __restrict__ g, bf16* __restrict__ x,
                                float* __restrict__ dump_hidden, int d, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  if (active && !active[r]) return;
  constexpr int kMaxPer = 8;
  float v[kMaxPer];
  float ss = 0.f;
#pragma unroll
  for (int c = 0; c < kMaxPer; ++c) {
    const int i = threadIdx.x + c * 1024;
    v[c] = 0.f;
    if (i < d) {
      v[c] = h[(size_t)r * d + i] + sum_partials(partial, sp, i, r);
      ss += v[c] * v[c];
    }
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / d + eps);
#pragma unroll
  for (int c = 0; c < kMaxPer; ++c) {
    const int i = threadIdx.x + c * 1024;
    if (i < d) {
      h[(size_t)r * d + i] = v[c];
      if (dump_hidden) dump_hidden[(size_t)r * d + i] = v[c];
      x[(size_t)r * d + i] = __float2bfloat16_rn(v[c] * inv * __bfloat162float(g[i]));
    }
  }
}

// act[r][f] = silu(gate) * up from the partials of the stacked [2F] projection.  grid (ceil(F/256), B)
__global__ void __launch_bounds__(256)
swiglu_partial_kernel(const float* __restrict__ partial, SplitInfo sp, bf16* __restrict__ act, int F) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y, f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= F) return;
  const float gt = sum_partials(partial, sp, f, r);
  const float up = sum_partials(partial, sp, F + f, r);
  act[(size_t)r * F + f] = __float2bfloat16_rn(gt / (1.f + __expf(-gt)) * up);
}

// ------------------------------------------------------------------------------------ LM head argmax
// Stage 1, grid n_tiles (of the vocabulary), block 128 (thread = vocabulary row of the tile):
// logits from partials for every row of the batch, optional dump, and the tile's best (value, id)
// per batch row; the lowest id wins a tie; EOS is left out when the row has a forced-EOS schedule.
// Stage 2 (inside bookkeeping_kernel) picks the best tile per row.
__device__ __forceinline__ uint32_t float_order_key(float f) {      // monotone float -> uint32
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(128)
lmhead_tile_argmax_kernel(const float* __restrict__ partial, SplitInfo sp, RowState st, float* __restrict__ dump_logits,
                          float* __restrict__ tile_val, int32_t* __restrict__ tile_idx, int B, int vocab, int n_tiles,
                          int eos_id) {
  __shared__ uint32_t s_key[4][kMaxBatch];
  __shared__ int s_id[4][kMaxBatch];
  pdl_launch_dependents();
  pdl_wait();
  const int tile = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int v = tile * 128 + threadIdx.x;
  for (int r = 0; r < B; ++r) {
    uint32_t key = 0;                              // below every real key
    if (st.active[r]) {
      if (v < vocab) {
        const float lg = sum_partials(partial, sp, v, r);
        if (dump_logits) dump_logits[(size_t)r * vocab + v] = lg;
        if (!(st.eos_at[r] > 0 && v == eos_id)) key = float_order_key(lg);
      }
      const uint32_t best = __reduce_max_sync(0xffffffffu, key);
      const uint32_t who = __ballot_sync(0xffffffffu, key == best);
      if (lane == 0) {
        s_key[warp][r] = best;
        s_id[warp][r] = tile * 128 + warp * 32 + (__ffs(who) - 1);     // lowest lane = lowest id
      }
    }
  }
  __syncthreads();
  for (int r = threadIdx.x; r < B; r += 128) {
    if (!st.active[r]) continue;
    uint32_t bk = s_key[0][r];
    int bi = s_id[0][r];
#pragma unroll
    for (int w = 1; w < 4; ++w)
      if (s_key[w][r] > bk) { bk = s_key[w][r]; bi = s_id[w][r]; }     // warps ascend in id: '>' keeps the lowest
    tile_val[(size_t)r * n_tiles + tile] = __uint_as_float(bk);       // order key, bit-cast
    tile_idx[(size_t)r * n_tiles + tile] = bi;
  }
}

// ------------------------------------------------------------------------------------ step bookkeeping
// One block of 1024 threads; warp w serves rows w, w+32, ...: final argmax over the vocabulary
// tiles, then the row's state update.  is_prefill: the prompt has just been cached (ctx_len set
// by the host) and this is generated token 1; otherwise the fed token becomes part of the cache.
__global__ void __launch_bounds__(1024)
bookkeeping_kernel(RowState st, const float* __restrict__ tile_val, const int32_t* __restrict__ tile_idx, int n_tiles,
                   const int32_t* __restrict__ forced, int32_t* __restrict__ next_tokens, int B, int eos_id,
                   int is_prefill) {
  __shared__ int s_still;
  pdl_launch_dependents();
  pdl_wait();
  if (threadIdx.x == 0) s_still = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int still = 0;
  for (int r = warp; r < B; r += 32) {
    int tok = eos_id;
    if (st.active[r]) {
      uint32_t bk = 0;
      int bi = 0x7fffffff;
      for (int t = lane; t < n_tiles; t += 32) {
        const uint32_t k = __float_as_uint(tile_val[(size_t)r * n_tiles + t]);
        const int id = tile_idx[(size_t)r * n_tiles + t];
        if (k > bk || (k == bk && id < bi)) { bk = k; bi = id; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const uint32_t ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ok > bk || (ok == bk && oi < bi)) { bk = ok; bi = oi; }
      }
      if (lane == 0) {
        if (!is_prefill) st.ctx_len[r] += 1;
        const int cap = st.scalars[0];
        const int gidx = st.gen[r] + 1;               // 1-based index of the token being emitted
        tok = (bi == 0x7fffffff) ? 0 : bi;
        if (st.eos_at[r] > 0 && gidx == st.eos_at[r]) tok = eos_id;
        if (forced) tok = forced[r];
        st.out_tokens[(size_t)r * st.max_new + (gidx - 1)] = tok;
        st.gen[r] = gidx;
        st.cur_tok[r] = tok;
        if (tok == eos_id) { st.finished[r] = 1; st.active[r] = 0; }
        else if (gidx >= cap) { st.active[r] = 0; }
        else still += 1;
      }
    }
    if (lane == 0 && next_tokens) next_tokens[r] = tok;
  }
  if (lane == 0 && still) atomicAdd(&s_still, still);
  __syncthreads();
  if (threadIdx.x == 0) st.scalars[1] = s_still;
}

// ------------------------------------------------------------------------------------ prompt-pass kernels
// x[t] = RMSNorm(h[t]) * g over T tokens.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const float* __restrict__ h, const bf16* __restrict__ g, bf16* __restrict__ x, int d, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const size_t r = blockIdx.x;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = h[r * d + i];
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    x[r * d + i] = __float2bfloat16_rn(h[r * d + i] * inv * __bfloat162float(g[i]));
}

// Gather each sequence's last token: h_last[s] = h[last[s]]; x_last[s] = RMSNorm(h_last[s]) * g.
__global__ void __launch_bounds__(256)
gather_last_rmsnorm_kernel(const float* __restrict__ h, const int32_t* __restrict__ last_tok, float* __restrict__ h_out,
                           const bf16* __restrict__ g, bf16* __restrict__ x_out, float* __restrict__ dump_hidden,
                           int d, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int s = blockIdx.x;
  const size_t t = (size_t)last_tok[s];
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = h[t * d + i];
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float inv = rsqrtf(ss / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = h[t * d + i];
    h_out[(size_t)s * d + i] = v;
    if (dump_hidden) dump_hidden[(size_t)s * d + i] = v;
    x_out[(size_t)s * d + i] = __float2bfloat16_rn(v * inv * __bfloat162float(g[i]));
  }
}

// In-place RoPE on q and k of the packed [T, 3d] projection, and copy of k,v into the pages.
// grid (T, H), block Dh/2.  tok_row / tok_pos give each token's row in the batch and position.
__global__ void rope_append_prefill_kernel(bf16* __restrict__ qkv, const int32_t* __restrict__ tok_row,
                                           const int32_t* __restrict__ tok_pos, RowState st, KvLayout kv, int layer,
                                           const float* __restrict__ inv_freq, int d, uint32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const int hd = blockIdx.y, i = threadIdx.x;
  const size_t t = blockIdx.x;
  const int r = tok_row[t], pos = tok_pos[t];
  const int Dh = kv.Dh, half = Dh >> 1;
  bf16* q = qkv + t * 3 * d + hd * Dh;
  bf16* k = q + d;
  const bf16* v = k + d;
  float sn, cs;
  sincosf((float)pos * inv_freq[i], &sn, &cs);
  const float q0 = __bfloat162float(q[i]), q1 = __bfloat162float(q[i + half]);
  const float k0 = __bfloat162float(k[i]), k1 = __bfloat162float(k[i + half]);
  const bf16 kr0 = __float2bfloat16_rn(k0 * cs - k1 * sn), kr1 = __float2bfloat16_rn(k1 * cs + k0 * sn);
  q[i] = __float2bfloat16_rn(q0 * cs - q1 * sn);
  q[i + half] = __float2bfloat16_rn(q1 * cs + q0 * sn);
  k[i] = kr0;
  k[i + half] = kr1;
  const int page = st.block_table[(size_t)r * st.max_pages + pos / kPageTokens];
  if (page < 0 || page >= kv.n_pages) {
    atomicCAS(status, 0u, (uint32_t)kStatusBadPage);
    return;
  }
  bf16* kbase = kv.pool + (size_t)layer * kv.layer_stride + (size_t)page * kv.page_elems +
                ((size_t)hd * kPageTokens + (pos % kPageTokens)) * Dh;
  bf16* vbase = kbase + (size_t)kv.H * kPageTokens * Dh;
  kbase[i] = kr0;
  kbase[i + half] = kr1;
  vbase[i] = v[i];
  vbase[i + half] = v[i + half];
}

// Causal attention over one prompt, tiled: CTA = (32 queries, head, sequence); 4 threads share a
// query (a quarter of the head each); keys/values are staged through shared memory 32 at a time.
// qkv: [T, 3d] with RoPE applied; out: [T, d].
template <int DH>
__global__ void __launch_bounds__(128)
attn_prefill_kernel(const bf16* __restrict__ qkv, const int32_t* __restrict__ cu_seqlens, bf16* __restrict__ out, int d) {
  constexpr int QT = 32, KT = 32, PART = DH / 4;
  __shared__ __align__(16) bf16 s_k[KT][DH];
  __shared__ __align__(16) bf16 s_v[KT][DH];
  pdl_launch_dependents();
  pdl_wait();
  const int hd = blockIdx.y, s = blockIdx.z;
  const int seq0 = cu_seqlens[s], len = cu_seqlens[s + 1] - seq0;
  const int qt0 = blockIdx.x * QT;
  if (qt0 >= len) return;
  const int qi = threadIdx.x >> 2, part = threadIdx.x & 3;
  const int qpos = qt0 + qi;
  const bool qvalid = qpos < len;
  const float qscale = rsqrtf((float)DH) * 1.4426950408889634f;
  float q[PART], acc[PART];
#pragma unroll
  for (int j = 0; j < PART; ++j) {
    q[j] = qvalid ? __bfloat162float(qkv[(size_t)(seq0 + qpos) * 3 * d + hd * DH + part * PART + j]) * qscale : 0.f;
    acc[j] = 0.f;
  }
  float m = -CUDART_INF_F, l = 0.f;
  const int k_end = min(len, qt0 + QT);            // causal: keys up to the tile's last query
  for (int kt0 = 0; kt0 < k_end; kt0 += KT) {
    __syncthreads();
    constexpr int CH = DH / 8;                     // 16-byte chunks per row
    for (int c = threadIdx.x; c < KT * CH; c += 128) {
      const int kr = c / CH, cc = c % CH;
      uint4 uk = make_uint4(0, 0, 0, 0), uv = uk;
      if (kt0 + kr < len) {
        const bf16* base = qkv + (size_t)(seq0 + kt0 + kr) * 3 * d + d + hd * DH + cc * 8;
        uk = *reinterpret_cast<const uint4*>(base);
        uv = *reinterpret_cast<const uint4*>(base + d);
      }
      *reinterpret_cast<uint4*>(&s_k[kr][cc * 8]) = uk;
      *reinterpret_cast<uint4*>(&s_v[kr][cc * 8]) = uv;
    }
    __syncthreads();
    const int kmax = min(KT, k_end - kt0);
    for (int j = 0; j < kmax; ++j) {
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < PART; e += 2) {
        const float2 kk = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&s_k[j][part * PART + e]));
        dot += q[e] * kk.x + q[e + 1] * kk.y;
      }
      dot += __shfl_xor_sync(0xffffffffu, dot, 1);
      dot += __shfl_xor_sync(0xffffffffu, dot, 2);
      if (kt0 + j <= qpos) {                        // causal mask (uniform within the 4-thread group)
        const float mn = fmaxf(m, dot);
        const float sc = exp2f(m - mn), pw = exp2f(dot - mn);
        l = l * sc + pw;
#pragma unroll
        for (int e = 0; e < PART; e += 2) {
          const float2 vv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&s_v[j][part * PART + e]));
          acc[e] = acc[e] * sc + pw * vv.x;
          acc[e + 1] = acc[e + 1] * sc + pw * vv.y;
        }
        m = mn;
      }
    }
  }
  if (qvalid) {
    const float inv = 1.f / l;
#pragma unroll
    for (int j = 0; j < PART; ++j)
      out[(size_t)(seq0 + qpos) * d + hd * DH + part * PART + j] = __float2bfloat16_rn(acc[j] * inv);
  }
}

// act[t][f] = silu(gu[t][f]) * gu[t][F+f] over T tokens.  grid (T, ceil(F/256))
__global__ void __launch_bounds__(256)
swiglu_kernel(const bf16* __restrict__ gu, bf16* __restrict__ act, int F) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t t = blockIdx.x;
  const int f = blockIdx.y * blockDim.x + threadIdx.x;
  if (f >= F) return;
  const float gt = __bfloat162float(gu[t * 2 * F + f]), up = __bfloat162float(gu[t * 2 * F + F + f]);
  act[t * F + f] = __float2bfloat16_rn(gt / (1.f + __expf(-gt)) * up);
}

}  // namespace ss
