// Kernels of the prompt pass, the weight repacking and the batch's first arg-max (sm_100a).
//
// Prompt pass (all prompt tokens of a chunk at once):
//   embed_rmsnorm -> [ qkv GEMM -> rope_append_prefill -> attn_prefill -> o GEMM (+= residual) ->
//   rmsnorm -> gate/up GEMM -> swiglu -> down GEMM (+= residual) -> rmsnorm ] x layers ->
//   gather_last_rmsnorm -> LM-head GEMM (fp32 partials) -> lmhead_tile_argmax -> bookkeeping
// The decode step itself is one persistent kernel (ss_decode_mega.cuh) and shares the small helpers here.
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
  int32_t* row_key;      // the row's key in the sampling counter (its query id inside a group)
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
// Row-major [rows, K] bf16 -> the GEMM's streaming layout: 32 KiB blocks in (tile, k-block) order, each
// the exact shared-memory image of a 256-row x 64-column tile under the 128-byte swizzle (row r at
// r*128 bytes, its 16-byte chunk c stored at chunk position c ^ (r & 7)).  Each half of a block is
// the image of a 128-row tile, which is what the prompt-pass GEMM loads.  One thread per 16-byte chunk.
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
  const long long tile = n / kTileN;
  const int r = (int)(n % kTileN), k = cc >> 3, c = cc & 7;
  uint8_t* blk = dst + ((size_t)tile * kb + k) * (size_t)kBlockBytes;
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

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 t = __bfloat1622float2(p[j]);
    f[2 * j] = t.x;
    f[2 * j + 1] = t.y;
  }
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

// ---- sampling at a temperature (Sec. 4.2 generates at T = 0.5) ------------------------------------------
// A draw from softmax(logits / T) is taken as argmax_v(logit_v / T + g_v) with Gumbel noise g_v = -log(-log(u_v)):
// every u_v comes from the counter-based generator Philox4x32-10 (Salmon et al., SC'11) at counter
// (vocabulary id, index of the generated token, row key, 0) and key (seed), so the arg-max machinery -- per
// tile, then over tiles, in any order -- yields the same token as a sequential draw would.
struct SampleCfg {
  float inv_temp;        // 1 / T, or 0 for greedy decoding
  uint32_t seed_lo, seed_hi;
};

__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                        uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += W0;
    k1 += W1;
  }
  return c0;
}
// The value whose arg-max decides the token: the logit itself (greedy) or logit / T + Gumbel noise.
__device__ __forceinline__ float decision_value(float logit, const SampleCfg& sc, int v, int gen_index, int row_key) {
  if (sc.inv_temp == 0.f) return logit;
  const uint32_t w = philox4x32_10_word0((uint32_t)v, (uint32_t)gen_index, (uint32_t)row_key, 0u, sc.seed_lo, sc.seed_hi);
  const float u = ((float)(w >> 9) + 0.5f) * (1.0f / 8388608.0f);      // 24 significant bits, never 0 or 1
  return fmaf(logit, sc.inv_temp, -logf(-logf(u)));
}

__global__ void __launch_bounds__(128)
lmhead_tile_argmax_kernel(const float* __restrict__ partial, SplitInfo sp, RowState st, float* __restrict__ dump_logits,
                          float* __restrict__ tile_val, int32_t* __restrict__ tile_idx, int B, int vocab, int n_tiles,
                          int eos_id, SampleCfg sc) {
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
        if (!(st.eos_at[r] > 0 && v == eos_id))
          key = float_order_key(decision_value(lg, sc, v, st.gen[r] + 1, st.row_key[r]));
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
                   const int32_t* __restrict__ forced, int32_t* __restrict__ next_tokens, int32_t* __restrict__ dump_choice,
                   int B, int eos_id, int is_prefill) {
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
        if (dump_choice) dump_choice[r] = tok;
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

// RoPE on q and k of the packed fp32 [T, 3d] projection, one rounding to bf16 afterwards: q, k, v go to the packed
// bf16 [T, 3d] operand of the prompt-pass attention and k, v into the pages.
// grid (T), block 256 = (256 / (Dh/2)) heads side by side x Dh/2 rotation pairs; the sine and cosine of a
// (token, pair) are computed once and used for every head.  tok_row / tok_pos give each token's row in the
// batch and position.
__global__ void __launch_bounds__(256)
rope_append_prefill_kernel(const float* __restrict__ qkv_f, bf16* __restrict__ qkv, const int32_t* __restrict__ tok_row,
                           const int32_t* __restrict__ tok_pos, RowState st, KvLayout kv, int layer,
                           const float* __restrict__ inv_freq, int d, uint32_t* status) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t t = blockIdx.x;
  const int r = tok_row[t], pos = tok_pos[t];
  const int Dh = kv.Dh, half = Dh >> 1;
  const int i = threadIdx.x % half, hsub = threadIdx.x / half, hpar = blockDim.x / half;
  float sn, cs;
  sincosf((float)pos * inv_freq[i], &sn, &cs);
  const int page = st.block_table[(size_t)r * st.max_pages + pos / kPageTokens];
  if (page < 0 || page >= kv.n_pages) {
    atomicCAS(status, 0u, (uint32_t)kStatusBadPage);
    return;
  }
  for (int hd = hsub; hd < kv.H; hd += hpar) {
    const float* qf = qkv_f + t * 3 * d + hd * Dh;
    const float* kf = qf + d;
    const float* vf = kf + d;
    bf16* q = qkv + t * 3 * d + hd * Dh;
    bf16* k = q + d;
    bf16* v = k + d;
    const float q0 = qf[i], q1 = qf[i + half], k0 = kf[i], k1 = kf[i + half];
    const bf16 kr0 = __float2bfloat16_rn(k0 * cs - k1 * sn), kr1 = __float2bfloat16_rn(k1 * cs + k0 * sn);
    const bf16 v0 = __float2bfloat16_rn(vf[i]), v1 = __float2bfloat16_rn(vf[i + half]);
    q[i] = __float2bfloat16_rn(q0 * cs - q1 * sn);
    q[i + half] = __float2bfloat16_rn(q1 * cs + q0 * sn);
    k[i] = kr0;
    k[i + half] = kr1;
    v[i] = v0;
    v[i + half] = v1;
    bf16* kbase = kv.pool + (size_t)layer * kv.layer_stride + (size_t)page * kv.page_elems +
                  ((size_t)hd * kPageTokens + (pos % kPageTokens)) * Dh;
    bf16* vbase = kbase + (size_t)kv.H * kPageTokens * Dh;
    kbase[i] = kr0;
    kbase[i + half] = kr1;
    vbase[i] = v0;
    vbase[i + half] = v1;
  }
}

// Causal attention over one prompt on the tensor cores (warp-level mma, m16n8k16, bf16 in, fp32 out).
// CTA = (64 queries, head, sequence), four warps of 16 queries; keys and values are staged through shared
// memory 32 at a time (values transposed, so that both B operands are read as pairs of consecutive
// elements); online softmax on the accumulator fragments; the probabilities are re-used in registers as the
// A operand of P.V.  qkv: [T, 3d] with RoPE applied; out: [T, d].
// Fragment layout of mma.m16n8k16 (g = lane / 4, q = lane % 4): A regs 0..3 hold rows g, g+8, g, g+8 and
// columns 2q..2q+1 (regs 0,1) or 2q+8..2q+9 (regs 2,3); B regs 0,1 hold k = 2q..2q+1 and 2q+8..2q+9 of
// column g; C regs 0,1 hold row g, columns 2q..2q+1, regs 2,3 row g+8.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

template <int DH>
__global__ void __launch_bounds__(128)
attn_prefill_kernel(const bf16* __restrict__ qkv, const int32_t* __restrict__ cu_seqlens, bf16* __restrict__ out, int d) {
  constexpr int QT = 64, KT = 32, KS = DH / 16, NB = DH / 8;
  constexpr int KPAD = DH + 8;                     // padded rows: conflict-free fragment loads
  constexpr int VPAD = KT + 8;
  __shared__ __align__(16) bf16 s_k[KT][KPAD];     // [key][dim]
  __shared__ __align__(16) bf16 s_vt[DH][VPAD];    // [dim][key]
  pdl_launch_dependents();
  pdl_wait();
  const int hd = blockIdx.y, s = blockIdx.z;
  const int seq0 = cu_seqlens[s], len = cu_seqlens[s + 1] - seq0;
  const int qt0 = blockIdx.x * QT;
  if (qt0 >= len) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q4 = lane & 3;
  const int row0 = qt0 + warp * 16 + g, row1 = row0 + 8;     // this thread's two query positions
  const float qscale = rsqrtf((float)DH) * 1.4426950408889634f;

  // Q fragments, kept for the whole kernel (rows beyond the prompt read row len-1: valid memory, never stored)
  uint32_t qa[KS][4];
  {
    const bf16* q0 = qkv + (size_t)(seq0 + min(row0, len - 1)) * 3 * d + hd * DH + q4 * 2;
    const bf16* q1 = qkv + (size_t)(seq0 + min(row1, len - 1)) * 3 * d + hd * DH + q4 * 2;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = *reinterpret_cast<const uint32_t*>(q0 + ks * 16);
      qa[ks][1] = *reinterpret_cast<const uint32_t*>(q1 + ks * 16);
      qa[ks][2] = *reinterpret_cast<const uint32_t*>(q0 + ks * 16 + 8);
      qa[ks][3] = *reinterpret_cast<const uint32_t*>(q1 + ks * 16 + 8);
    }
  }
  float o[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }
  float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;

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
      const bf16* pv = reinterpret_cast<const bf16*>(&uv);
#pragma unroll
      for (int e = 0; e < 8; ++e) s_vt[cc * 8 + e][kr] = pv[e];
    }
    __syncthreads();
    if (kt0 > qt0 + warp * 16 + 15) continue;      // every key of the tile is after this warp's last query

    // S = Q K^T for 16 queries x 32 keys
    float sc[KT / 8][4];
#pragma unroll
    for (int nb = 0; nb < KT / 8; ++nb) {
      sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(&s_k[nb * 8 + g][ks * 16 + q4 * 2]);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(&s_k[nb * 8 + g][ks * 16 + q4 * 2 + 8]);
        mma_bf16_16816(sc[nb], qa[ks], b0, b1);
      }
    }
    // scale, causal / length mask, running maxima
    float mx0 = m0, mx1 = m1;
#pragma unroll
    for (int nb = 0; nb < KT / 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = kt0 + nb * 8 + q4 * 2 + e;
        sc[nb][e] = (key <= row0 && key < len) ? sc[nb][e] * qscale : -CUDART_INF_F;
        sc[nb][2 + e] = (key <= row1 && key < len) ? sc[nb][2 + e] * qscale : -CUDART_INF_F;
        mx0 = fmaxf(mx0, sc[nb][e]);
        mx1 = fmaxf(mx1, sc[nb][2 + e]);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float r0s = (mx0 == -CUDART_INF_F) ? 1.f : exp2f(m0 - mx0);     // exp2f(-inf) = 0 on the first tile
    const float r1s = (mx1 == -CUDART_INF_F) ? 1.f : exp2f(m1 - mx1);
    m0 = mx0;
    m1 = mx1;
    l0 *= r0s;
    l1 *= r1s;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      o[nb][0] *= r0s; o[nb][1] *= r0s;
      o[nb][2] *= r1s; o[nb][3] *= r1s;
    }
    // probabilities, as A fragments of P V (two 16-key steps)
    uint32_t pa[KT / 16][4];
#pragma unroll
    for (int nb = 0; nb < KT / 8; ++nb) {
      float p[4];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        p[e] = (sc[nb][e] == -CUDART_INF_F) ? 0.f : exp2f(sc[nb][e] - m0);
        p[2 + e] = (sc[nb][2 + e] == -CUDART_INF_F) ? 0.f : exp2f(sc[nb][2 + e] - m1);
      }
      l0 += p[0] + p[1];
      l1 += p[2] + p[3];
      pa[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16x2(p[0], p[1]);
      pa[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16x2(p[2], p[3]);
    }
    // O += P V
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
      for (int kk = 0; kk < KT / 16; ++kk) {
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(&s_vt[nb * 8 + g][kk * 16 + q4 * 2]);
        const uint32_t b1 = *reinterpret_cast<const uint32_t*>(&s_vt[nb * 8 + g][kk * 16 + q4 * 2 + 8]);
        mma_bf16_16816(o[nb], pa[kk], b0, b1);
      }
    }
  }
  // row sums over the four lanes of a row, then the output
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = 1.f / l0, i1 = 1.f / l1;
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    if (row0 < len)
      *reinterpret_cast<uint32_t*>(out + (size_t)(seq0 + row0) * d + hd * DH + nb * 8 + q4 * 2) =
          pack_bf16x2(o[nb][0] * i0, o[nb][1] * i0);
    if (row1 < len)
      *reinterpret_cast<uint32_t*>(out + (size_t)(seq0 + row1) * d + hd * DH + nb * 8 + q4 * 2) =
          pack_bf16x2(o[nb][2] * i1, o[nb][3] * i1);
  }
}

// act[t][f] = silu(gu[t][f]) * gu[t][F+f] over T tokens (gu fp32, act bf16: one rounding), 8 features per thread
// (F a multiple of 8).  grid (T, ceil(F / 2048)), block 256.
__global__ void __launch_bounds__(256)
swiglu_kernel(const float* __restrict__ gu, bf16* __restrict__ act, int F) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t t = blockIdx.x;
  const int f0 = (blockIdx.y * blockDim.x + threadIdx.x) * 8;
  if (f0 >= F) return;
  const float4* g4 = reinterpret_cast<const float4*>(gu + t * 2 * F + f0);
  const float4* u4 = reinterpret_cast<const float4*>(gu + t * 2 * F + F + f0);
  const float4 ga = g4[0], gb = g4[1], ua = u4[0], ub = u4[1];
  const float gt[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
  const float up[8] = {ua.x, ua.y, ua.z, ua.w, ub.x, ub.y, ub.z, ub.w};
  __align__(16) bf16 ob[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) ob[j] = __float2bfloat16_rn(gt[j] / (1.f + __expf(-gt[j])) * up[j]);
  *reinterpret_cast<uint4*>(act + t * F + f0) = *reinterpret_cast<const uint4*>(ob);
}

}  // namespace ss
