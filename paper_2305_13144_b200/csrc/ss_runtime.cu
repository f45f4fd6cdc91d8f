// Host runtime behind the C ABI: context, arena carve-up, weight repacking, key/value page
// allocator, kernel sequencing (prompt pass, decode steps) and the group loop of Sec. 4.1
// (micro-batches, caps, failure collection and recomputation).
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "ss_decode_mega.cuh"

using namespace ss;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t kAlign = 1024;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int round_up(int a, int b) { return ceil_div(a, b) * b; }

// Projection matrices live in the tiled streaming layout (see repack_weights_kernel).
struct LayerWeights {
  bf16 *attn_norm, *ffn_norm;
  uint8_t *wqkv, *wo, *wgu, *wdown;
};

inline size_t tiled_bytes(int64_t n_out, int64_t K) {
  return (size_t)ceil_div((int)n_out, kTileN) * ceil_div((int)K, kTileK) * (size_t)kBlockBytes;
}

// Split of a decode projection: 256-row tiles x k-blocks in equal contiguous ranges over the CTAs.
struct DecodeSplit {
  int n_tiles, kb, gsplit, max_seg;
  long long total;
};
DecodeSplit plan_decode(int n_out, int K, int n_sm) {
  DecodeSplit p{};
  p.n_tiles = ceil_div(n_out, kTileN);
  p.kb = ceil_div(K, kTileK);
  p.total = (long long)p.n_tiles * p.kb;
  p.gsplit = (int)std::min<long long>(n_sm, p.total);
  const int ipc = std::max(1, (int)((p.total + p.gsplit - 1) / p.gsplit));
  p.max_seg = (ipc + p.kb - 2) / p.kb + 1;
  return p;
}

GemmPlan plan_gemm(int n_out, int K, int NT, int tok_tiles, int mode, int n_sm) {
  GemmPlan p{};
  p.n_out = n_out;
  p.K = K;
  p.n_tiles = ceil_div(n_out, kTileM);
  p.kb = ceil_div(K, kTileK);
  p.NT = NT;
  const long long total = (long long)p.n_tiles * p.kb;
  if (mode == kGemmPartial) {
    p.gridx = (int)std::min<long long>(n_sm, total);
    p.gridy = 1;
  } else {
    p.gridx = p.n_tiles;
    p.gridy = tok_tiles;
  }
  const int ipc = std::max(1, (int)((total + p.gridx - 1) / p.gridx));
  p.max_seg = (ipc + p.kb - 2) / p.kb + 1;
  const int stage_bytes = kTileM * kTileK * 2 + NT * kTileK * 2;
  const int budget = 227 * 1024 - 2048;                       // header + alignment slack
  p.stages = std::max(2, std::min(kGemmMaxStages, budget / stage_bytes));
  p.smem_bytes = 2048 + p.stages * stage_bytes;
  int cols = 32;
  while (cols < 2 * NT) cols <<= 1;
  p.tmem_cols = cols;
  return p;
}

SplitInfo split_of(const GemmPlan& p, const TileSeg* tiles) {
  SplitInfo s;
  s.gridx = p.gridx;
  s.kb = p.kb;
  s.max_seg = p.max_seg;
  s.NT = p.NT;
  s.total = (long long)p.n_tiles * p.kb;
  s.tiles = tiles;
  return s;
}

// Per tile: where its partial segments live (depends on the split only, not on the token tile).
std::vector<TileSeg> tile_table(const GemmPlan& p) {
  SplitInfo s = split_of(p, nullptr);
  std::vector<TileSeg> t(p.n_tiles);
  for (int tile = 0; tile < p.n_tiles; ++tile) {
    const long long x0 = (long long)tile * p.kb;
    const int c0 = split_owner(s, x0), c1 = split_owner(s, x0 + p.kb - 1);
    const int seg0 = tile - (int)(split_begin(s, c0) / p.kb);
    t[tile] = {c0 * p.max_seg + seg0, c0 + 1, c1, 0};
  }
  return t;
}

std::vector<TileSeg> decode_tile_table(const DecodeSplit& p) {
  SplitInfo s{};
  s.gridx = p.gsplit;
  s.kb = p.kb;
  s.max_seg = p.max_seg;
  s.total = p.total;
  std::vector<TileSeg> t(p.n_tiles);
  for (int tile = 0; tile < p.n_tiles; ++tile) {
    const long long x0 = (long long)tile * p.kb;
    const int c0 = split_owner(s, x0), c1 = split_owner(s, x0 + p.kb - 1);
    const int seg0 = tile - (int)(split_begin(s, c0) / p.kb);
    t[tile] = {c0 * p.max_seg + seg0, c0 + 1, c1, 0};
  }
  return t;
}

}  // namespace

struct ss_ctx {
  ss_model_cfg m;
  ss_runtime_cfg rt;
  cudaStream_t stream;
  int n_sm = 0;
  bool use_pdl = true;
  bool trace_on = false;
  long long wait_limit = 4000000000LL;   // SM cycles (about 2 s) any wait inside a kernel may last
  int clock_khz = 1965000;
  int last_cuda = 0;
  int64_t launches = 0;
  EncodeTiledFn encode = nullptr;

  // ---- arena
  uint8_t* arena = nullptr;
  size_t arena_bytes = 0;
  // weights
  bf16 *embed = nullptr, *final_norm = nullptr;
  uint8_t* lm_head = nullptr;
  uint8_t* staging = nullptr;      // one row-major tensor on its way into the tiled layout
  size_t staging_bytes = 0;
  std::vector<LayerWeights> layers;
  std::vector<uint8_t> loaded;     // per tensor slot
  int n_loaded = 0, n_expected = 0;
  // misc device
  float* inv_freq = nullptr;
  uint32_t* status = nullptr;
  RowState st{};
  KvLayout kv{};
  int32_t *d_tokens = nullptr, *d_tok_row = nullptr, *d_tok_pos = nullptr, *d_cu = nullptr, *d_last = nullptr;
  // prompt-pass activations (R rows)
  int R = 0;
  float* h = nullptr;
  bf16 *x = nullptr, *qkv = nullptr, *attn_o = nullptr, *act = nullptr;
  float *qkv_f = nullptr, *gu = nullptr;   // q,k,v and gate/up as they leave their GEMMs (fp32: rounded once, after RoPE / SwiGLU)
  // decode activations (kMaxBatch rows)
  float* h_dec = nullptr;
  bf16 *x_dec = nullptr, *o_dec = nullptr, *act_dec = nullptr;
  float* partial = nullptr;
  size_t partial_bytes = 0;
  TileSeg* tbl[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};   // decode step: qkv, o, gate/up, down, lm head
  TileSeg* tbl_lm_prompt = nullptr;                                  // LM head after the prompt pass (128-row tiles)
  float* rowss = nullptr;          // [kMaxBatch][kMaxSlices]
  unsigned long long* grid_ctr = nullptr;
  unsigned long long* trace = nullptr;  // stage-boundary time stamps of the last decode step
  int trace_len = 0;
  unsigned long long grid_epochs = 0;   // grid barriers passed by all launches so far
  const uint8_t** wptr_dev = nullptr;
  const bf16** norm_dev = nullptr;
  float* tile_val = nullptr;       // [kMaxBatch][n_tiles of the vocabulary]
  int32_t* tile_idx = nullptr;
  int n_tiles_lm = 0;
  // tensor maps for activation operands, keyed by (buffer id, box rows)
  std::map<std::pair<int, int>, CUtensorMap> xmaps;
  // the tiled projection matrices seen as lines of 128 bytes (for the paired prompt-pass GEMM), [4 * layer + type]
  std::vector<CUtensorMap> wmaps;

  // ---- page allocator
  std::vector<int32_t> free_pages;
  std::vector<int32_t> batch_pages;      // pages that go back to the pool when the batch in flight is released
  // ---- kept prompts (App. C: the instruction's keys and values computed once, for the perception pass, and used
  // again by the generation): pages that outlive the batch that filled them, by caller-chosen id
  struct KeptPrompt {
    std::vector<int32_t> pages;          // covering positions [0, len)
    int32_t len;                         // tokens kept
    int32_t last_tok;                    // token at position len - 1 (fed again when a batch resumes from here)
  };
  std::map<int32_t, KeptPrompt> kept;
  std::vector<std::vector<int32_t>> row_pages;   // batch in flight: every row's pages in block-table order
  std::vector<int32_t> batch_tokens, batch_cu;   // its prompts (host copy), empty for a resumed batch
  int prompt_cache_mode = 0;                     // ss_run_group / ss_run_batches: 0 off, 1 keep, 2 resume
  std::vector<int32_t> cache_keep_len;           // mode 1: tokens to keep per query

  // ---- batch state (host mirror)
  int B = 0;
  int cap = 0;
  bool in_batch = false;
  std::vector<int32_t> prompt_len;
  int32_t* pinned = nullptr;     // [0] n_active, [1] status
  // ---- sampling (greedy while inv_temp == 0)
  SampleCfg sample{0.f, 0u, 0u};
  std::vector<int32_t> next_row_keys;   // keys of the next batch's rows; empty = 0, 1, 2, ...
};

namespace {

int cuda_fail(ss_ctx* c, cudaError_t e) {
  c->last_cuda = (int)e;
  return SS_ERR_CUDA;
}
#define SS_CUDA(c, expr)                                \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) return cuda_fail((c), _e);   \
  } while (0)

template <class... KArgs, class... Args>
cudaError_t launch(ss_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = c->use_pdl ? 1 : 0;
  c->launches++;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

int make_map(ss_ctx* c, CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    c->last_cuda = (int)r;
    return SS_ERR_CUDA;
  }
  return SS_OK;
}

// A tiled weight matrix as a 2-D tensor of 128-byte lines (64 bf16 each); box = 128 lines = one CTA's half of a block.
// The lines already hold the swizzled shared-memory image, so the copy itself does not swizzle.
int make_line_map(ss_ctx* c, CUtensorMap* out, const void* base, size_t bytes) {
  cuuint64_t dims[2] = {(cuuint64_t)kTileK, (cuuint64_t)(bytes / 128)};
  cuuint64_t strides[1] = {128};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)kTileM};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    c->last_cuda = (int)r;
    return SS_ERR_CUDA;
  }
  return SS_OK;
}

// activation operand map (cached): id 0 = x, 1 = attn_o, 2 = act (prompt pass); 3 = x_dec, 4 = o_dec, 5 = act_dec
int xmap(ss_ctx* c, int id, int box_rows, const CUtensorMap** out) {
  auto key = std::make_pair(id, box_rows);
  auto it = c->xmaps.find(key);
  if (it == c->xmaps.end()) {
    const int d = c->m.d_model, F = c->m.d_ffn;
    const void* base = nullptr;
    int64_t rows = 0, cols = 0;
    switch (id) {
      case 0: base = c->x; rows = c->R; cols = d; break;
      case 1: base = c->attn_o; rows = c->R; cols = d; break;
      case 2: base = c->act; rows = c->R; cols = F; break;
      case 3: base = c->x_dec; rows = kMaxBatch; cols = d; break;
      case 4: base = c->o_dec; rows = kMaxBatch; cols = d; break;
      default: base = c->act_dec; rows = kMaxBatch; cols = F; break;
    }
    CUtensorMap m;
    int rc = make_map(c, &m, base, rows, cols, box_rows);
    if (rc != SS_OK) return rc;
    it = c->xmaps.emplace(key, m).first;
  }
  *out = &it->second;
  return SS_OK;
}

int run_gemm(ss_ctx* c, const uint8_t* w_tiled, const CUtensorMap& mx, const GemmPlan& p, int mode, int n_tok,
             void* out_bf16, float* out_f32, int ld_out) {
  GemmArgs a{};
  a.p = p;
  a.w_tiled = w_tiled;
  a.mode = mode;
  a.n_tok = n_tok;
  a.partial = c->partial;
  a.out_bf16 = out_bf16;
  a.out_f32 = out_f32;
  a.ld_out = ld_out;
  a.status = c->status;
  if (mode == kGemmPartial) {
    const size_t need = (size_t)p.gridx * p.max_seg * p.NT * 128 * sizeof(float);
    if (need > c->partial_bytes) return SS_ERR_CAPACITY;
  }
  // the weight tensor map is unused with tiled weights; the activation map stands in for it
  SS_CUDA(c, launch(c, gemm_wx_kernel, dim3(p.gridy, p.gridx), dim3(kGemmThreads), (size_t)p.smem_bytes, mx, mx, a));
  return SS_OK;
}

// The same product on pairs of CTAs (gemm_wx_pair_kernel): token tiles of 256, direct epilogues only.
int run_gemm_pair(ss_ctx* c, const CUtensorMap& mw, const CUtensorMap& mx, int n_out, int K, int mode, int n_tok,
                  void* out_bf16, float* out_f32, int ld_out) {
  GemmArgs a{};
  a.p.n_out = n_out;
  a.p.K = K;
  a.p.n_tiles = 2 * ceil_div(n_out, kTileN);
  a.p.kb = ceil_div(K, kTileK);
  a.p.NT = kPairTokens;
  a.p.stages = std::min(kGemmMaxStages, (227 * 1024 - 2048) / kPairStageBytes);
  a.p.smem_bytes = 2048 + a.p.stages * kPairStageBytes;
  a.mode = mode;
  a.n_tok = n_tok;
  a.out_bf16 = out_bf16;
  a.out_f32 = out_f32;
  a.ld_out = ld_out;
  a.status = c->status;
  a.p.gridy = ceil_div(n_tok, kPairTokens);                          // token tiles
  const int n_units = (a.p.n_tiles / 2) * a.p.gridy;
  a.p.gridx = std::min(n_units, c->n_sm / 2);                        // pairs of CTAs, each walking its units
  SS_CUDA(c, launch(c, gemm_wx_pair_kernel, dim3(2 * a.p.gridx), dim3(kGemmThreads), (size_t)a.p.smem_bytes, mw, mx, a));
  return SS_OK;
}

struct ArenaPlan {
  size_t total = 0;
  size_t take(size_t bytes) {
    size_t off = total;
    total = align_up(total + bytes);
    return off;
  }
};

struct Offsets {
  size_t embed, lm_head, final_norm, staging, staging_bytes, weights_end;
  std::vector<size_t> attn_norm, wqkv, wo, ffn_norm, wgu, wdown;
  size_t inv_freq, status, rows, block_table, out_tokens, tok, h, x, qkv, qkv_f, attn_o, gu, act;
  size_t h_dec, x_dec, o_dec, act_dec, partial, kv;
  size_t tbl[5], tbl_lm_prompt, tile_val, tile_idx, rowss, grid_ctr, wptr, norm_ptr, trace;
  size_t partial_bytes;
  int R, max_pages, n_pages;
  size_t total;
};

int validate_model(const ss_model_cfg* m, const ss_runtime_cfg* rt) {
  if (!m || !rt) return SS_ERR_ARG;
  if (m->n_layers < 0 || m->d_model <= 0 || m->n_heads <= 0 || m->d_ffn <= 0 || m->vocab <= 0) return SS_ERR_ARG;
  if (m->eos_id < 0 || m->eos_id >= m->vocab) return SS_ERR_ARG;
  if (m->n_heads * m->head_dim != m->d_model) return SS_ERR_ARG;
  if (m->head_dim != 64 && m->head_dim != 128) return SS_ERR_UNSUPPORTED;
  if (m->d_model % 64 || m->d_model > 8192 || m->d_ffn % 8) return SS_ERR_UNSUPPORTED;
  if (rt->max_batch < 1 || rt->max_batch > kMaxBatch) return SS_ERR_ARG;
  if (rt->max_ctx < 2 || rt->max_prefill_tokens < 1 || rt->max_new_tokens < 1 || rt->kv_pool_tokens < 1) return SS_ERR_ARG;
  return SS_OK;
}

void layout(const ss_model_cfg& m, const ss_runtime_cfg& rt, int n_sm, Offsets& o) {
  ArenaPlan a;
  const size_t d = m.d_model, F = m.d_ffn, V = m.vocab;
  o.embed = a.take(V * d * 2);
  o.attn_norm.resize(m.n_layers); o.wqkv.resize(m.n_layers); o.wo.resize(m.n_layers);
  o.ffn_norm.resize(m.n_layers); o.wgu.resize(m.n_layers); o.wdown.resize(m.n_layers);
  for (int l = 0; l < m.n_layers; ++l) {
    o.attn_norm[l] = a.take(d * 2);
    o.wqkv[l] = a.take(tiled_bytes(3 * d, d));
    o.wo[l] = a.take(tiled_bytes(d, d));
    o.ffn_norm[l] = a.take(d * 2);
    o.wgu[l] = a.take(tiled_bytes(2 * F, d));
    o.wdown[l] = a.take(tiled_bytes(d, F));
  }
  o.final_norm = a.take(d * 2);
  o.lm_head = a.take(tiled_bytes(V, d));
  o.weights_end = a.total;
  o.staging_bytes = std::max(std::max(V * d, F * d), d * d) * 2;
  o.staging = a.take(o.staging_bytes);
  o.inv_freq = a.take(m.head_dim / 2 * sizeof(float));
  o.status = a.take(64);
  o.rows = a.take((size_t)kMaxBatch * 4 * 8 + 64);           // 7 row arrays + scalars
  o.max_pages = ceil_div(rt.max_ctx, kPageTokens);
  o.block_table = a.take((size_t)kMaxBatch * o.max_pages * 4);
  o.out_tokens = a.take((size_t)kMaxBatch * rt.max_new_tokens * 4);
  o.R = round_up(std::max(rt.max_prefill_tokens, kMaxBatch), 256);
  o.tok = a.take(((size_t)o.R * 3 + 2 * kMaxBatch + 8) * 4);
  o.h = a.take((size_t)o.R * d * 4);
  o.x = a.take((size_t)o.R * d * 2);
  o.qkv = a.take((size_t)o.R * 3 * d * 2);
  o.qkv_f = a.take((size_t)o.R * 3 * d * 4);
  o.attn_o = a.take((size_t)o.R * d * 2);
  o.gu = a.take((size_t)o.R * 2 * F * 4);
  o.act = a.take((size_t)o.R * F * 2);
  o.h_dec = a.take((size_t)kMaxBatch * d * 4);
  o.x_dec = a.take((size_t)kMaxBatch * d * 2);
  o.o_dec = a.take((size_t)kMaxBatch * d * 2);
  o.act_dec = a.take((size_t)kMaxBatch * F * 2);
  // partial work space: the largest decode GEMM at the widest token tile
  const int NTmax = round_up(rt.max_batch, 16);
  size_t pb = 0;
  const int shapes[5][2] = {{(int)(3 * d), (int)d}, {(int)d, (int)d}, {(int)(2 * F), (int)d}, {(int)d, (int)F}, {(int)V, (int)d}};
  for (auto& s : shapes) {
    const DecodeSplit p = plan_decode(s[0], s[1], n_sm);
    pb = std::max(pb, (size_t)p.gsplit * p.max_seg * NTmax * kTileN * sizeof(float));
  }
  {
    const GemmPlan p = plan_gemm((int)V, (int)d, NTmax, 1, kGemmPartial, n_sm);
    pb = std::max(pb, (size_t)p.gridx * p.max_seg * p.NT * 128 * sizeof(float));
  }
  o.partial_bytes = pb;
  o.partial = a.take(pb);
  o.rowss = a.take((size_t)kMaxBatch * kMaxSlices * 4);
  o.grid_ctr = a.take(64);
  o.wptr = a.take((size_t)(4 * m.n_layers + 1) * sizeof(void*));
  o.norm_ptr = a.take((size_t)(2 * m.n_layers + 1) * sizeof(void*));
  o.trace = a.take((size_t)(2 + 4 * (4 * m.n_layers + 1)) * 8);
  for (int i = 0; i < 5; ++i) o.tbl[i] = a.take((size_t)ceil_div(shapes[i][0], kTileN) * sizeof(TileSeg));
  o.tbl_lm_prompt = a.take((size_t)ceil_div((int)V, kTileM) * sizeof(TileSeg));
  o.tile_val = a.take((size_t)kMaxBatch * ceil_div((int)V, kTileM) * 4);
  o.tile_idx = a.take((size_t)kMaxBatch * ceil_div((int)V, kTileM) * 4);
  o.n_pages = (int)((rt.kv_pool_tokens + kPageTokens - 1) / kPageTokens) + rt.max_batch;
  const size_t page_bytes = (size_t)2 * m.n_heads * kPageTokens * m.head_dim * 2;
  o.kv = a.take((size_t)std::max(1, m.n_layers) * o.n_pages * page_bytes);
  o.total = a.total;
}

// SMs of the current device; 148 (a B200) when no device can be asked, e.g. when sizing an arena on a host
// without a GPU.
int query_sms() {
  int dev = 0, n = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) n = v;
  }
  return n;
}

struct WeightSlot {
  void* dst;          // plain tensors: destination; tiled: base of the tiled matrix
  int64_t rows, cols; // expected shape of the source
  int slot;
  bool tiled;
  int row_off;        // tiled: row offset inside the stacked matrix
};

int weight_slot(const ss_ctx* c, const std::string& name, WeightSlot* out) {
  const int64_t d = c->m.d_model, F = c->m.d_ffn, V = c->m.vocab;
  auto plain = [&](void* p, int64_t r, int64_t cc, int s) { *out = {p, r, cc, s, false, 0}; return SS_OK; };
  auto tiled = [&](void* p, int64_t r, int64_t cc, int s, int64_t off) { *out = {p, r, cc, s, true, (int)off}; return SS_OK; };
  if (name == "embed") return plain(c->embed, V, d, 0);
  if (name == "lm_head") return tiled(c->lm_head, V, d, 1, 0);
  if (name == "final_norm") return plain(c->final_norm, 1, d, 2);
  if (name.size() > 2 && name[0] == 'l') {
    size_t dot = name.find('.');
    if (dot == std::string::npos) return SS_ERR_ARG;
    int l = atoi(name.substr(1, dot - 1).c_str());
    if (l < 0 || l >= c->m.n_layers) return SS_ERR_ARG;
    const std::string k = name.substr(dot + 1);
    const LayerWeights& w = c->layers[l];
    const int base = 3 + l * 9;
    if (k == "attn_norm") return plain(w.attn_norm, 1, d, base + 0);
    if (k == "wq") return tiled(w.wqkv, d, d, base + 1, 0);
    if (k == "wk") return tiled(w.wqkv, d, d, base + 2, d);
    if (k == "wv") return tiled(w.wqkv, d, d, base + 3, 2 * d);
    if (k == "wo") return tiled(w.wo, d, d, base + 4, 0);
    if (k == "ffn_norm") return plain(w.ffn_norm, 1, d, base + 5);
    if (k == "w_gate") return tiled(w.wgu, F, d, base + 6, 0);
    if (k == "w_up") return tiled(w.wgu, F, d, base + 7, F);
    if (k == "w_down") return tiled(w.wdown, d, F, base + 8, 0);
  }
  return SS_ERR_ARG;
}

// A non-zero status word: the step that set it was abandoned half way.  The error is reported once; the word
// and the grid-barrier counter (left in an unknown state by the abort) are cleared so that the context can
// start a new batch.
int report_device_status(ss_ctx* c, uint32_t word) {
  cudaMemsetAsync(c->grid_ctr, 0, 8, c->stream);
  cudaMemsetAsync(c->status, 0, 4, c->stream);
  cudaStreamSynchronize(c->stream);
  c->grid_epochs = 0;
  return word == (uint32_t)kStatusBadPage ? SS_ERR_STATE : SS_ERR_DEVICE_TIMEOUT;
}

double weight_bytes_per_step(const ss_model_cfg& m) {
  const double d = m.d_model, F = m.d_ffn, V = m.vocab;
  return m.n_layers * (4 * d * d + 3 * d * F + 2 * d) * 2.0 + V * d * 2.0 + d * 2.0;
}
double kv_bytes_per_token(const ss_model_cfg& m) { return 2.0 * m.d_model * 2.0 * m.n_layers; }

// The decode kernel's instantiations: head size 64 / 128, batches up to 64 rows / wider, without / with the stage trace.
template <int DH>
const void* mega_kernel_fn_dh(bool wide, bool trace) {
  if (wide) return trace ? (const void*)decode_step_mega_kernel<DH, true, true> : (const void*)decode_step_mega_kernel<DH, true, false>;
  return trace ? (const void*)decode_step_mega_kernel<DH, false, true> : (const void*)decode_step_mega_kernel<DH, false, false>;
}
const void* mega_kernel_fn(int head_dim, bool wide, bool trace) {
  return head_dim == 128 ? mega_kernel_fn_dh<128>(wide, trace) : mega_kernel_fn_dh<64>(wide, trace);
}

// ------------------------------------------------------------------------------------ decode step
// One cooperative launch of the persistent kernel (see ss_decode_mega.cuh).
int enqueue_decode_step(ss_ctx* c, const ss_step_opts* opts, int32_t* next_tokens) {
  const ss_model_cfg& m = c->m;
  const int B = c->B, d = m.d_model, F = m.d_ffn, V = m.vocab;
  const int NT = round_up(B, 16);
  const CUtensorMap *mx, *mo, *ma;
  int rc;
  const int xr = NT > 128 ? 128 : NT;          // activation rows per TMA load
  if ((rc = xmap(c, 3, xr, &mx)) || (rc = xmap(c, 4, xr, &mo)) || (rc = xmap(c, 5, xr, &ma))) return rc;
  MegaArgs a{};
  a.n_layers = m.n_layers; a.d = d; a.H = m.n_heads; a.Dh = m.head_dim; a.F = F; a.V = V; a.eos_id = m.eos_id;
  a.eps = m.rms_eps;
  a.wptr = c->wptr_dev;
  a.norm_ptr = c->norm_dev;
  a.embed = c->embed;
  a.inv_freq = c->inv_freq;
  const int shp[5][2] = {{3 * d, d}, {d, d}, {2 * F, d}, {d, F}, {V, d}};
  size_t need_partial = 0;
  int tab_entries = 0;
  for (int i = 0; i < 4; ++i) tab_entries += ceil_div(shp[i][0], kTileN);
  int tab_off = 0;
  for (int i = 0; i < 5; ++i) {
    const DecodeSplit p = plan_decode(shp[i][0], shp[i][1], c->n_sm);
    const int off = (i < 4 && tab_entries <= kSegTabEntries) ? tab_off : -1;   // the per-layer tables, if they fit
    tab_off += p.n_tiles;
    a.shape[i] = {p.n_tiles, p.kb, p.max_seg, p.gsplit, p.total, c->tbl[i], off};
    need_partial = std::max(need_partial, (size_t)p.gsplit * p.max_seg * NT * kTileN * sizeof(float));
  }
  if (need_partial > c->partial_bytes) return SS_ERR_CAPACITY;
  a.B = B; a.NT = NT;
  a.m_tiles = NT > 128 ? 2 : 1;
  a.x_rows = NT > 128 ? 128 : NT;
  const int stage_bytes = kBlockBytes + a.m_tiles * a.x_rows * kTileK * 2;
  const int header = (int)sizeof(MegaSmem) + 1024;
  a.stages = std::max(2, std::min(kMegaMaxStages, (227 * 1024 - header) / stage_bytes));
  const size_t smem = (size_t)header + (size_t)a.stages * stage_bytes;
  a.st = c->st; a.kv = c->kv;
  a.h = c->h_dec; a.x = c->x_dec; a.o = c->o_dec; a.act = c->act_dec;
  a.rowss = c->rowss; a.partial = c->partial;
  a.tile_val = c->tile_val; a.tile_idx = c->tile_idx; a.n_tiles_lm = c->n_tiles_lm;
  a.forced = opts ? opts->forced_tokens : nullptr;
  a.next_tokens = next_tokens;
  a.dump_logits = opts ? opts->dump_logits : nullptr;
  a.dump_hidden = opts ? opts->dump_hidden : nullptr;
  a.dump_choice = opts ? opts->dump_choice : nullptr;
  a.sample = c->sample;
  a.grid_ctr = c->grid_ctr;
  a.grid_base = c->grid_epochs * (unsigned long long)c->n_sm;
  a.status = c->status;
  a.trace = c->trace_on ? c->trace : nullptr;
  a.wait_limit = c->wait_limit;
  void* args[4] = {(void*)mx, (void*)mo, (void*)ma, (void*)&a};
  const bool wide = NT > 64;
  const void* fn = mega_kernel_fn(m.head_dim, wide, a.trace != nullptr);
  SS_CUDA(c, cudaLaunchCooperativeKernel(fn, dim3(c->n_sm), dim3(kMegaThreads), args, smem, c->stream));
  c->grid_epochs += 1 + 2 * (unsigned long long)(4 * m.n_layers + 1);
  c->launches++;
  return SS_OK;
}

// ------------------------------------------------------------------------------------ prompt pass (one chunk of whole sequences)
int enqueue_prefill_chunk(ss_ctx* c, int s0, int s1, const int32_t* cu, int T) {
  const ss_model_cfg& m = c->m;
  const int d = m.d_model, F = m.d_ffn, H = m.n_heads, Dh = m.head_dim, V = m.vocab;
  const int nseq = s1 - s0;
  int max_len = 0;
  for (int s = s0; s < s1; ++s) max_len = std::max(max_len, cu[s + 1] - cu[s]);
  // more than half a pair's token tile: the paired kernel (token tiles of 256, two CTAs per 256 x 256 tile)
  const bool pair = T > kPairTokens / 2;
  const int NT = pair ? kPairTokens / 2 : std::min(256, round_up(T, 16));
  const int tok_tiles = ceil_div(T, NT);
  const CUtensorMap *mx, *mo, *ma;
  int rc;
  if ((rc = xmap(c, 0, NT, &mx)) || (rc = xmap(c, 1, NT, &mo)) || (rc = xmap(c, 2, NT, &ma))) return rc;
  const GemmPlan p_qkv = plan_gemm(3 * d, d, NT, tok_tiles, kGemmDirectF32, c->n_sm);
  const GemmPlan p_o = plan_gemm(d, d, NT, tok_tiles, kGemmDirectF32Add, c->n_sm);
  const GemmPlan p_gu = plan_gemm(2 * F, d, NT, tok_tiles, kGemmDirectF32, c->n_sm);
  const GemmPlan p_dn = plan_gemm(d, F, NT, tok_tiles, kGemmDirectF32Add, c->n_sm);
  // one projection: on pairs of CTAs, or one CTA per tile for short chunks
  auto project = [&](int l, int type, const uint8_t* w, const CUtensorMap& act, const GemmPlan& pl, int n_out, int K,
                     int mode, float* out, int ld) -> int {
    if (pair) return run_gemm_pair(c, c->wmaps[4 * l + type], act, n_out, K, mode, T, nullptr, out, ld);
    return run_gemm(c, w, act, pl, mode, T, nullptr, out, ld);
  };
  const bf16* first_norm = m.n_layers ? c->layers[0].attn_norm : c->final_norm;
  SS_CUDA(c, launch(c, embed_rmsnorm_kernel, dim3(T), dim3(256), 0, (const int32_t*)c->d_tokens, (const int32_t*)nullptr,
                    (const bf16*)c->embed, first_norm, c->h, c->x, d, m.rms_eps, V));
  for (int l = 0; l < m.n_layers; ++l) {
    const LayerWeights& w = c->layers[l];
    if ((rc = project(l, 0, w.wqkv, *mx, p_qkv, 3 * d, d, kGemmDirectF32, c->qkv_f, 3 * d))) return rc;
    SS_CUDA(c, launch(c, rope_append_prefill_kernel, dim3(T), dim3(256), 0, (const float*)c->qkv_f, c->qkv, (const int32_t*)c->d_tok_row,
                      (const int32_t*)c->d_tok_pos, c->st, c->kv, l, (const float*)c->inv_freq, d, c->status));
    const dim3 ag(ceil_div(max_len, 64), H, nseq);
    if (Dh == 128)
      SS_CUDA(c, launch(c, attn_prefill_kernel<128>, ag, dim3(128), 0, (const bf16*)c->qkv, (const int32_t*)c->d_cu, c->attn_o, d));
    else
      SS_CUDA(c, launch(c, attn_prefill_kernel<64>, ag, dim3(128), 0, (const bf16*)c->qkv, (const int32_t*)c->d_cu, c->attn_o, d));
    if ((rc = project(l, 1, w.wo, *mo, p_o, d, d, kGemmDirectF32Add, c->h, d))) return rc;
    SS_CUDA(c, launch(c, rmsnorm_kernel, dim3(T), dim3(256), 0, (const float*)c->h, (const bf16*)w.ffn_norm, c->x, d, m.rms_eps));
    if ((rc = project(l, 2, w.wgu, *mx, p_gu, 2 * F, d, kGemmDirectF32, c->gu, 2 * F))) return rc;
    SS_CUDA(c, launch(c, swiglu_kernel, dim3(T, ceil_div(F, 2048)), dim3(256), 0, (const float*)c->gu, c->act, F));
    if ((rc = project(l, 3, w.wdown, *ma, p_dn, d, F, kGemmDirectF32Add, c->h, d))) return rc;
    if (l + 1 < m.n_layers)
      SS_CUDA(c, launch(c, rmsnorm_kernel, dim3(T), dim3(256), 0, (const float*)c->h,
                        (const bf16*)c->layers[l + 1].attn_norm, c->x, d, m.rms_eps));
  }
  return SS_OK;
}

}  // namespace

// ======================================================================================= C ABI
extern "C" {

const char* ss_strerror(int code) {
  switch (code) {
    case SS_OK: return "ok";
    case SS_ERR_ARG: return "bad argument";
    case SS_ERR_CAPACITY: return "buffer or arena too small";
    case SS_ERR_KV_BUDGET: return "batch does not fit the key/value pool";
    case SS_ERR_STATE: return "call out of order";
    case SS_ERR_CUDA: return "CUDA call failed";
    case SS_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
    case SS_ERR_UNSUPPORTED: return "shape not supported by the kernels";
    default: return "unknown error";
  }
}

int ss_arena_bytes(const ss_model_cfg* model, const ss_runtime_cfg* rt, size_t* out_bytes) {
  int rc = validate_model(model, rt);
  if (rc) return rc;
  if (!out_bytes) return SS_ERR_ARG;
  Offsets o;
  layout(*model, *rt, query_sms(), o);  // the split tables and partial sums are sized by the SM count
  *out_bytes = o.total;
  return SS_OK;
}

int ss_create(const ss_model_cfg* model, const ss_runtime_cfg* rt, void* dev_arena, size_t arena_bytes, void* stream,
              ss_ctx** out) {
  int rc = validate_model(model, rt);
  if (rc) return rc;
  if (!dev_arena || !out || ((uintptr_t)dev_arena % kAlign)) return SS_ERR_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) return SS_ERR_CUDA;
  Offsets o;
  const int n_sm = query_sms();
  layout(*model, *rt, n_sm, o);
  if (arena_bytes < o.total) return SS_ERR_CAPACITY;
  ss_ctx* c = new ss_ctx();
  c->m = *model;
  c->rt = *rt;
  c->stream = (cudaStream_t)stream;
  c->n_sm = n_sm;
  {
    int dev = 0, khz = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev) == cudaSuccess && khz > 0)
      c->clock_khz = khz;
  }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn) {
    delete c;
    return SS_ERR_CUDA;
  }
  c->encode = (EncodeTiledFn)fn;
  uint8_t* A = (uint8_t*)dev_arena;
  c->arena = A;
  c->arena_bytes = arena_bytes;
  const int64_t d = model->d_model, F = model->d_ffn, V = model->vocab;
  c->embed = (bf16*)(A + o.embed);
  c->lm_head = A + o.lm_head;
  c->staging = A + o.staging;
  c->staging_bytes = o.staging_bytes;
  c->final_norm = (bf16*)(A + o.final_norm);
  c->layers.resize(model->n_layers);
  auto fail = [&](int code) { delete c; return code; };
  for (int l = 0; l < model->n_layers; ++l) {
    LayerWeights& w = c->layers[l];
    w.attn_norm = (bf16*)(A + o.attn_norm[l]);
    w.wqkv = A + o.wqkv[l];
    w.wo = A + o.wo[l];
    w.ffn_norm = (bf16*)(A + o.ffn_norm[l]);
    w.wgu = A + o.wgu[l];
    w.wdown = A + o.wdown[l];
  }
  // tiles that reach beyond a matrix's rows or columns must read as zero
  if (cudaMemsetAsync(A + o.embed, 0, o.weights_end - o.embed, c->stream) != cudaSuccess) return fail(SS_ERR_CUDA);
  c->n_expected = 3 + 9 * model->n_layers;
  c->loaded.assign(c->n_expected, 0);
  c->inv_freq = (float*)(A + o.inv_freq);
  c->status = (uint32_t*)(A + o.status);
  int32_t* rows = (int32_t*)(A + o.rows);
  c->st.ctx_len = rows + 0 * kMaxBatch;
  c->st.cur_tok = rows + 1 * kMaxBatch;
  c->st.gen = rows + 2 * kMaxBatch;
  c->st.active = rows + 3 * kMaxBatch;
  c->st.finished = rows + 4 * kMaxBatch;
  c->st.eos_at = rows + 5 * kMaxBatch;
  c->st.row_key = rows + 6 * kMaxBatch;
  c->st.scalars = rows + 7 * kMaxBatch;
  c->st.block_table = (int32_t*)(A + o.block_table);
  c->st.out_tokens = (int32_t*)(A + o.out_tokens);
  c->st.max_pages = o.max_pages;
  c->st.max_new = rt->max_new_tokens;
  c->R = o.R;
  int32_t* tk = (int32_t*)(A + o.tok);
  c->d_tokens = tk;
  c->d_tok_row = tk + o.R;
  c->d_tok_pos = tk + 2 * (size_t)o.R;
  c->d_cu = tk + 3 * (size_t)o.R;
  c->d_last = c->d_cu + kMaxBatch + 4;
  c->h = (float*)(A + o.h);
  c->x = (bf16*)(A + o.x);
  c->qkv = (bf16*)(A + o.qkv);
  c->attn_o = (bf16*)(A + o.attn_o);
  c->gu = (float*)(A + o.gu);
  c->qkv_f = (float*)(A + o.qkv_f);
  c->act = (bf16*)(A + o.act);
  c->h_dec = (float*)(A + o.h_dec);
  c->x_dec = (bf16*)(A + o.x_dec);
  c->o_dec = (bf16*)(A + o.o_dec);
  c->act_dec = (bf16*)(A + o.act_dec);
  c->partial = (float*)(A + o.partial);
  c->partial_bytes = o.partial_bytes;
  c->rowss = (float*)(A + o.rowss);
  c->grid_ctr = (unsigned long long*)(A + o.grid_ctr);
  c->wptr_dev = (const uint8_t**)(A + o.wptr);
  c->trace = (unsigned long long*)(A + o.trace);
  c->trace_len = 2 + 4 * (4 * model->n_layers + 1);
  c->norm_dev = (const bf16**)(A + o.norm_ptr);
  {
    std::vector<const uint8_t*> wp;
    std::vector<const bf16*> np;
    for (int l = 0; l < model->n_layers; ++l) {
      const LayerWeights& w = c->layers[l];
      wp.push_back(w.wqkv); wp.push_back(w.wo); wp.push_back(w.wgu); wp.push_back(w.wdown);
      np.push_back(w.attn_norm); np.push_back(w.ffn_norm);
    }
    wp.push_back(c->lm_head);
    np.push_back(c->final_norm);
    if (cudaMemcpy(c->wptr_dev, wp.data(), wp.size() * sizeof(void*), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(c->norm_dev, np.data(), np.size() * sizeof(void*), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(A + o.rowss, 0, o.wptr - o.rowss) != cudaSuccess)
      return fail(SS_ERR_CUDA);
  }
  c->wmaps.resize((size_t)4 * model->n_layers);
  for (int l = 0; l < model->n_layers; ++l) {
    const LayerWeights& w = c->layers[l];
    const uint8_t* base[4] = {w.wqkv, w.wo, w.wgu, w.wdown};
    const size_t bytes[4] = {tiled_bytes(3 * d, d), tiled_bytes(d, d), tiled_bytes(2 * F, d), tiled_bytes(d, F)};
    for (int t = 0; t < 4; ++t)
      if (int rc2 = make_line_map(c, &c->wmaps[4 * l + t], base[t], bytes[t])) return fail(rc2);
  }
  c->tile_val = (float*)(A + o.tile_val);
  c->tile_idx = (int32_t*)(A + o.tile_idx);
  c->n_tiles_lm = ceil_div((int)V, kTileM);
  {
    const int shp[5][2] = {{(int)(3 * d), (int)d}, {(int)d, (int)d}, {(int)(2 * F), (int)d}, {(int)d, (int)F}, {(int)V, (int)d}};
    for (int i = 0; i < 5; ++i) {
      c->tbl[i] = (TileSeg*)(A + o.tbl[i]);
      const std::vector<TileSeg> t = decode_tile_table(plan_decode(shp[i][0], shp[i][1], c->n_sm));
      if (cudaMemcpy(c->tbl[i], t.data(), t.size() * sizeof(TileSeg), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(SS_ERR_CUDA);
    }
    c->tbl_lm_prompt = (TileSeg*)(A + o.tbl_lm_prompt);
    const std::vector<TileSeg> t = tile_table(plan_gemm((int)V, (int)d, 16, 1, kGemmPartial, c->n_sm));
    if (cudaMemcpy(c->tbl_lm_prompt, t.data(), t.size() * sizeof(TileSeg), cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(SS_ERR_CUDA);
  }
  c->kv.pool = (bf16*)(A + o.kv);
  c->kv.page_elems = (size_t)2 * model->n_heads * kPageTokens * model->head_dim;
  c->kv.layer_stride = (size_t)o.n_pages * c->kv.page_elems;
  c->kv.n_pages = o.n_pages;
  c->kv.H = model->n_heads;
  c->kv.Dh = model->head_dim;
  c->free_pages.resize(o.n_pages);
  for (int i = 0; i < o.n_pages; ++i) c->free_pages[i] = o.n_pages - 1 - i;

  // rotary inverse frequencies, exact in double then rounded once
  std::vector<float> inv(model->head_dim / 2);
  for (int i = 0; i < model->head_dim / 2; ++i)
    inv[i] = (float)std::pow((double)model->rope_theta, -2.0 * i / model->head_dim);
  cudaError_t e = cudaMemcpyAsync(c->inv_freq, inv.data(), inv.size() * 4, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->status, 0, 64, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(rows, 0, (size_t)kMaxBatch * 4 * 8 + 64, c->stream);
  // activation operands must be finite wherever a TMA box may reach beyond the valid rows
  if (e == cudaSuccess) e = cudaMemsetAsync(A + o.h, 0, o.partial - o.h, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->pinned, 64, cudaHostAllocDefault);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gemm_wx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gemm_wx_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  for (int v = 0; v < 8 && e == cudaSuccess; ++v)
    e = cudaFuncSetAttribute(mega_kernel_fn((v & 1) ? 128 : 64, (v & 2) != 0, (v & 4) != 0), cudaFuncAttributeMaxDynamicSharedMemorySize,
                             227 * 1024);
  if (e != cudaSuccess) {
    c->last_cuda = (int)e;
    delete c;
    return SS_ERR_CUDA;
  }
  *out = c;
  return SS_OK;
}

int ss_destroy(ss_ctx* c) {
  if (!c) return SS_ERR_ARG;
  cudaStreamSynchronize(c->stream);
  if (c->pinned) cudaFreeHost(c->pinned);
  delete c;
  return SS_OK;
}

int ss_load_weights(ss_ctx* c, const ss_tensor_desc* t, int32_t n) {
  if (!c || (n > 0 && !t) || n < 0) return SS_ERR_ARG;
  for (int i = 0; i < n; ++i) {
    if (!t[i].name || !t[i].data) return SS_ERR_ARG;
    WeightSlot ws;
    int rc = weight_slot(c, t[i].name, &ws);
    if (rc) return rc;
    if (t[i].rows * t[i].cols != ws.rows * ws.cols || (ws.rows > 1 && (t[i].rows != ws.rows || t[i].cols != ws.cols)))
      return SS_ERR_ARG;
    const size_t bytes = (size_t)ws.rows * ws.cols * 2;
    if (!ws.tiled) {
      SS_CUDA(c, cudaMemcpyAsync(ws.dst, t[i].data, bytes,
                                 t[i].is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream));
    } else {
      const void* src = t[i].data;
      if (!t[i].is_device || ((uintptr_t)src & 15)) {
        if (bytes > c->staging_bytes) return SS_ERR_CAPACITY;
        SS_CUDA(c, cudaMemcpyAsync(c->staging, src, bytes,
                                   t[i].is_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice, c->stream));
        src = c->staging;
      }
      const long long chunks = (long long)ws.rows * (ws.cols / 8);
      repack_weights_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, c->stream>>>(
          (const uint4*)src, ws.rows, (int)ws.cols, (uint8_t*)ws.dst, ws.row_off, ceil_div((int)ws.cols, kTileK));
      SS_CUDA(c, cudaGetLastError());
      c->launches++;
      // the staging buffer (or the caller's tensor) is free again once the repack has run
      SS_CUDA(c, cudaStreamSynchronize(c->stream));
    }
    if (!c->loaded[ws.slot]) { c->loaded[ws.slot] = 1; c->n_loaded++; }
  }
  SS_CUDA(c, cudaStreamSynchronize(c->stream));
  return SS_OK;
}

int ss_release_batch(ss_ctx* c) {
  if (!c) return SS_ERR_ARG;
  for (int32_t p : c->batch_pages) c->free_pages.push_back(p);
  c->batch_pages.clear();
  c->row_pages.clear();
  c->in_batch = false;
  c->B = 0;
  return SS_OK;
}

int ss_prefill(ss_ctx* c, const int32_t* tokens, const int32_t* cu, int32_t B, const int32_t* eos_at, int32_t cap,
               const ss_step_opts* opts, int32_t* first_tokens) {
  if (!c || !tokens || !cu || B < 1 || cap < 1) return SS_ERR_ARG;
  if (c->n_loaded != c->n_expected || c->in_batch) return SS_ERR_STATE;
  if (B > c->rt.max_batch || cap > c->rt.max_new_tokens) return SS_ERR_CAPACITY;
  if (cu[0] != 0) return SS_ERR_ARG;
  const ss_model_cfg& m = c->m;
  // admission: pages for the worst case of every row
  size_t need_pages = 0;
  for (int r = 0; r < B; ++r) {
    const int len = cu[r + 1] - cu[r];
    if (len < 1) return SS_ERR_ARG;
    if (len > c->rt.max_prefill_tokens || len + cap > c->rt.max_ctx) return SS_ERR_CAPACITY;
    need_pages += ceil_div(len + cap, kPageTokens);
    if (eos_at && eos_at[r] < 1) return SS_ERR_ARG;
  }
  if (need_pages > c->free_pages.size()) return SS_ERR_KV_BUDGET;
  const int Ttot = cu[B];
  for (int i = 0; i < Ttot; ++i)
    if (tokens[i] < 0 || tokens[i] >= m.vocab) return SS_ERR_ARG;

  // host-side batch state
  std::vector<int32_t> bt((size_t)B * c->st.max_pages, -1);
  c->batch_pages.clear();
  c->prompt_len.assign(B, 0);
  c->row_pages.assign(B, {});
  c->batch_tokens.assign(tokens, tokens + Ttot);
  c->batch_cu.assign(cu, cu + B + 1);
  for (int r = 0; r < B; ++r) {
    const int len = cu[r + 1] - cu[r];
    c->prompt_len[r] = len;
    const int np = ceil_div(len + cap, kPageTokens);
    for (int p = 0; p < np; ++p) {
      const int32_t pg = c->free_pages.back();
      c->free_pages.pop_back();
      c->batch_pages.push_back(pg);
      c->row_pages[r].push_back(pg);
      bt[(size_t)r * c->st.max_pages + p] = pg;
    }
  }
  c->in_batch = true;
  c->B = B;
  c->cap = cap;
  std::vector<int32_t> rows((size_t)kMaxBatch * 8, 0);
  for (int r = 0; r < B; ++r) {
    rows[0 * kMaxBatch + r] = c->prompt_len[r];   // ctx_len after the prompt pass
    rows[3 * kMaxBatch + r] = 1;                  // active
    rows[5 * kMaxBatch + r] = eos_at ? eos_at[r] : 0;
    rows[6 * kMaxBatch + r] = r < (int)c->next_row_keys.size() ? c->next_row_keys[r] : r;
  }
  c->next_row_keys.clear();
  rows[7 * kMaxBatch + 0] = cap;
  rows[7 * kMaxBatch + 1] = B;
  int rc = SS_OK;
  auto bail = [&](int code) { ss_release_batch(c); return code; };
#define SS_CUDA_B(expr)                                              \
  do {                                                               \
    cudaError_t _e = (expr);                                         \
    if (_e != cudaSuccess) { c->last_cuda = (int)_e; return bail(SS_ERR_CUDA); } \
  } while (0)
  SS_CUDA_B(cudaMemcpyAsync(c->st.ctx_len, rows.data(), rows.size() * 4, cudaMemcpyHostToDevice, c->stream));
  SS_CUDA_B(cudaMemcpyAsync(c->st.block_table, bt.data(), bt.size() * 4, cudaMemcpyHostToDevice, c->stream));

  // chunks of whole sequences
  std::vector<int32_t> tok_row, tok_pos, cu_loc, last;
  int s0 = 0;
  while (s0 < B) {
    int s1 = s0, T = 0;
    while (s1 < B && T + (cu[s1 + 1] - cu[s1]) <= c->rt.max_prefill_tokens) { T += cu[s1 + 1] - cu[s1]; ++s1; }
    tok_row.resize(T); tok_pos.resize(T); cu_loc.assign(1, 0); last.clear();
    int t = 0;
    for (int s = s0; s < s1; ++s) {
      const int len = cu[s + 1] - cu[s];
      for (int p = 0; p < len; ++p, ++t) { tok_row[t] = s; tok_pos[t] = p; }
      cu_loc.push_back(t);
      last.push_back(t - 1);
    }
    SS_CUDA_B(cudaMemcpyAsync(c->d_tokens, tokens + cu[s0], (size_t)T * 4, cudaMemcpyHostToDevice, c->stream));
    SS_CUDA_B(cudaMemcpyAsync(c->d_tok_row, tok_row.data(), (size_t)T * 4, cudaMemcpyHostToDevice, c->stream));
    SS_CUDA_B(cudaMemcpyAsync(c->d_tok_pos, tok_pos.data(), (size_t)T * 4, cudaMemcpyHostToDevice, c->stream));
    SS_CUDA_B(cudaMemcpyAsync(c->d_cu, cu_loc.data(), cu_loc.size() * 4, cudaMemcpyHostToDevice, c->stream));
    SS_CUDA_B(cudaMemcpyAsync(c->d_last, last.data(), last.size() * 4, cudaMemcpyHostToDevice, c->stream));
    if ((rc = enqueue_prefill_chunk(c, s0, s1, cu, T))) return bail(rc);
    SS_CUDA_B(launch(c, gather_last_rmsnorm_kernel, dim3(s1 - s0), dim3(256), 0, (const float*)c->h,
                     (const int32_t*)c->d_last, c->h_dec + (size_t)s0 * m.d_model, (const bf16*)c->final_norm,
                     c->x_dec + (size_t)s0 * m.d_model,
                     (opts && opts->dump_hidden) ? opts->dump_hidden + (size_t)s0 * m.d_model : (float*)nullptr,
                     m.d_model, m.rms_eps));
    // the host vectors above are reused by the next chunk
    SS_CUDA_B(cudaStreamSynchronize(c->stream));
    s0 = s1;
  }
  // LM head on the last tokens, first generated token, bookkeeping
  const int NT = round_up(B, 16);
  const CUtensorMap* mx;
  if ((rc = xmap(c, 3, NT, &mx))) return bail(rc);
  const GemmPlan p_lm = plan_gemm(m.vocab, m.d_model, NT, 1, kGemmPartial, c->n_sm);
  if ((rc = run_gemm(c, c->lm_head, *mx, p_lm, kGemmPartial, B, nullptr, nullptr, 0))) return bail(rc);
  SS_CUDA_B(launch(c, lmhead_tile_argmax_kernel, dim3(c->n_tiles_lm), dim3(128), 0, (const float*)c->partial,
                   split_of(p_lm, c->tbl_lm_prompt), c->st, opts ? opts->dump_logits : (float*)nullptr, c->tile_val,
                   c->tile_idx, B, m.vocab, c->n_tiles_lm, m.eos_id, c->sample));
  SS_CUDA_B(launch(c, bookkeeping_kernel, dim3(1), dim3(1024), 0, c->st, (const float*)c->tile_val,
                   (const int32_t*)c->tile_idx, c->n_tiles_lm, opts ? opts->forced_tokens : (const int32_t*)nullptr,
                   first_tokens, opts ? opts->dump_choice : (int32_t*)nullptr, B, m.eos_id, 1));
#undef SS_CUDA_B
  return SS_OK;
}

int ss_keep_prompts(ss_ctx* c, const int32_t* ids, const int32_t* keep_len) {
  if (!c || !ids || !keep_len) return SS_ERR_ARG;
  if (!c->in_batch || c->batch_cu.empty()) return SS_ERR_STATE;      // no batch, or one that was itself resumed
  const int B = c->B;
  for (int r = 0; r < B; ++r) {
    if (keep_len[r] < 2 || keep_len[r] > c->prompt_len[r]) return SS_ERR_ARG;
    for (int q = 0; q < r; ++q)
      if (ids[q] == ids[r]) return SS_ERR_ARG;
  }
  for (int r = 0; r < B; ++r) {
    auto old = c->kept.find(ids[r]);
    if (old != c->kept.end()) {
      for (int32_t p : old->second.pages) c->free_pages.push_back(p);
      c->kept.erase(old);
    }
    const int n_keep = ceil_div(keep_len[r], kPageTokens);
    ss_ctx::KeptPrompt k;
    k.pages.assign(c->row_pages[r].begin(), c->row_pages[r].begin() + n_keep);
    k.len = keep_len[r];
    k.last_tok = c->batch_tokens[c->batch_cu[r] + keep_len[r] - 1];
    // these pages no longer go back to the pool with the batch
    for (int32_t p : k.pages) {
      auto it = std::find(c->batch_pages.begin(), c->batch_pages.end(), p);
      if (it != c->batch_pages.end()) { *it = c->batch_pages.back(); c->batch_pages.pop_back(); }
    }
    c->kept.emplace(ids[r], std::move(k));
  }
  return SS_OK;
}

int ss_drop_prompts(ss_ctx* c, const int32_t* ids, int32_t n) {
  if (!c || n < -1 || (n > 0 && !ids)) return SS_ERR_ARG;
  if (c->in_batch) return SS_ERR_STATE;
  if (n == -1) {
    for (auto& kv : c->kept)
      for (int32_t p : kv.second.pages) c->free_pages.push_back(p);
    c->kept.clear();
    return SS_OK;
  }
  for (int i = 0; i < n; ++i) {
    auto it = c->kept.find(ids[i]);
    if (it == c->kept.end()) continue;
    for (int32_t p : it->second.pages) c->free_pages.push_back(p);
    c->kept.erase(it);
  }
  return SS_OK;
}

int ss_resume(ss_ctx* c, const int32_t* ids, int32_t B, const int32_t* eos_at, int32_t cap, const ss_step_opts* opts,
              int32_t* first_tokens) {
  if (!c || !ids || B < 1 || cap < 1) return SS_ERR_ARG;
  if (c->n_loaded != c->n_expected || c->in_batch) return SS_ERR_STATE;
  if (B > c->rt.max_batch || cap > c->rt.max_new_tokens) return SS_ERR_CAPACITY;
  size_t need_pages = 0;
  for (int r = 0; r < B; ++r) {
    auto it = c->kept.find(ids[r]);
    if (it == c->kept.end()) return SS_ERR_STATE;
    for (int q = 0; q < r; ++q)
      if (ids[q] == ids[r]) return SS_ERR_ARG;
    const int len = it->second.len;
    if (len + cap > c->rt.max_ctx) return SS_ERR_CAPACITY;
    if (eos_at && eos_at[r] < 1) return SS_ERR_ARG;
    need_pages += (size_t)ceil_div(len + cap, kPageTokens) - it->second.pages.size();
  }
  if (need_pages > c->free_pages.size()) return SS_ERR_KV_BUDGET;
  std::vector<int32_t> bt((size_t)B * c->st.max_pages, -1);
  std::vector<int32_t> rows((size_t)kMaxBatch * 8, 0);
  c->batch_pages.clear();
  c->batch_tokens.clear();
  c->batch_cu.clear();
  c->prompt_len.assign(B, 0);
  c->row_pages.assign(B, {});
  for (int r = 0; r < B; ++r) {
    const ss_ctx::KeptPrompt& k = c->kept[ids[r]];
    c->prompt_len[r] = k.len;
    c->row_pages[r] = k.pages;
    const int np = ceil_div(k.len + cap, kPageTokens);
    for (int p = (int)k.pages.size(); p < np; ++p) {
      const int32_t pg = c->free_pages.back();
      c->free_pages.pop_back();
      c->batch_pages.push_back(pg);
      c->row_pages[r].push_back(pg);
    }
    for (int p = 0; p < np; ++p) bt[(size_t)r * c->st.max_pages + p] = c->row_pages[r][p];
    // the row stands one token before the end of its kept prompt: that token is fed again by the first step
    rows[0 * kMaxBatch + r] = k.len - 1;
    rows[1 * kMaxBatch + r] = k.last_tok;
    rows[3 * kMaxBatch + r] = 1;
    rows[5 * kMaxBatch + r] = eos_at ? eos_at[r] : 0;
    rows[6 * kMaxBatch + r] = r < (int)c->next_row_keys.size() ? c->next_row_keys[r] : r;
  }
  c->next_row_keys.clear();
  rows[7 * kMaxBatch + 0] = cap;
  rows[7 * kMaxBatch + 1] = B;
  c->in_batch = true;
  c->B = B;
  c->cap = cap;
  auto bail = [&](int code) { ss_release_batch(c); return code; };
  cudaError_t e = cudaMemcpyAsync(c->st.ctx_len, rows.data(), rows.size() * 4, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->st.block_table, bt.data(), bt.size() * 4, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);          // the host vectors go out of scope
  if (e != cudaSuccess) { c->last_cuda = (int)e; return bail(SS_ERR_CUDA); }
  int rc = enqueue_decode_step(c, opts, first_tokens);
  if (rc) return bail(rc);
  return SS_OK;
}

int ss_set_prompt_cache(ss_ctx* c, int32_t mode, const int32_t* keep_len, int32_t n) {
  if (!c || mode < 0 || mode > 2 || n < 0 || (mode == 1 && (!keep_len || n < 1))) return SS_ERR_ARG;
  c->prompt_cache_mode = mode;
  c->cache_keep_len.clear();
  if (mode == 1) c->cache_keep_len.assign(keep_len, keep_len + n);
  return SS_OK;
}

int ss_decode_step(ss_ctx* c, const ss_step_opts* opts, int32_t* next_tokens, int32_t* n_active_host) {
  if (!c) return SS_ERR_ARG;
  if (!c->in_batch) return SS_ERR_STATE;
  int rc = enqueue_decode_step(c, opts, next_tokens);
  if (rc) return rc;
  if (n_active_host)
    SS_CUDA(c, cudaMemcpyAsync(n_active_host, c->st.scalars + 1, 4, cudaMemcpyDeviceToHost, c->stream));
  return SS_OK;
}

int ss_decode_steps(ss_ctx* c, int32_t n_steps, int32_t* n_active_host) {
  if (!c || n_steps < 0) return SS_ERR_ARG;
  if (!c->in_batch) return SS_ERR_STATE;
  for (int s = 0; s < n_steps; ++s) {
    int rc = enqueue_decode_step(c, nullptr, nullptr);
    if (rc) return rc;
  }
  if (n_active_host)
    SS_CUDA(c, cudaMemcpyAsync(n_active_host, c->st.scalars + 1, 4, cudaMemcpyDeviceToHost, c->stream));
  return SS_OK;
}

int ss_read_batch(ss_ctx* c, int32_t* out_tokens, int32_t stride, int32_t* out_len, uint8_t* out_status) {
  if (!c || !out_len || !out_status || (out_tokens && stride < 1)) return SS_ERR_ARG;
  if (!c->in_batch) return SS_ERR_STATE;
  const int B = c->B;
  std::vector<int32_t> gen(B), fin(B);
  SS_CUDA(c, cudaMemcpyAsync(gen.data(), c->st.gen, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaMemcpyAsync(fin.data(), c->st.finished, (size_t)B * 4, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaMemcpyAsync(c->pinned + 1, c->status, 4, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaStreamSynchronize(c->stream));
  if (c->pinned[1] != 0) return report_device_status(c, (uint32_t)c->pinned[1]);
  for (int r = 0; r < B; ++r) {
    if (out_tokens && gen[r] > stride) return SS_ERR_CAPACITY;
    out_len[r] = gen[r];
    out_status[r] = fin[r] ? 1 : 0;
  }
  if (out_tokens) {
    for (int r = 0; r < B; ++r)
      if (gen[r] > 0)
        SS_CUDA(c, cudaMemcpyAsync(out_tokens + (size_t)r * stride, c->st.out_tokens + (size_t)r * c->st.max_new,
                                   (size_t)gen[r] * 4, cudaMemcpyDeviceToHost, c->stream));
    SS_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  return SS_OK;
}

int ss_step_model_bytes(const ss_ctx* c, const int32_t* ctx_len, const uint8_t* active, int32_t B, double* out) {
  if (!c || !ctx_len || !out || B < 0) return SS_ERR_ARG;
  double bytes = weight_bytes_per_step(c->m);
  const double kvt = kv_bytes_per_token(c->m);
  for (int r = 0; r < B; ++r)
    if (!active || active[r]) bytes += kvt * ((double)ctx_len[r] + 1.0) + (double)c->m.d_model * 2.0;
  *out = bytes;
  return SS_OK;
}

int ss_last_device_status(ss_ctx* c, uint32_t* out) {
  if (!c || !out) return SS_ERR_ARG;
  SS_CUDA(c, cudaMemcpyAsync(c->pinned + 1, c->status, 4, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaStreamSynchronize(c->stream));
  *out = (uint32_t)c->pinned[1];
  return SS_OK;
}

int ss_set_sampling(ss_ctx* c, float temperature, uint64_t seed) {
  if (!c || !(temperature >= 0.f) || !std::isfinite(temperature)) return SS_ERR_ARG;
  c->sample.inv_temp = temperature > 0.f ? 1.f / temperature : 0.f;
  c->sample.seed_lo = (uint32_t)(seed & 0xffffffffu);
  c->sample.seed_hi = (uint32_t)(seed >> 32);
  return SS_OK;
}

int ss_set_row_keys(ss_ctx* c, const int32_t* keys, int32_t n) {
  if (!c || n < 0 || n > kMaxBatch || (n > 0 && !keys)) return SS_ERR_ARG;
  c->next_row_keys.assign(keys, keys + n);
  return SS_OK;
}

int ss_set_wait_limit_ms(ss_ctx* c, int32_t ms) {
  if (!c || ms < 1 || ms > 60000) return SS_ERR_ARG;
  c->wait_limit = (long long)ms * c->clock_khz;
  return SS_OK;
}

int ss_selftest_wait_timeout(ss_ctx* c, int32_t limit_us) {
  if (!c || limit_us < 1 || limit_us > 1000000) return SS_ERR_ARG;
  if (c->in_batch) return SS_ERR_STATE;
  const long long limit = (long long)limit_us * c->clock_khz / 1000;
  unsigned long long base = c->grid_epochs * (unsigned long long)c->n_sm;
  unsigned long long* ctr = c->grid_ctr;
  uint32_t* status = c->status;
  void* args[4] = {(void*)&ctr, (void*)&base, (void*)&limit, (void*)&status};
  SS_CUDA(c, cudaLaunchCooperativeKernel((const void*)grid_wait_selftest_kernel, dim3(c->n_sm), dim3(32), args, 0, c->stream));
  c->launches++;
  SS_CUDA(c, cudaMemcpyAsync(c->pinned + 1, c->status, 4, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaStreamSynchronize(c->stream));
  if (c->pinned[1] != 0) return report_device_status(c, (uint32_t)c->pinned[1]);
  // the wait came through although an arrival was missing: the counter no longer matches the epochs
  cudaMemsetAsync(c->grid_ctr, 0, 8, c->stream);
  cudaStreamSynchronize(c->stream);
  c->grid_epochs = 0;
  return SS_OK;
}

int ss_set_trace(ss_ctx* c, int32_t on) {
  if (!c) return SS_ERR_ARG;
  c->trace_on = on != 0;
  return SS_OK;
}

int ss_step_trace(ss_ctx* c, uint64_t* out, int32_t cap, int32_t* n) {
  if (!c || !out || !n) return SS_ERR_ARG;
  if (!c->trace_on) return SS_ERR_STATE;
  *n = c->trace_len;
  if (cap < c->trace_len) return SS_ERR_CAPACITY;
  SS_CUDA(c, cudaMemcpyAsync(out, c->trace, (size_t)c->trace_len * 8, cudaMemcpyDeviceToHost, c->stream));
  SS_CUDA(c, cudaStreamSynchronize(c->stream));
  return SS_OK;
}

int ss_last_cuda_error(const ss_ctx* c) { return c ? c->last_cuda : 0; }
int64_t ss_kernel_launches(const ss_ctx* c) { return c ? c->launches : 0; }

}  // extern "C"

// Runs the micro-batches batches[0..n_batches) (rows: order[first_row .. first_row + n_rows)) one after the other:
// prompt pass, decode until every row has finished or the cap, read back.  Rows the cap cut (cap < max_new, no EOS)
// are appended to `fails`; the others get their final tokens, length and status.  Adds to `gs`, writes one log record
// per batch from log[*n_log] on.
static int run_batch_list(ss_ctx* c, const ss_sched_cfg* cfg, const int32_t* prompt_tokens, const int64_t* prompt_off,
                          const int32_t* eos_at, const int32_t* order, const ss_batch_desc* batches, int32_t n_batches,
                          int32_t* out_tokens, const int64_t* out_off, int32_t* out_len, uint8_t* out_status,
                          std::vector<int32_t>& fails, ss_batch_log* log, int32_t log_cap, int32_t* n_log,
                          ss_group_stats& gs) {
  cudaEvent_t ev[3] = {nullptr, nullptr, nullptr};       // batch start, prompt pass done, decode done
  auto cleanup = [&](int code) {
    for (auto& e : ev)
      if (e) cudaEventDestroy(e);
    if (c->in_batch) ss_release_batch(c);
    return code;
  };
  // every CUDA failure below leaves through cleanup(): events destroyed, pages of a batch in flight returned
#define SS_CUDA_G(expr)                                                          \
  do {                                                                           \
    cudaError_t _e = (expr);                                                     \
    if (_e != cudaSuccess) { c->last_cuda = (int)_e; return cleanup(SS_ERR_CUDA); } \
  } while (0)
  for (auto& e : ev) SS_CUDA_G(cudaEventCreate(&e));
  const double W = weight_bytes_per_step(c->m), kvt = kv_bytes_per_token(c->m);
  std::vector<int32_t> toks, cu, eos_b, len_b, tok_b;
  std::vector<uint8_t> st_b;
  int rc;
  for (int32_t bi = 0; bi < n_batches; ++bi) {
    const ss_batch_desc b = batches[bi];
    const int32_t* rows_src = order + b.first_row;
    const int B = b.n_rows;
    if (log && *n_log >= log_cap) return cleanup(SS_ERR_CAPACITY);
    toks.clear();
    cu.assign(1, 0);
    eos_b.clear();
    int max_target = 0;
    for (int r = 0; r < B; ++r) {
      const int q = rows_src[r];
      toks.insert(toks.end(), prompt_tokens + prompt_off[q], prompt_tokens + prompt_off[q + 1]);
      cu.push_back((int32_t)toks.size());
      if (eos_at) { eos_b.push_back(eos_at[q]); max_target = std::max(max_target, eos_at[q]); }
    }
    c->next_row_keys.assign(rows_src, rows_src + B);      // a row's sampling key is its query id, in every pass
    // prompt reuse (App. C): a batch whose queries all have kept prompts starts from them instead of a prompt pass
    bool resume = c->prompt_cache_mode == 2;
    for (int r = 0; r < B && resume; ++r) resume = c->kept.count(rows_src[r]) != 0;
    SS_CUDA_G(cudaEventRecord(ev[0], c->stream));
    if (resume) rc = ss_resume(c, rows_src, B, eos_at ? eos_b.data() : nullptr, b.cap, nullptr, nullptr);
    else rc = ss_prefill(c, toks.data(), cu.data(), B, eos_at ? eos_b.data() : nullptr, b.cap, nullptr, nullptr);
    if (rc) return cleanup(rc);
    if (c->prompt_cache_mode == 1 && !resume) {
      std::vector<int32_t> kl(B);
      for (int r = 0; r < B; ++r) {
        const int q = rows_src[r];
        if (q >= (int)c->cache_keep_len.size()) return cleanup(SS_ERR_ARG);
        kl[r] = c->cache_keep_len[q];
      }
      if ((rc = ss_keep_prompts(c, rows_src, kl.data()))) return cleanup(rc);
    }
    SS_CUDA_G(cudaEventRecord(ev[1], c->stream));
    if (eos_at) {
      // lengths are forced, so the number of steps is known: the longest target or the cap
      const int steps = std::min(b.cap, max_target);
      if ((rc = ss_decode_steps(c, steps - 1, nullptr))) return cleanup(rc);
    } else {
      int done = 1;
      while (done < b.cap) {
        const int chunk = std::min(8, b.cap - done);
        if ((rc = ss_decode_steps(c, chunk, c->pinned))) return cleanup(rc);
        SS_CUDA_G(cudaStreamSynchronize(c->stream));
        done += chunk;
        if (c->pinned[0] == 0) break;
      }
    }
    SS_CUDA_G(cudaEventRecord(ev[2], c->stream));
    len_b.assign(B, 0);
    st_b.assign(B, 0);
    tok_b.assign((size_t)B * cfg->max_new_tokens, 0);
    if ((rc = ss_read_batch(c, tok_b.data(), cfg->max_new_tokens, len_b.data(), st_b.data()))) return cleanup(rc);
    ss_release_batch(c);
    float pf = 0, dc = 0;
    cudaEventElapsedTime(&pf, ev[0], ev[1]);
    cudaEventElapsedTime(&dc, ev[1], ev[2]);
    int steps = 0, n_failed = 0;
    for (int r = 0; r < B; ++r) {
      const int q = rows_src[r];
      steps = std::max(steps, len_b[r]);
      const bool failed = !st_b[r] && b.cap < cfg->max_new_tokens;
      if (failed) {
        fails.push_back(q);
        ++n_failed;
      } else {
        out_len[q] = len_b[r];
        out_status[q] = st_b[r];
        std::copy(tok_b.begin() + (size_t)r * cfg->max_new_tokens,
                  tok_b.begin() + (size_t)r * cfg->max_new_tokens + len_b[r], out_tokens + out_off[q]);
        gs.useful_tokens += len_b[r];
      }
      const double nr = std::max(0, len_b[r] - 1);     // decode steps the row took part in
      gs.model_bytes += kvt * (nr * (cu[r + 1] - cu[r]) + nr * (nr + 1) / 2.0);
    }
    gs.model_bytes += W * std::max(0, steps - 1);
    if (log) log[*n_log] = {b.first_row, B, b.cap, b.is_recompute, steps, n_failed, pf, dc};
    ++*n_log;
    gs.n_batches += 1;
    gs.steps += steps;
    gs.row_steps += (int64_t)B * steps;
    gs.prefill_ms += pf;
    gs.decode_ms += dc;
    gs.n_failed += n_failed;
  }
#undef SS_CUDA_G
  return cleanup(SS_OK);
}

extern "C" {

int ss_run_batches(ss_ctx* c, const ss_sched_cfg* cfg, const int32_t* prompt_tokens, const int64_t* prompt_off,
                   const int32_t* eos_at, int32_t n, const int32_t* order, int32_t n_order, const ss_batch_desc* batches,
                   int32_t n_batches, int32_t* out_tokens, const int64_t* out_off, int32_t* out_len, uint8_t* out_status,
                   int32_t* fail_rows, int32_t* n_fail, ss_batch_log* log, int32_t log_cap, int32_t* n_log,
                   ss_group_stats* stats) {
  if (!c || !cfg || n < 0 || n_batches < 0 || n_order < 0 || !n_log || !n_fail) return SS_ERR_ARG;
  if (n_batches > 0 && (!prompt_tokens || !prompt_off || !order || !batches || !out_tokens || !out_off || !out_len ||
                        !out_status || !fail_rows))
    return SS_ERR_ARG;
  int rc = validate_sched_cfg(cfg);
  if (rc) return rc;
  if (c->in_batch) return SS_ERR_STATE;
  if (cfg->max_new_tokens > c->rt.max_new_tokens) return SS_ERR_CAPACITY;
  for (int32_t i = 0; i < n_batches; ++i) {
    const ss_batch_desc& b = batches[i];
    if (b.n_rows < 1 || b.first_row < 0 || (int64_t)b.first_row + b.n_rows > n_order || b.cap < 1 ||
        b.cap > cfg->max_new_tokens)
      return SS_ERR_ARG;
    for (int r = 0; r < b.n_rows; ++r) {
      const int32_t q = order[b.first_row + r];
      if (q < 0 || q >= n) return SS_ERR_ARG;
      if (out_off[q + 1] - out_off[q] < cfg->max_new_tokens) return SS_ERR_CAPACITY;
    }
  }
  cudaEvent_t g0 = nullptr, g1 = nullptr;
  if (cudaEventCreate(&g0) != cudaSuccess || cudaEventCreate(&g1) != cudaSuccess) {
    if (g0) cudaEventDestroy(g0);
    return SS_ERR_CUDA;
  }
  ss_group_stats gs{};
  const int64_t launches0 = c->launches;
  std::vector<int32_t> fails;
  *n_log = 0;
  cudaEventRecord(g0, c->stream);
  rc = run_batch_list(c, cfg, prompt_tokens, prompt_off, eos_at, order, batches, n_batches, out_tokens, out_off,
                      out_len, out_status, fails, log, log_cap, n_log, gs);
  if (rc == SS_OK) {
    cudaEventRecord(g1, c->stream);
    if (cudaEventSynchronize(g1) != cudaSuccess) rc = SS_ERR_CUDA;
    else cudaEventElapsedTime(&gs.total_ms, g0, g1);
  }
  cudaEventDestroy(g0);
  cudaEventDestroy(g1);
  if (rc) return rc;
  std::copy(fails.begin(), fails.end(), fail_rows);
  *n_fail = (int32_t)fails.size();
  gs.kernel_launches = c->launches - launches0;
  if (stats) *stats = gs;
  return SS_OK;
}

int ss_run_group(ss_ctx* c, const ss_sched_cfg* cfg, const int32_t* prompt_tokens, const int64_t* prompt_off,
                 const int32_t* pred_len, const int32_t* perm, const int32_t* eos_at, int32_t n, int32_t* out_tokens,
                 const int64_t* out_off, int32_t* out_len, uint8_t* out_status, int32_t* order, ss_batch_log* log,
                 int32_t log_cap, int32_t* n_log, ss_group_stats* stats) {
  if (!c || !cfg || n < 0 || !n_log) return SS_ERR_ARG;
  if (n > 0 && (!prompt_tokens || !prompt_off || !pred_len || !out_tokens || !out_off || !out_len || !out_status || !order))
    return SS_ERR_ARG;
  int rc = validate_sched_cfg(cfg);
  if (rc) return rc;
  if (c->in_batch) return SS_ERR_STATE;
  if (cfg->max_new_tokens > c->rt.max_new_tokens) return SS_ERR_CAPACITY;
  for (int i = 0; i < n; ++i)
    if (out_off[i + 1] - out_off[i] < cfg->max_new_tokens) return SS_ERR_CAPACITY;

  std::vector<int32_t> plen(n);
  for (int i = 0; i < n; ++i) plen[i] = (int32_t)(prompt_off[i + 1] - prompt_off[i]);
  std::vector<int32_t> ord;
  std::vector<ss_batch_desc> plan;
  if ((rc = plan_first_pass(*cfg, plen.data(), pred_len, perm, n, ord, plan))) return rc;

  cudaEvent_t g0 = nullptr, g1 = nullptr;
  if (cudaEventCreate(&g0) != cudaSuccess || cudaEventCreate(&g1) != cudaSuccess) {
    if (g0) cudaEventDestroy(g0);
    return SS_ERR_CUDA;
  }
  auto done = [&](int code) { cudaEventDestroy(g0); cudaEventDestroy(g1); return code; };
  ss_group_stats gs{};
  const int64_t launches0 = c->launches;
  std::vector<int32_t> fails;
  *n_log = 0;
  cudaEventRecord(g0, c->stream);
  // first pass
  rc = run_batch_list(c, cfg, prompt_tokens, prompt_off, eos_at, ord.data(), plan.data(), (int32_t)plan.size(),
                      out_tokens, out_off, out_len, out_status, fails, log, log_cap, n_log, gs);
  if (rc) return done(rc);
  // the rows the caps cut, in collection order, regenerated from their prompts in batches of B0 with cap = max_new
  // (Sec. 4.1, failure collection and recomputation); they are listed behind the first-pass order
  const size_t n_fail = fails.size();
  ord.insert(ord.end(), fails.begin(), fails.end());
  std::vector<ss_batch_desc> again;
  for (size_t i = 0; i < n_fail; i += (size_t)cfg->base_batch)
    again.push_back({(int32_t)(n + i), (int32_t)std::min<size_t>(cfg->base_batch, n_fail - i), cfg->max_new_tokens, 1});
  std::vector<int32_t> fails2;
  rc = run_batch_list(c, cfg, prompt_tokens, prompt_off, eos_at, ord.data(), again.data(), (int32_t)again.size(),
                      out_tokens, out_off, out_len, out_status, fails2, log, log_cap, n_log, gs);
  if (rc) return done(rc);
  gs.n_failed = (int32_t)n_fail;
  for (int i = 0; i < n; ++i) order[i] = ord[i];
  for (size_t i = 0; i < n_fail; ++i) order[n + i] = fails[i];
  for (size_t i = n_fail; i < (size_t)n; ++i) order[n + i] = -1;
  cudaEventRecord(g1, c->stream);
  if (cudaEventSynchronize(g1) != cudaSuccess) return done(SS_ERR_CUDA);
  cudaEventElapsedTime(&gs.total_ms, g0, g1);
  gs.kernel_launches = c->launches - launches0;
  if (stats) *stats = gs;
  return done(SS_OK);
}

}  // extern "C"
