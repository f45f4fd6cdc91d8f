// Internal declarations shared by the host runtime and the kernel launchers.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "seqsched.h"

namespace ss {

// ---- scheduler (ss_sched.cpp) ------------------------------------------------------------
int validate_sched_cfg(const ss_sched_cfg* c);
int32_t length_bin(int32_t x, const ss_sched_cfg& c);
int32_t batch_allowance(int32_t L, const ss_sched_cfg& c);
int plan_first_pass(const ss_sched_cfg& c, const int32_t* prompt_len, const int32_t* pred_len,
                    const int32_t* perm, int32_t n, std::vector<int32_t>& order,
                    std::vector<ss_batch_desc>& out);

// ---- constants ---------------------------------------------------------------------------
constexpr int kPageTokens = 32;        // tokens per key/value page
constexpr int kTileM = 128;            // weight rows per GEMM tile (tcgen05 M)
constexpr int kTileK = 64;             // bf16 elements per 128-byte swizzled row
constexpr int kTileN = 256;            // weight rows per block of the tiled layout (tcgen05 N of the decode step)
constexpr int kBlockBytes = kTileN * kTileK * 2;   // one (256-row tile, k-block) block: 32 KiB
constexpr int kMaxBatch = 256;

// Device status codes (which bounded wait expired / which check failed).
enum : uint32_t {
  kStatusOk = 0,
  kStatusProducerTimeout = 1,
  kStatusMmaTimeout = 2,
  kStatusEpilogueTimeout = 3,
  kStatusBadPage = 4,
};

// ---- GEMM:  D[n_out, tok] = W[n_out, K] . X[tok, K]^T  -------------------------------------
// The tile-iteration space (n_tiles x kb) is cut into `gridx` equal contiguous ranges, one per
// CTA (split along K where a range ends inside a tile).  In kGemmPartial mode every (CTA,
// tile) segment is written as an fp32 partial; the consumer kernel adds the segments of a tile
// in CTA order, so the result does not depend on timing.
enum GemmMode : int { kGemmPartial = 0, kGemmDirectBf16 = 1, kGemmDirectF32Add = 2, kGemmDirectF32 = 3 };

struct GemmPlan {
  int n_out, K, n_tiles, kb;
  int NT;              // token tile (tcgen05 N), multiple of 16, <= 256
  int gridx, gridy;    // CTAs along the iteration space / token tiles
  int max_seg;         // partial slots per CTA
  int stages;
  int smem_bytes;
  int tmem_cols;
};

struct GemmArgs {
  GemmPlan p;
  const void* w_tiled; // weights repacked as contiguous 32 KiB (256-row tile, k-block) images, or null (row-major via TMA)
  int mode;
  int n_tok;           // valid tokens
  float* partial;      // [gridx*max_seg][NT][128]
  void* out_bf16;      // [tok][ld_out]
  float* out_f32;
  int ld_out;
  uint32_t* status;
};

// Where the partial sums of one 128-row tile live: the first segment in slot `slot0`, the others
// in segment 0 of CTAs c_next..c_last (a CTA that starts inside a tile has it as its first tile).
struct TileSeg {
  int32_t slot0, c_next, c_last, pad;
};

// Partial-slot bookkeeping shared by the GEMM and its consumers.
struct SplitInfo {
  int gridx, kb, max_seg, NT;
  long long total;          // n_tiles * kb
  const TileSeg* tiles;     // device table [n_tiles], or null (then the consumers derive it)
};

}  // namespace ss
