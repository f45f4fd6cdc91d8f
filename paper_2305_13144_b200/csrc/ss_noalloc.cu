// ss_logits_noalloc(): the LM-head projection for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- inside a region that is being
// captured into a CUDA graph by the caller's framework, inside a memory-pool callback, in a
// process whose device memory is fully handed out to another allocator, or in a real-time loop
// where an allocation (and the implicit synchronisation it can bring) is not acceptable.  Such a
// caller owns its inputs and outputs but has nowhere to put the two temporaries the projection
// needs (the normalised bf16 activations and the fp32 split-K partial sums).  Here they live in
// one file-scope __device__ array of fixed size that every GPU which loads this library carries
// until the process exits.
//
// Same arithmetic as the LM head inside ss_prefill()/ss_decode_step(): x = RMSNorm(h) * g in bf16,
// the tcgen05 weight-streaming GEMM with fp32 partials, partials added in CTA order.
#include <mutex>

#include "ss_gemm.cuh"

using namespace ss;

namespace {

constexpr size_t kScratchBytes = 8u << 20;            // 8 MiB, all of it
constexpr int kNoAllocMaxRows = 16;                    // tokens per call
constexpr int kNoAllocMaxD = 8192;
constexpr size_t kXBytes = (size_t)kNoAllocMaxRows * kNoAllocMaxD * 2;   // bf16 activations, 256 KiB
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;     // device address of g_noalloc_scratch on this device
  int n_sm = 0;
};
std::mutex g_mu;
DeviceSetup g_dev[kMaxDevices];
EncodeTiledFn g_encode = nullptr;

// x[r] = RMSNorm(h[r]) * g as bf16; rows r >= n_rows of the 16-row operand are zeroed.
__global__ void __launch_bounds__(256)
noalloc_rmsnorm_kernel(const float* __restrict__ h, const __nv_bfloat16* __restrict__ g, __nv_bfloat16* __restrict__ x,
                       int n_rows, int d, float eps) {
  __shared__ float red[8];
  const int r = blockIdx.x;
  if (r >= n_rows) {
    for (int i = threadIdx.x; i < d; i += blockDim.x) x[(size_t)r * d + i] = __float2bfloat16_rn(0.f);
    return;
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = h[(size_t)r * d + i];
    ss += v * v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) tot += red[w];
  const float inv = rsqrtf(tot / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    x[(size_t)r * d + i] = __float2bfloat16_rn(h[(size_t)r * d + i] * inv * __bfloat162float(g[i]));
}

// logits[r][v] = sum of the partials of output row v for token r, in CTA order.  If a bounded wait of the
// projection gave up (status word non-zero) the partials are not all there: the whole output becomes NaN,
// which is how this call, having already returned, reports the failure.
__global__ void __launch_bounds__(256)
noalloc_reduce_kernel(const float* __restrict__ partial, SplitInfo sp, float* __restrict__ logits, int V,
                      const uint32_t* __restrict__ status) {
  const int r = blockIdx.y, v = blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= V) return;
  const bool failed = *status != 0u;
  logits[(size_t)r * V + v] = failed ? __int_as_float(0x7fc00000) : sum_partials_derived(partial, sp, v, r);
}

int setup_device(int dev, DeviceSetup** out) {
  if (dev < 0 || dev >= kMaxDevices) return SS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceSetup& s = g_dev[dev];
  if (!s.ready) {
    // The array's name is only a host-side handle; the kernels need its address on THIS device.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return SS_ERR_CUDA;
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return SS_ERR_CUDA;
    if (cudaFuncSetAttribute(gemm_wx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return SS_ERR_CUDA;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qr;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn)
        return SS_ERR_CUDA;
      g_encode = (EncodeTiledFn)fn;
    }
    s.scratch = (unsigned char*)p;
    s.n_sm = n;
    s.ready = true;
  }
  *out = &s;
  return SS_OK;
}

int encode_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)kTileK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? SS_OK : SS_ERR_CUDA;
}

}  // namespace

extern "C" int ss_logits_noalloc(const float* hidden, const void* norm_gain, const void* lm_head, int32_t n_rows,
                                 int32_t d_model, int32_t vocab, float rms_eps, float* logits, void* stream) {
  if (!hidden || !norm_gain || !lm_head || !logits) return SS_ERR_ARG;
  if (n_rows < 1 || d_model < 64 || vocab < 1) return SS_ERR_ARG;
  if (((uintptr_t)lm_head & 15) || (d_model % 64)) return SS_ERR_UNSUPPORTED;
  if (n_rows > kNoAllocMaxRows || d_model > kNoAllocMaxD) return SS_ERR_CAPACITY;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SS_ERR_CUDA;
  (void)cudaGetLastError();   // an error left behind by the caller's earlier work is not this call's
  DeviceSetup* s = nullptr;
  int rc = setup_device(dev, &s);
  if (rc) return rc;

  // split of the (tile, k-block) space over the SMs, as in the engine's decode step
  GemmPlan p{};
  p.n_out = vocab;
  p.K = d_model;
  p.n_tiles = (vocab + kTileM - 1) / kTileM;
  p.kb = d_model / kTileK;
  p.NT = kNoAllocMaxRows;
  const long long total = (long long)p.n_tiles * p.kb;
  p.gridx = (int)(total < s->n_sm ? total : s->n_sm);
  p.gridy = 1;
  const int ipc = (int)((total + p.gridx - 1) / p.gridx);
  p.max_seg = (ipc + p.kb - 2) / p.kb + 1;
  const int stage_bytes = kTileM * kTileK * 2 + p.NT * kTileK * 2;
  p.stages = (227 * 1024 - 2048) / stage_bytes;
  if (p.stages > kGemmMaxStages) p.stages = kGemmMaxStages;
  p.smem_bytes = 2048 + p.stages * stage_bytes;
  p.tmem_cols = 32;
  const size_t partial_bytes = (size_t)p.gridx * p.max_seg * p.NT * 128 * sizeof(float);
  if (kXBytes + 256 + partial_bytes > kScratchBytes) return SS_ERR_CAPACITY;   // vocabulary too large for the array

  __nv_bfloat16* x = reinterpret_cast<__nv_bfloat16*>(s->scratch);
  uint32_t* status = reinterpret_cast<uint32_t*>(s->scratch + kXBytes);
  float* partial = reinterpret_cast<float*>(s->scratch + kXBytes + 256);
  cudaStream_t st = (cudaStream_t)stream;

  CUtensorMap mw, mx;
  if (encode_map(&mw, lm_head, vocab, d_model, kTileM) || encode_map(&mx, x, kNoAllocMaxRows, d_model, p.NT))
    return SS_ERR_CUDA;
  // the status word must start at zero; x and the partials are rewritten below
  if (cudaMemsetAsync(status, 0, 256, st) != cudaSuccess) return SS_ERR_CUDA;
  noalloc_rmsnorm_kernel<<<kNoAllocMaxRows, 256, 0, st>>>(hidden, (const __nv_bfloat16*)norm_gain, x, n_rows, d_model,
                                                          rms_eps);
  GemmArgs a{};
  a.p = p;
  a.mode = kGemmPartial;
  a.n_tok = n_rows;
  a.partial = partial;
  a.status = status;
  gemm_wx_kernel<<<dim3(1, p.gridx), kGemmThreads, p.smem_bytes, st>>>(mw, mx, a);
  SplitInfo sp;
  sp.gridx = p.gridx; sp.kb = p.kb; sp.max_seg = p.max_seg; sp.NT = p.NT; sp.total = total; sp.tiles = nullptr;
  noalloc_reduce_kernel<<<dim3((vocab + 255) / 256, n_rows), 256, 0, st>>>(partial, sp, logits, vocab, status);
  return cudaGetLastError() == cudaSuccess ? SS_OK : SS_ERR_CUDA;
}
