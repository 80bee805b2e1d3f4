// Internal declarations shared by the library's translation units (not part of the C boundary).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <atomic>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/vit.h"

namespace vit {

typedef __nv_bfloat16 bf16;

// Epilogue selector of the linear kernels.
enum Epilogue : int {
  EPI_BIAS = 0,          // out = acc + bias
  EPI_BIAS_GELU = 1,     // out = gelu(acc + bias), erf form
  EPI_BIAS_RESIDUAL = 2, // out = acc + bias + residual[row, col]
  EPI_BIAS_POS = 3,      // patch embed: row r of the GEMM is patch r % n_patches of image r / n_patches;
                         // out[image*T + t0 + patch, col] = acc + bias + pos[t0 + patch, col], T = t0 + n_patches
  // LayerNorm of the input rows folded into the product (bf16 tensor-core kernel only): with the
  // gain folded into the weight, wg[n,k] = g[k] w[n,k], the kernel multiplies the raw rows and applies
  //   out[m,n] = rstd[m] (acc[m,n] - mean[m] c1[n]) + c0[n],  c1[n] = sum_k wg[n,k],  c0[n] = sum_k b[k] w[n,k] + bias[n]
  // which equals LN(a)[m,:] . w[n,:] + bias[n] without a normalised copy of a ever being written.
  EPI_LN_BIAS = 4,
  EPI_LN_BIAS_GELU = 5
};

struct LinearArgs {
  int M, N, K;            // out[M,N] = a[M,K] . w[N,K]^T
  const void* a;          // activation type, row stride lda elements
  int lda;
  const void* w;          // activation type, row stride K... (ldw elements)
  int ldw;
  const float* bias;      // [N]
  int epilogue;
  const void* residual;   // EPI_BIAS_RESIDUAL: [M, N] stride ldo; may alias out
  const float* pos;       // EPI_BIAS_POS: [T, N] fp32
  const float2* ln_stats; // EPI_LN_*: [M] (mean, 1/sqrt(var + eps)) of the rows of a
  const float* ln_c1;     // EPI_LN_*: [N] row sums of the gain-folded weight; bias holds c0
  int n_patches;          // EPI_BIAS_POS
  int first_patch_token;  // EPI_BIAS_POS: t0, the number of special tokens before the patches
  void* out;              // activation type, row stride ldo
  int ldo;
  int tiling;             // bf16 tensor-core kernel: TILING_AUTO (shape-only cost model) or a forced tiling
};

// Tilings of the tensor-core linear kernel (LinearArgs::tiling).
enum Tiling : int { TILING_AUTO = 0, TILING_128x128 = 1, TILING_128x256 = 2, TILING_PAIR_256x256 = 3 };

struct LayerWeights {
  const float *ln1_g, *ln1_b, *bqkv, *bo, *ln2_g, *ln2_b, *b1, *b2;
  const void *Wqkv, *Wo, *W1, *W2;   // activation type, [out, in]; bf16 mode: Wqkv and W1 carry the LayerNorm gain
  const float *qkv_c1, *qkv_c0, *fc1_c1, *fc1_c0;   // bf16 mode: the folded LayerNorm's column vectors (see EPI_LN_BIAS)
};

// Tensor maps are pure functions of (base address, extents, row pitch, box, swizzle).  The same
// few maps recur on every call (weights always; activations as long as the caller reuses its
// buffers), so a handle remembers them instead of asking the driver four to ten times per launch.
struct TensorMapKey {
  const void* base;
  uint64_t rows, cols, ld;
  uint32_t box_rows, box_cols, swizzle;
  bool operator==(const TensorMapKey& o) const {
    return base == o.base && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows &&
           box_cols == o.box_cols && swizzle == o.swizzle;
  }
};
struct TensorMapKeyHash {
  size_t operator()(const TensorMapKey& k) const {
    uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
    for (uint64_t v : {k.rows, k.cols, k.ld, (uint64_t)k.box_rows, (uint64_t)k.box_cols, (uint64_t)k.swizzle})
      h = (h ^ v) * 0x9E3779B97F4A7C15ull + (h >> 29);
    return (size_t)h;
  }
};
struct TensorMapCache {
  std::mutex mu;
  std::unordered_map<TensorMapKey, CUtensorMap, TensorMapKeyHash> maps;
  // Returns the cached map or encodes it with `encode(CUtensorMap*) -> bool`.  cache == nullptr: always encode.
  template <typename Encode>
  static bool get(TensorMapCache* cache, const TensorMapKey& key, CUtensorMap* out, Encode encode) {
    if (!cache) return encode(out);
    std::lock_guard<std::mutex> lock(cache->mu);
    auto it = cache->maps.find(key);
    if (it != cache->maps.end()) { *out = it->second; return true; }
    if (!encode(out)) return false;
    if (cache->maps.size() >= 4096) cache->maps.clear();     // callers that never reuse buffers
    cache->maps.emplace(key, *out);
    return true;
  }
};

struct ProfRecord { cudaEvent_t begin, end; int cls; };

struct Handle {
  vit_config cfg;
  int device;                        // the CUDA device the handle was created on
  int T, n_patches, d, patch_k, patch_k_pad;
  size_t act_bytes;                  // bytes of one activation element
  void* dev_blob;                    // every parameter, one allocation
  size_t dev_blob_bytes;
  const void* patch_W;               // [H, patch_k_pad]
  const float *patch_b, *cls, *dist, *pos;          // dist: distillation token (nullptr without one)
  LayerWeights* layers;              // host array [L]
  const float *lnf_g, *lnf_b, *head_b, *head_dist_b;
  const void *head_W, *head_dist_W;  // [classes, H]; head_dist_*: second classifier (nullptr without a distillation token)
  int* dev_status;                   // device: [0] status word (0 = ok), [1] snapshot slot of vit_check_status
  std::mutex status_mutex;
  std::atomic<uint64_t> launches;
  bool profiling;                    // event pair around every launch (single-threaded use)
  std::vector<ProfRecord> prof;
  TensorMapCache tmaps;
};

// ---- kernel launchers (each returns a cudaError_t from the launch) ------------------------
// bf16 family
cudaError_t launch_layernorm_bf16(const bf16* x, const float* g, const float* b, float eps,
                                  bf16* y, int rows, int cols, cudaStream_t s);
cudaError_t launch_linear_tc(const LinearArgs& a, int* dev_status, cudaStream_t s, TensorMapCache* cache = nullptr);   // tcgen05 GEMM
// per-row LayerNorm statistics: stats[r] = (mean, 1 / sqrt(biased variance + eps)) of x[r, :]
cudaError_t launch_rowstats_bf16(const bf16* x, float eps, float2* stats, int rows, int cols, cudaStream_t s);
// attention: the tcgen05 kernel where it supports the shape, else the warp-level mma kernel
cudaError_t launch_attention_bf16(const bf16* qkv, bf16* out, int images, int T, int heads, int d,
                                  int* dev_status, cudaStream_t s, TensorMapCache* cache = nullptr);
bool attention_tc_supported(int T, int d);
cudaError_t launch_attention_tc(const bf16* qkv, bf16* out, int images, int T, int heads, int d,
                                int* dev_status, cudaStream_t s, TensorMapCache* cache = nullptr);
// fp32 family (SIMT)
cudaError_t launch_layernorm_f32(const float* x, const float* g, const float* b, float eps,
                                 float* y, int rows, int cols, cudaStream_t s);
cudaError_t launch_linear_f32(const LinearArgs& a, cudaStream_t s);
cudaError_t launch_attention_f32(const float* qkv, float* out, int images, int T, int heads, int d,
                                 cudaStream_t s);
// book-ends, both families (act_bf16 selects the element type)
cudaError_t launch_im2col(const float* pixels, void* cols, int images, int C, int S, int P,
                          int k_pad, bool act_bf16, cudaStream_t s);
// special tokens: token 0 = cls + pos[0]; token 1 = dist + pos[1] when dist != nullptr
cudaError_t launch_cls_rows(const float* cls, const float* dist, const float* pos, void* tokens, int images,
                            int T, int H, bool act_bf16, cudaStream_t s);
// W2 / bias2 != nullptr: second classifier on token 1, logits = mean of the two (feat_scratch then
// holds two feature rows per image)
cudaError_t launch_head(const void* tokens, const float* g, const float* b, float eps,
                        const void* W, const float* bias, const void* W2, const float* bias2,
                        float* feat_scratch, float* logits,
                        int images, int T, int H, int classes, bool act_bf16, cudaStream_t s);

// head with the feature scratch in a fixed device array of VIT_HEAD_STATIC_MAX_FLOATS floats
cudaError_t launch_head_static(const void* tokens, const float* g, const float* b, float eps,
                               const void* W, const float* bias, const void* W2, const float* bias2,
                               float* logits, int images, int T,
                               int H, int classes, bool act_bf16, cudaStream_t s);

cudaError_t launch_wait_probe(long long limit_cycles, int* dev_status, cudaStream_t s);
// *snapshot = atomic exchange of *status with 0, on stream s
cudaError_t launch_status_take(int* status, int* snapshot, cudaStream_t s);

bool tc_gemm_init();   // resolves the driver's tensor-map encoder; false if unavailable

// Function attributes (the opt-in to more than 48 KB of dynamic shared memory) and the SM count
// belong to a device, not to the process: each kernel instantiation keeps one bit per device.
struct PerDeviceFlag {
  std::atomic<uint64_t> mask{0};
};
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(PerDeviceFlag& done, Kernel kernel, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && (done.mask.load(std::memory_order_acquire) >> dev & 1)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && tracked) done.mask.fetch_or((uint64_t)1 << dev, std::memory_order_release);
  return e;
}
int current_device_sm_count();   // SMs of the current device (cached per device); 0 on error

}  // namespace vit
