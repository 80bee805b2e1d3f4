// LayerNorm, the fp32 (SIMT) kernel family, and the two book-ends' small kernels.
#include "vit_internal.h"

#include <mutex>

namespace vit {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float gelu_erf(float v) {
  return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
}

// ------------------------------------------------------------------------------------------
// LayerNorm, bf16 in / bf16 out.  One warp per row, the row lives in registers (NCH 16-byte
// chunks per lane), statistics in fp32 with a two-pass variance, warp-shuffle reductions.
// HBM-bound: reads and writes each element once.
// ------------------------------------------------------------------------------------------
template <int NCH>
__global__ void __launch_bounds__(256)
layernorm_bf16_kernel(const bf16* __restrict__ x, const float* __restrict__ g,
                      const float* __restrict__ b, float eps, bf16* __restrict__ y, int rows,
                      int cols) {
  const int row = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
  const int lane = threadIdx.x & 31;
  // launched with programmatic stream serialization: wait for the producer of x, then let the
  // consumer of y start its own set-up
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (row >= rows) return;
  const int nvec = cols >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * cols);
  uint4 u[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) {            // all loads in flight before the first use
    const int idx = lane + 32 * i;
    u[i] = idx < nvec ? __ldg(xr + idx) : make_uint4(0, 0, 0, 0);
  }
  // bf16 -> fp32 is a shift (low half) or a mask (high half) of the 32-bit word
  float v[NCH][8];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[i][2 * e] = __uint_as_float(w[e] << 16);
      v[i][2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
      sum += v[i][2 * e] + v[i][2 * e + 1];          // padded chunks are zero
    }
  }
  const float mean = warp_sum(sum) / (float)cols;
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const bool in = lane + 32 * i < nvec;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      v[i][e] = in ? v[i][e] - mean : 0.f;
      sq = fmaf(v[i][e], v[i][e], sq);
    }
  }
  const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)cols + eps);
  uint4* yr = reinterpret_cast<uint4*>(y + (size_t)row * cols);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      const float4 g0 = __ldg(reinterpret_cast<const float4*>(g) + 2 * idx);
      const float4 g1 = __ldg(reinterpret_cast<const float4*>(g) + 2 * idx + 1);
      const float4 b0 = __ldg(reinterpret_cast<const float4*>(b) + 2 * idx);
      const float4 b1 = __ldg(reinterpret_cast<const float4*>(b) + 2 * idx + 1);
      const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
      const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
      uint4 o;
      __nv_bfloat162* ho = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
      for (int e = 0; e < 4; ++e)
        ho[e] = __floats2bfloat162_rn(v[i][2 * e] * rstd * gg[2 * e] + bb[2 * e],
                                      v[i][2 * e + 1] * rstd * gg[2 * e + 1] + bb[2 * e + 1]);
      yr[idx] = o;
    }
  }
}

cudaError_t launch_layernorm_bf16(const bf16* x, const float* g, const float* b, float eps,
                                  bf16* y, int rows, int cols, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  if (cols % 8 != 0 || cols > 8 * 256) return cudaErrorInvalidValue;
  const int nch = (cols / 8 + 31) / 32;
  const int threads = 256;
  const unsigned blocks = (unsigned)(((size_t)rows * 32 + threads - 1) / threads);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(threads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t err = cudaSuccess;
#define LN_CASE(N) \
  case N: err = cudaLaunchKernelEx(&cfg, layernorm_bf16_kernel<N>, x, g, b, eps, y, rows, cols); break;
  switch (nch) {
    LN_CASE(1) LN_CASE(2) LN_CASE(3) LN_CASE(4) LN_CASE(5) LN_CASE(6) LN_CASE(7) LN_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef LN_CASE
  return err;
}

// ------------------------------------------------------------------------------------------
// LayerNorm statistics only: stats[row] = (mean, 1 / sqrt(biased variance + eps)).  Same warp-
// per-row scheme as the kernel above (128-bit loads, the row in registers, two-pass variance,
// shuffle reductions); the normalisation itself is applied by the consumer (the QKV and fc1
// GEMMs fold it into their epilogue), so nothing but 8 bytes per row is written.
// ------------------------------------------------------------------------------------------
template <int NCH>
__global__ void __launch_bounds__(256)
rowstats_bf16_kernel(const bf16* __restrict__ x, float eps, float2* __restrict__ stats, int rows, int cols) {
  const int row = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
  const int lane = threadIdx.x & 31;
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (row >= rows) return;
  const int nvec = cols >> 3;
  const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)row * cols);
  uint4 u[NCH];
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int idx = lane + 32 * i;
    u[i] = idx < nvec ? __ldg(xr + idx) : make_uint4(0, 0, 0, 0);
  }
  // unpacked pairs (low half by shift, high half by mask); sums on packed two-wide fp32 instructions
  float2 v[NCH][4];
  float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const uint32_t w[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[i][e] = make_float2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xffff0000u));
      sum2 = __fadd2_rn(sum2, v[i][e]);          // padded chunks are zero
    }
  }
  const float mean = warp_sum(sum2.x + sum2.y) / (float)cols;
  const float2 nmean = make_float2(-mean, -mean);
  float2 sq2 = make_float2(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    if (lane + 32 * i < nvec) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 c = __fadd2_rn(v[i][e], nmean);
        sq2 = __ffma2_rn(c, c, sq2);
      }
    }
  }
  const float rstd = 1.0f / sqrtf(warp_sum(sq2.x + sq2.y) / (float)cols + eps);
  if (lane == 0) stats[row] = make_float2(mean, rstd);
}

cudaError_t launch_rowstats_bf16(const bf16* x, float eps, float2* stats, int rows, int cols, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  if (cols % 8 != 0 || cols > 8 * 256) return cudaErrorInvalidValue;
  const int nch = (cols / 8 + 31) / 32;
  const int threads = 256;
  const unsigned blocks = (unsigned)(((size_t)rows * 32 + threads - 1) / threads);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(threads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t err = cudaSuccess;
#define RS_CASE(N) \
  case N: err = cudaLaunchKernelEx(&cfg, rowstats_bf16_kernel<N>, x, eps, stats, rows, cols); break;
  switch (nch) {
    RS_CASE(1) RS_CASE(2) RS_CASE(3) RS_CASE(4) RS_CASE(5) RS_CASE(6) RS_CASE(7) RS_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef RS_CASE
  return err;
}

// fp32 LayerNorm: one warp per row, two passes over global memory.
__global__ void layernorm_f32_kernel(const float* __restrict__ x, const float* __restrict__ g,
                                     const float* __restrict__ b, float eps, float* __restrict__ y,
                                     int rows, int cols) {
  const int row = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float* xr = x + (size_t)row * cols;
  float sum = 0.f;
  for (int i = lane; i < cols; i += 32) sum += xr[i];
  const float mean = warp_sum(sum) / (float)cols;
  float sq = 0.f;
  for (int i = lane; i < cols; i += 32) {
    const float c = xr[i] - mean;
    sq += c * c;
  }
  const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)cols + eps);
  float* yr = y + (size_t)row * cols;
  for (int i = lane; i < cols; i += 32) yr[i] = (xr[i] - mean) * rstd * g[i] + b[i];
}

cudaError_t launch_layernorm_f32(const float* x, const float* g, const float* b, float eps,
                                 float* y, int rows, int cols, cudaStream_t s) {
  if (rows <= 0) return cudaSuccess;
  const int threads = 256;
  const unsigned blocks = (unsigned)(((size_t)rows * 32 + threads - 1) / threads);
  layernorm_f32_kernel<<<blocks, threads, 0, s>>>(x, g, b, eps, y, rows, cols);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// fp32 linear: out = epi(a . w^T + bias).  64x64 tile, 16-deep k slices in shared memory,
// each of 256 threads owns a 4x4 block.  Sums run in k order, plain FFMA.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
linear_f32_kernel(LinearArgs p) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const float* A = static_cast<const float*>(p.a);
  const float* W = static_cast<const float*>(p.w);
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < p.K; k0 += 16) {
    for (int i = tid; i < 64 * 16; i += 256) {
      const int r = i >> 4, k = i & 15;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + k;
      As[k][r] = (gm < p.M && gk < p.K) ? A[(size_t)gm * p.lda + gk] : 0.f;
      Ws[k][r] = (gn < p.N && gk < p.K) ? W[(size_t)gn * p.ldw + gk] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* out = static_cast<float*>(p.out);
  const float* res = static_cast<const float*>(p.residual);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = m0 + ty * 4 + i;
    if (r >= p.M) continue;
    size_t orow = (size_t)r;
    const float* posrow = nullptr;
    if (p.epilogue == EPI_BIAS_POS) {
      const int img = r / p.n_patches, pt = r % p.n_patches;
      const int t0 = p.first_patch_token > 0 ? p.first_patch_token : 1;
      orow = (size_t)img * (p.n_patches + t0) + t0 + pt;
      posrow = p.pos + (size_t)(t0 + pt) * p.N;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c >= p.N) continue;
      float v = acc[i][j] + p.bias[c];
      if (p.epilogue == EPI_BIAS_GELU) v = gelu_erf(v);
      else if (p.epilogue == EPI_BIAS_RESIDUAL) v += res[(size_t)r * p.ldo + c];
      else if (p.epilogue == EPI_BIAS_POS) v += posrow[c];
      out[orow * p.ldo + c] = v;
    }
  }
}

cudaError_t launch_linear_f32(const LinearArgs& a, cudaStream_t s) {
  if (a.M <= 0 || a.N <= 0) return cudaSuccess;
  dim3 grid((a.N + 63) / 64, (a.M + 63) / 64);
  linear_f32_kernel<<<grid, 256, 0, s>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// fp32 attention: one warp per query row; scores for all T keys in shared memory.
// grid = (images*heads, query blocks), 4 warps per block.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
attention_f32_kernel(const float* __restrict__ qkv, float* __restrict__ out, int T, int heads,
                     int d) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* sc = smem + warp * (T + d);
  float* qv = sc + T;
  const int img = blockIdx.x / heads, hd = blockIdx.x % heads;
  const int H = heads * d;
  const size_t ld = (size_t)3 * H;
  const float* base = qkv + (size_t)img * T * ld + (size_t)hd * d;
  const float scale = 1.0f / sqrtf((float)d);
  for (int t = blockIdx.y * 4 + warp; t < T; t += gridDim.y * 4) {
    for (int c = lane; c < d; c += 32) qv[c] = base[(size_t)t * ld + c];
    __syncwarp();
    float mx = -INFINITY;
    for (int u = lane; u < T; u += 32) {
      const float* kr = base + (size_t)u * ld + H;
      float s = 0.f;
      for (int c = 0; c < d; ++c) s = fmaf(qv[c], kr[c], s);
      s *= scale;
      sc[u] = s;
      mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int u = lane; u < T; u += 32) {
      const float e = expf(sc[u] - mx);
      sc[u] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    __syncwarp();
    const float inv = 1.0f / sum;
    for (int c = lane; c < d; c += 32) {
      float o = 0.f;
      for (int u = 0; u < T; ++u) o = fmaf(sc[u], base[(size_t)u * ld + 2 * H + c], o);
      out[((size_t)img * T + t) * H + (size_t)hd * d + c] = o * inv;
    }
    __syncwarp();
  }
}

cudaError_t launch_attention_f32(const float* qkv, float* out, int images, int T, int heads, int d,
                                 cudaStream_t s) {
  if (images <= 0) return cudaSuccess;
  const size_t smem = (size_t)4 * (T + d) * sizeof(float);
  if (smem > 48 * 1024) return cudaErrorInvalidValue;
  dim3 grid(images * heads, (T + 31) / 32);
  attention_f32_kernel<<<grid, 128, smem, s>>>(qkv, out, T, heads, d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Patch embedding helpers.
// im2col: pixels fp32 [n, C, S, S] -> rows [n*G*G, k_pad], column c*P*P + i*P + j, zero padded
// from C*P*P to k_pad.  One thread writes 8 consecutive columns.
// ------------------------------------------------------------------------------------------
template <typename TOut>
__global__ void im2col_kernel(const float* __restrict__ px, TOut* __restrict__ cols, int images,
                              int C, int S, int P, int k_pad) {
  const int G = S / P, K = C * P * P, PP = P * P;
  const int chunks = k_pad >> 3;
  const size_t total = (size_t)images * G * G * chunks;
  for (size_t idx = blockIdx.x * (size_t)blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int q = (int)(idx % chunks);
    const size_t row = idx / chunks;
    const int pt = (int)(row % (G * G));
    const int img = (int)(row / (G * G));
    const int py = pt / G, pxx = pt % G;
    float v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int k = q * 8 + e;
      if (k < K) {
        const int c = k / PP, r = k % PP, i = r / P, j = r % P;
        v[e] = __ldg(px + (((size_t)img * C + c) * S + (py * P + i)) * S + (pxx * P + j));
      } else {
        v[e] = 0.f;
      }
    }
    TOut* o = cols + row * k_pad + q * 8;
    if (sizeof(TOut) == 2) {                      // bf16: the eight columns as one 16-byte store
      uint4 w;
      __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
      for (int e = 0; e < 4; ++e) h2[e] = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
      *reinterpret_cast<uint4*>(o) = w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = (TOut)v[e];
    }
  }
}

cudaError_t launch_im2col(const float* pixels, void* cols, int images, int C, int S, int P,
                          int k_pad, bool act_bf16, cudaStream_t s) {
  if (images <= 0) return cudaSuccess;
  if (k_pad % 8 != 0) return cudaErrorInvalidValue;
  const int G = S / P;
  const size_t total = (size_t)images * G * G * (k_pad / 8);
  const int threads = 256;
  const unsigned blocks = (unsigned)((total + threads - 1) / threads < 148u * 64u
                                         ? (total + threads - 1) / threads
                                         : 148u * 64u);
  if (act_bf16)
    im2col_kernel<bf16><<<blocks, threads, 0, s>>>(pixels, (bf16*)cols, images, C, S, P, k_pad);
  else
    im2col_kernel<float><<<blocks, threads, 0, s>>>(pixels, (float*)cols, images, C, S, P, k_pad);
  return cudaGetLastError();
}

// Special tokens of every image: token 0 = cls + pos[0]; token 1 = dist + pos[1] when the model
// has a distillation token (n_special = 2).
template <typename TOut>
__global__ void cls_rows_kernel(const float* __restrict__ cls, const float* __restrict__ dist,
                                const float* __restrict__ pos, TOut* __restrict__ tokens, int images,
                                int T, int H, int n_special) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= images * n_special * H) return;
  const int c = i % H, r = (i / H) % n_special, img = i / (H * n_special);
  const float v = (r == 0 ? cls[c] : dist[c]) + pos[(size_t)r * H + c];
  tokens[((size_t)img * T + r) * H + c] = (TOut)v;
}

cudaError_t launch_cls_rows(const float* cls, const float* dist, const float* pos, void* tokens, int images,
                            int T, int H, bool act_bf16, cudaStream_t s) {
  if (images <= 0) return cudaSuccess;
  const int n_special = dist ? 2 : 1;
  const int threads = 256, blocks = (images * n_special * H + threads - 1) / threads;
  if (act_bf16)
    cls_rows_kernel<bf16><<<blocks, threads, 0, s>>>(cls, dist, pos, (bf16*)tokens, images, T, H, n_special);
  else
    cls_rows_kernel<float><<<blocks, threads, 0, s>>>(cls, dist, pos, (float*)tokens, images, T, H, n_special);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Classification head: (1) LayerNorm of the class token (and of the distillation token, if the
// model has one) of every image into fp32 features, (2) logits[img, c] = feat[img] . W[c] + bias[c],
// one warp per class looping over images; with two classifiers the mean of the two.
// ------------------------------------------------------------------------------------------
template <typename TIn>
__global__ void head_ln_kernel(const TIn* __restrict__ tokens, const float* __restrict__ g,
                               const float* __restrict__ b, float eps, float* __restrict__ feat,
                               int images, int T, int H, int n_special) {
  const int idx = (int)((blockIdx.x * (size_t)blockDim.x + threadIdx.x) >> 5);   // image * n_special + token
  const int lane = threadIdx.x & 31;
  if (idx >= images * n_special) return;
  const int img = idx / n_special, r = idx % n_special;
  const TIn* xr = tokens + ((size_t)img * T + r) * H;
  float sum = 0.f;
  for (int i = lane; i < H; i += 32) sum += (float)xr[i];
  const float mean = warp_sum(sum) / (float)H;
  float sq = 0.f;
  for (int i = lane; i < H; i += 32) {
    const float c = (float)xr[i] - mean;
    sq += c * c;
  }
  const float rstd = 1.0f / sqrtf(warp_sum(sq) / (float)H + eps);
  for (int i = lane; i < H; i += 32)
    feat[(size_t)idx * H + i] = ((float)xr[i] - mean) * rstd * g[i] + b[i];
}

// One warp per class and group of HEAD_IMGS images: a weight element is loaded once and used
// for every image of the group, and the groups give the grid enough warps to hide latency.
constexpr int HEAD_IMGS = 8;
template <typename TW>
__global__ void __launch_bounds__(256)
head_logits_kernel(const float* __restrict__ feat, const TW* __restrict__ W,
                   const float* __restrict__ bias, const TW* __restrict__ W2,
                   const float* __restrict__ bias2, float* __restrict__ logits, int images, int H,
                   int classes) {
  const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int img0 = blockIdx.y * HEAD_IMGS;
  if (c >= classes) return;
  const int n_special = W2 ? 2 : 1;
  float acc[HEAD_IMGS];
#pragma unroll
  for (int j = 0; j < HEAD_IMGS; ++j) acc[j] = 0.f;
  for (int r = 0; r < n_special; ++r) {
    const TW* wr = (r == 0 ? W : W2) + (size_t)c * H;
    for (int i = lane; i < H; i += 32) {
      const float w = (float)wr[i];
#pragma unroll
      for (int j = 0; j < HEAD_IMGS; ++j) {
        const int img = img0 + j < images ? img0 + j : images - 1;
        acc[j] = fmaf(feat[((size_t)img * n_special + r) * H + i], w, acc[j]);
      }
    }
  }
  const float bc = W2 ? bias[c] + bias2[c] : bias[c];
  const float scale = W2 ? 0.5f : 1.0f;
#pragma unroll
  for (int j = 0; j < HEAD_IMGS; ++j) {
    const float s = warp_sum(acc[j]);
    if (lane == 0 && img0 + j < images) logits[(size_t)(img0 + j) * classes + c] = (s + bc) * scale;
  }
}

cudaError_t launch_head(const void* tokens, const float* g, const float* b, float eps,
                        const void* W, const float* bias, const void* W2, const float* bias2, float* feat,
                        float* logits, int images, int T, int H, int classes, bool act_bf16, cudaStream_t s) {
  if (images <= 0) return cudaSuccess;
  const int n_special = W2 ? 2 : 1;
  const int threads = 256;
  const unsigned b1 = (unsigned)(((size_t)images * n_special * 32 + threads - 1) / threads);
  const dim3 b2((unsigned)((classes + 7) / 8), (unsigned)((images + HEAD_IMGS - 1) / HEAD_IMGS));
  if (act_bf16) {
    head_ln_kernel<bf16><<<b1, threads, 0, s>>>((const bf16*)tokens, g, b, eps, feat, images, T, H, n_special);
    head_logits_kernel<bf16><<<b2, threads, 0, s>>>(feat, (const bf16*)W, bias, (const bf16*)W2, bias2, logits, images, H, classes);
  } else {
    head_ln_kernel<float><<<b1, threads, 0, s>>>((const float*)tokens, g, b, eps, feat, images, T, H, n_special);
    head_logits_kernel<float><<<b2, threads, 0, s>>>(feat, (const float*)W, bias, (const float*)W2, bias2, logits, images, H, classes);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Head without caller scratch: the class-token features go to a fixed array that is part of
// the library image, for callers that have no way to allocate device memory.
// In host code the array's name is only a handle for the runtime; the address the kernels need
// is looked up once per device with cudaGetSymbolAddress while that device is current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) float g_head_static_scratch[VIT_HEAD_STATIC_MAX_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_ptr[kMaxDevices] = {};
}  // namespace

cudaError_t launch_head_static(const void* tokens, const float* g, const float* b, float eps,
                               const void* W, const float* bias, const void* W2, const float* bias2,
                               float* logits, int images, int T,
                               int H, int classes, bool act_bf16, cudaStream_t s) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
      float* ptr = nullptr;
      e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_head_static_scratch);
      if (e != cudaSuccess) return e;
      if (ptr == nullptr) return cudaErrorInvalidSymbol;
      g_static_ptr[dev] = ptr;
    }
    scratch = g_static_ptr[dev];
  }
  // Every feature the logits kernel reads is written by the LayerNorm kernel of the same call
  // first, so nothing in the array has to start at zero.
  return launch_head(tokens, g, b, eps, W, bias, W2, bias2, scratch, logits, images, T, H, classes, act_bf16, s);
}

}  // namespace vit
