// C boundary: configuration checks, parameter upload, the per-layer kernel sequence of a stage,
// the book-ends and the stage runner.  Everything here is host code; the arithmetic is in the
// kernels it launches.
#include "vit_internal.h"

#include <cuda_bf16.h>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

using namespace vit;

struct vit_handle : public vit::Handle {};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool config_ok(const vit_config* c) {
  if (!c) return false;
  if (c->image_size <= 0 || c->patch_size <= 0 || c->channels <= 0) return false;
  if (c->image_size % c->patch_size) return false;
  if (c->hidden <= 0 || c->heads <= 0 || c->hidden % c->heads) return false;
  const int d = c->hidden / c->heads;
  if (d % 16 || d > 128) return false;
  if (c->hidden % 64 || c->hidden > 2048) return false;
  if (c->mlp_dim <= 0 || c->mlp_dim % 64) return false;
  if (c->layers <= 0 || c->num_classes <= 0 || c->max_microbatch <= 0) return false;
  if (c->dtype != VIT_BF16 && c->dtype != VIT_FP32) return false;
  if (!(c->ln_eps >= 0.f)) return false;
  if (c->extra_tokens != 0 && c->extra_tokens != 1) return false;
  const int g = c->image_size / c->patch_size;
  if (g * g + 1 + c->extra_tokens > 512) return false;
  return true;
}

struct Shape {
  int T, Np, d, Kpe, Kpad, X;      // X: special tokens besides the class token
  size_t H, F, C;
  explicit Shape(const vit_config& c) {
    const int g = c.image_size / c.patch_size;
    Np = g * g;
    X = c.extra_tokens;
    T = Np + 1 + X;
    d = c.hidden / c.heads;
    Kpe = c.channels * c.patch_size * c.patch_size;
    Kpad = (Kpe + 63) / 64 * 64;
    H = c.hidden; F = c.mlp_dim; C = c.num_classes;
  }
};

size_t param_count(const vit_config& c) {
  const Shape s(c);
  size_t n = s.H * s.Kpe + s.H + s.H + (size_t)s.X * s.H + (size_t)s.T * s.H;
  const size_t per_layer = 2 * s.H + 3 * s.H * s.H + 3 * s.H + s.H * s.H + s.H + 2 * s.H +
                           s.F * s.H + s.F + s.H * s.F + s.H;
  n += per_layer * c.layers;
  n += 2 * s.H + (1 + (size_t)s.X) * (s.C * s.H + s.C);
  return n;
}

size_t stage_ws_bytes(const vit_config& c, int mb) {
  const Shape s(c);
  const size_t act = c.dtype == VIT_BF16 ? 2 : 4;
  const size_t M = (size_t)mb * s.T;
  const size_t wide = 3 * s.H > s.F ? 3 * s.H : s.F;
  return align_up(M * s.H * act, 256) + align_up(M * wide * act, 256) + align_up(M * sizeof(float2), 256);
}
size_t embed_ws_bytes(const vit_config& c, int mb) {
  const Shape s(c);
  const size_t act = c.dtype == VIT_BF16 ? 2 : 4;
  return align_up((size_t)mb * s.Np * s.Kpad * act, 256);
}
size_t head_ws_bytes(const vit_config& c, int mb) {
  const Shape s(c);
  return align_up((size_t)mb * (1 + s.X) * s.H * sizeof(float), 256);
}
size_t call_ws_bytes(const vit_config& c, int mb) {
  size_t w = stage_ws_bytes(c, mb);
  if (embed_ws_bytes(c, mb) > w) w = embed_ws_bytes(c, mb);
  if (head_ws_bytes(c, mb) > w) w = head_ws_bytes(c, mb);
  return w;
}
struct PipeLayout { size_t pixels, logits, tokens, scratch, total; };
PipeLayout pipe_layout(const vit_config& c, int mb) {
  const Shape s(c);
  const size_t act = c.dtype == VIT_BF16 ? 2 : 4;
  PipeLayout l;
  size_t off = 0;
  l.pixels = off; off += align_up((size_t)mb * c.channels * c.image_size * c.image_size * 4, 256);
  l.logits = off; off += align_up((size_t)mb * s.C * 4, 256);
  l.tokens = off; off += align_up((size_t)mb * s.T * s.H * act, 256);
  l.scratch = off; off += call_ws_bytes(c, mb);
  l.total = off;
  return l;
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

// Converts n fp32 values to the device element type into dst (host staging).
void convert_matrix(const float* src, void* dst, size_t rows, size_t cols, size_t cols_pad, bool to_bf16,
                    const float* col_scale = nullptr) {
  if (to_bf16) {
    bf16* d = static_cast<bf16*>(dst);
    for (size_t r = 0; r < rows; ++r) {
      if (col_scale)
        for (size_t c = 0; c < cols; ++c) d[r * cols_pad + c] = __float2bfloat16_rn(src[r * cols + c] * col_scale[c]);
      else
        for (size_t c = 0; c < cols; ++c) d[r * cols_pad + c] = __float2bfloat16_rn(src[r * cols + c]);
      for (size_t c = cols; c < cols_pad; ++c) d[r * cols_pad + c] = __float2bfloat16_rn(0.f);
    }
  } else {
    float* d = static_cast<float*>(dst);
    for (size_t r = 0; r < rows; ++r) {
      memcpy(d + r * cols_pad, src + r * cols, cols * sizeof(float));
      for (size_t c = cols; c < cols_pad; ++c) d[r * cols_pad + c] = 0.f;
    }
  }
}

// Brackets one kernel launch with a pair of events on its stream while profiling is on.
struct ProfScope {
  Handle* h; cudaStream_t s; int cls; cudaEvent_t a = nullptr, b = nullptr;
  ProfScope(Handle* h_, cudaStream_t s_, int cls_) : h(h_), s(s_), cls(cls_) {
    if (!h->profiling) return;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { a = b = nullptr; return; }
    cudaEventRecord(a, s);
  }
  ~ProfScope() {
    if (!a) return;
    cudaEventRecord(b, s);
    h->prof.push_back(ProfRecord{a, b, cls});
  }
};

#define VIT_LAUNCH(h, cls, expr)                     \
  do {                                               \
    ProfScope prof__((h), s, (cls));                 \
    cudaError_t e__ = (expr);                        \
    if (e__ != cudaSuccess) return VIT_ERR_CUDA;     \
    (h)->launches.fetch_add(1, std::memory_order_relaxed); \
  } while (0)

int linear(Handle* h, int cls, const LinearArgs& a, cudaStream_t s) {
  if (h->cfg.dtype == VIT_BF16) VIT_LAUNCH(h, cls, launch_linear_tc(a, h->dev_status, s, &h->tmaps));
  else VIT_LAUNCH(h, cls, launch_linear_f32(a, s));
  return VIT_OK;
}

// A handle's parameters, status word and kernel attributes live on the device it was created on.
bool on_own_device(const vit_handle* h) {
  int dev = -1;
  return h && cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

int check_call(const vit_handle* h, int mb, const void* ws, size_t ws_bytes, size_t need) {
  if (!h || mb < 1 || mb > h->cfg.max_microbatch || !ws || misaligned(ws)) return VIT_ERR_INVALID_ARG;
  if (!on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (ws_bytes < need) return VIT_ERR_WORKSPACE;
  return VIT_OK;
}

int check_stages(const vit_handle* h, const int32_t* stage_layers, int n_stages) {
  if (!stage_layers || n_stages < 1) return VIT_ERR_INVALID_ARG;
  long long sum = 0;
  for (int i = 0; i < n_stages; ++i) {
    if (stage_layers[i] < 1) return VIT_ERR_RANGE;
    sum += stage_layers[i];
  }
  return sum == h->cfg.layers ? VIT_OK : VIT_ERR_RANGE;
}

int run_pipeline(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch, int mb,
                 const float* pixels, float* logits, void* const* wss, size_t ws_bytes,
                 void* const* streams, int n_streams, bool host_io) {
  if (!h || !pixels || !logits || !wss || !streams || n_streams < 1 || batch < 1 || mb < 1 ||
      mb > h->cfg.max_microbatch || !on_own_device(h))
    return VIT_ERR_INVALID_ARG;
  if (!host_io && (misaligned(pixels) || misaligned(logits))) return VIT_ERR_INVALID_ARG;
  int st = check_stages(h, stage_layers, n_stages);
  if (st != VIT_OK) return st;
  const PipeLayout lay = pipe_layout(h->cfg, mb);
  if (ws_bytes < lay.total) return VIT_ERR_WORKSPACE;
  for (int i = 0; i < n_streams; ++i)
    if (!wss[i] || misaligned(wss[i])) return VIT_ERR_INVALID_ARG;
  const size_t img_elems = (size_t)h->cfg.channels * h->cfg.image_size * h->cfg.image_size;
  const size_t scratch_bytes = lay.total - lay.scratch;
  int m = 0;
  for (int first = 0; first < batch; first += mb, ++m) {
    const int n = batch - first < mb ? batch - first : mb;
    cudaStream_t s = static_cast<cudaStream_t>(streams[m % n_streams]);
    uint8_t* ws = static_cast<uint8_t*>(wss[m % n_streams]);
    void* tokens = ws + lay.tokens;
    void* scratch = ws + lay.scratch;
    const float* px = pixels + (size_t)first * img_elems;
    float* lg = logits + (size_t)first * h->cfg.num_classes;
    if (host_io) {
      float* dpx = reinterpret_cast<float*>(ws + lay.pixels);
      if (cudaMemcpyAsync(dpx, px, (size_t)n * img_elems * 4, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return VIT_ERR_CUDA;
      px = dpx;
      lg = reinterpret_cast<float*>(ws + lay.logits);
    }
    st = vit_patch_embed(h, n, px, tokens, scratch, scratch_bytes, s);
    if (st != VIT_OK) return st;
    int lb = 0;
    for (int i = 0; i < n_stages; ++i) {
      st = vit_run_stage(h, lb, lb + stage_layers[i], n, tokens, tokens, scratch, scratch_bytes, s);
      if (st != VIT_OK) return st;
      lb += stage_layers[i];
    }
    st = vit_head(h, n, tokens, lg, scratch, scratch_bytes, s);
    if (st != VIT_OK) return st;
    if (host_io) {
      if (cudaMemcpyAsync(logits + (size_t)first * h->cfg.num_classes, lg,
                          (size_t)n * h->cfg.num_classes * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return VIT_ERR_CUDA;
    }
  }
  return VIT_OK;
}

}  // namespace

extern "C" {

size_t vit_param_count(const vit_config* cfg) { return config_ok(cfg) ? param_count(*cfg) : 0; }

size_t vit_workspace_bytes(const vit_config* cfg, int microbatch) {
  if (!config_ok(cfg) || microbatch < 1) return 0;
  return call_ws_bytes(*cfg, microbatch);
}

size_t vit_pipeline_workspace_bytes(const vit_config* cfg, int microbatch) {
  if (!config_ok(cfg) || microbatch < 1) return 0;
  return pipe_layout(*cfg, microbatch).total;
}

int vit_create(const vit_config* cfg, const float* host_params, size_t n_params, vit_handle** out) {
  if (!cfg || !host_params || !out) return VIT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return VIT_ERR_CONFIG;
  if (n_params != param_count(*cfg)) return VIT_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return VIT_ERR_NO_DEVICE;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return VIT_ERR_NO_DEVICE;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (major != 10) return VIT_ERR_NO_DEVICE;
  if (!tc_gemm_init()) return VIT_ERR_NO_DEVICE;

  const Shape s(*cfg);
  const bool b16 = cfg->dtype == VIT_BF16;
  const size_t act = b16 ? 2 : 4;
  const int L = cfg->layers;

  // device blob layout: every tensor 256-byte aligned
  struct Item { size_t src, rows, cols, cols_pad; bool matrix; size_t dst; const float* col_scale; };
  std::vector<Item> items;
  size_t src = 0, dst = 0;
  auto add = [&](size_t rows, size_t cols, size_t cols_pad, bool matrix) {
    Item it{src, rows, cols, cols_pad, matrix, dst, nullptr};
    items.push_back(it);
    src += rows * cols;
    dst += align_up(rows * cols_pad * (matrix ? act : 4), 256);
    return items.size() - 1;
  };
  const size_t i_pw = add(s.H, s.Kpe, s.Kpad, true);
  const size_t i_pb = add(1, s.H, s.H, false);
  const size_t i_cls = add(1, s.H, s.H, false);
  const size_t i_dist = s.X ? add(1, s.H, s.H, false) : 0;
  const size_t i_pos = add(s.T, s.H, s.H, false);
  std::vector<size_t> li(L);
  for (int l = 0; l < L; ++l) {
    li[l] = add(1, s.H, s.H, false);      // ln1.g
    add(1, s.H, s.H, false);              // ln1.b
    add(3 * s.H, s.H, s.H, true);         // Wqkv
    add(1, 3 * s.H, 3 * s.H, false);      // bqkv
    add(s.H, s.H, s.H, true);             // Wo
    add(1, s.H, s.H, false);              // bo
    add(1, s.H, s.H, false);              // ln2.g
    add(1, s.H, s.H, false);              // ln2.b
    add(s.F, s.H, s.H, true);             // W1
    add(1, s.F, s.F, false);              // b1
    add(s.H, s.F, s.F, true);             // W2
    add(1, s.H, s.H, false);              // b2
  }
  const size_t i_lnfg = add(1, s.H, s.H, false);
  const size_t i_lnfb = add(1, s.H, s.H, false);
  const size_t i_hw = add(s.C, s.H, s.H, true);
  const size_t i_hb = add(1, s.C, s.C, false);
  const size_t i_hdw = s.X ? add(s.C, s.H, s.H, true) : 0;
  const size_t i_hdb = s.X ? add(1, s.C, s.C, false) : 0;
  if (src != n_params) return VIT_ERR_INVALID_ARG;
  // bf16 mode: LayerNorm 1 and 2 are folded into the QKV and fc1 products.  The gain goes into the
  // weight (wg[n,k] = g[k] w[n,k], rounded to bf16); per layer four derived vectors follow the
  // parameters: c1[n] = sum_k wg[n,k] and c0[n] = bias[n] + sum_k shift[k] w[n,k] for each of the two.
  struct Derived { size_t dst, w_item, g_item, b_item, bias_item; };
  std::vector<Derived> derived;
  std::vector<size_t> ld(L, 0);
  if (b16) {
    for (int l = 0; l < L; ++l) {
      const size_t b = li[l];
      items[b + 2].col_scale = host_params + items[b + 0].src;      // Wqkv * ln1.g
      items[b + 8].col_scale = host_params + items[b + 6].src;      // W1 * ln2.g
      ld[l] = derived.size();
      for (int which = 0; which < 2; ++which) {
        const size_t w = b + (which ? 8 : 2), g = b + (which ? 6 : 0);
        const size_t n = items[w].rows;
        for (int v = 0; v < 2; ++v) {                                // c1 then c0
          derived.push_back(Derived{dst, w, g, g + 1, w + 1});
          dst += align_up(n * sizeof(float), 256);
        }
      }
    }
  }
  const size_t blob_bytes = dst;

  uint8_t* staging = static_cast<uint8_t*>(malloc(blob_bytes));
  if (!staging) return VIT_ERR_CUDA;
  {
    unsigned nt = std::thread::hardware_concurrency();
    if (nt < 1) nt = 1;
    if (nt > 16) nt = 16;
    std::vector<std::thread> pool;
    for (unsigned t = 0; t < nt; ++t) {
      pool.emplace_back([&, t]() {
        for (size_t i = t; i < items.size(); i += nt) {
          const Item& it = items[i];
          convert_matrix(host_params + it.src, staging + it.dst, it.rows, it.cols, it.cols_pad,
                         it.matrix && b16, it.col_scale);
        }
        for (size_t i = t; i < derived.size(); i += nt) {
          const Derived& d = derived[i];
          const Item& w = items[d.w_item];
          const float* W = host_params + w.src;
          const float* g = host_params + items[d.g_item].src;
          const float* sh = host_params + items[d.b_item].src;
          const float* bias = host_params + items[d.bias_item].src;
          float* out = reinterpret_cast<float*>(staging + d.dst);
          const bool is_c1 = (i % 2) == 0;
          for (size_t n = 0; n < w.rows; ++n) {
            double acc = is_c1 ? 0.0 : (double)bias[n];
            for (size_t k = 0; k < w.cols; ++k) {
              const float wv = W[n * w.cols + k];
              acc += is_c1 ? (double)__bfloat162float(__float2bfloat16_rn(wv * g[k]))
                           : (double)sh[k] * (double)__bfloat162float(__float2bfloat16_rn(wv));
            }
            out[n] = (float)acc;
          }
        }
      });
    }
    for (auto& th : pool) th.join();
  }

  void* dev_blob = nullptr;
  int* dev_status = nullptr;
  if (cudaMalloc(&dev_blob, blob_bytes) != cudaSuccess) { free(staging); return VIT_ERR_CUDA; }
  if (cudaMalloc(&dev_status, 2 * sizeof(int)) != cudaSuccess) { cudaFree(dev_blob); free(staging); return VIT_ERR_CUDA; }
  cudaError_t e = cudaMemcpy(dev_blob, staging, blob_bytes, cudaMemcpyHostToDevice);
  free(staging);
  if (e == cudaSuccess) e = cudaMemset(dev_status, 0, 2 * sizeof(int));
  if (e != cudaSuccess) { cudaFree(dev_blob); cudaFree(dev_status); return VIT_ERR_CUDA; }

  vit_handle* h = new (std::nothrow) vit_handle();
  if (!h) { cudaFree(dev_blob); cudaFree(dev_status); return VIT_ERR_CUDA; }
  h->cfg = *cfg;
  h->device = dev;
  h->T = s.T; h->n_patches = s.Np; h->d = s.d; h->patch_k = s.Kpe; h->patch_k_pad = s.Kpad;
  h->act_bytes = act;
  h->dev_blob = dev_blob;
  h->dev_blob_bytes = blob_bytes;
  h->dev_status = dev_status;
  h->launches.store(0);
  h->profiling = false;
  const uint8_t* B = static_cast<const uint8_t*>(dev_blob);
  auto fp = [&](size_t i) { return reinterpret_cast<const float*>(B + items[i].dst); };
  auto vp = [&](size_t i) { return static_cast<const void*>(B + items[i].dst); };
  h->patch_W = vp(i_pw); h->patch_b = fp(i_pb); h->cls = fp(i_cls); h->dist = s.X ? fp(i_dist) : nullptr; h->pos = fp(i_pos);
  h->layers = new LayerWeights[L];
  for (int l = 0; l < L; ++l) {
    const size_t b = li[l];
    LayerWeights& w = h->layers[l];
    w.ln1_g = fp(b); w.ln1_b = fp(b + 1); w.Wqkv = vp(b + 2); w.bqkv = fp(b + 3);
    w.Wo = vp(b + 4); w.bo = fp(b + 5); w.ln2_g = fp(b + 6); w.ln2_b = fp(b + 7);
    w.W1 = vp(b + 8); w.b1 = fp(b + 9); w.W2 = vp(b + 10); w.b2 = fp(b + 11);
    w.qkv_c1 = w.qkv_c0 = w.fc1_c1 = w.fc1_c0 = nullptr;
    if (b16) {
      auto dp = [&](size_t i) { return reinterpret_cast<const float*>(B + derived[ld[l] + i].dst); };
      w.qkv_c1 = dp(0); w.qkv_c0 = dp(1); w.fc1_c1 = dp(2); w.fc1_c0 = dp(3);
    }
  }
  h->lnf_g = fp(i_lnfg); h->lnf_b = fp(i_lnfb); h->head_W = vp(i_hw); h->head_b = fp(i_hb);
  h->head_dist_W = s.X ? vp(i_hdw) : nullptr; h->head_dist_b = s.X ? fp(i_hdb) : nullptr;
  *out = h;
  return VIT_OK;
}

int vit_destroy(vit_handle* h) {
  if (!h) return VIT_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  for (const ProfRecord& r : h->prof) { cudaEventDestroy(r.begin); cudaEventDestroy(r.end); }
  cudaFree(h->dev_blob);
  cudaFree(h->dev_status);
  delete[] h->layers;
  delete h;
  return VIT_OK;
}

int vit_patch_embed(vit_handle* h, int mb, const float* pixels, void* tokens_out, void* ws,
                    size_t ws_bytes, void* stream) {
  int st = check_call(h, mb, ws, ws_bytes, h ? embed_ws_bytes(h->cfg, mb) : 0);
  if (st != VIT_OK) return st;
  if (!pixels || !tokens_out || misaligned(pixels) || misaligned(tokens_out)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const vit_config& c = h->cfg;
  const bool b16 = c.dtype == VIT_BF16;
  VIT_LAUNCH(h, VIT_PROF_EMBED, launch_im2col(pixels, ws, mb, c.channels, c.image_size, c.patch_size, h->patch_k_pad, b16, s));
  LinearArgs a{};
  a.M = mb * h->n_patches; a.N = c.hidden; a.K = h->patch_k_pad;
  a.a = ws; a.lda = h->patch_k_pad;
  a.w = h->patch_W; a.ldw = h->patch_k_pad;
  a.bias = h->patch_b;
  a.epilogue = EPI_BIAS_POS;
  a.pos = h->pos; a.n_patches = h->n_patches; a.first_patch_token = 1 + c.extra_tokens;
  a.out = tokens_out; a.ldo = c.hidden;
  st = linear(h, VIT_PROF_EMBED, a, s);
  if (st != VIT_OK) return st;
  VIT_LAUNCH(h, VIT_PROF_EMBED, launch_cls_rows(h->cls, h->dist, h->pos, tokens_out, mb, h->T, c.hidden, b16, s));
  return VIT_OK;
}

int vit_run_stage(vit_handle* h, int layer_begin, int layer_end, int mb, const void* in, void* out,
                  void* ws, size_t ws_bytes, void* stream) {
  int st = check_call(h, mb, ws, ws_bytes, h ? stage_ws_bytes(h->cfg, mb) : 0);
  if (st != VIT_OK) return st;
  if (!(0 <= layer_begin && layer_begin < layer_end && layer_end <= h->cfg.layers)) return VIT_ERR_RANGE;
  if (!in || !out || misaligned(in) || misaligned(out)) return VIT_ERR_INVALID_ARG;
  const vit_config& c = h->cfg;
  const size_t M = (size_t)mb * h->T;
  const size_t H = c.hidden, F = c.mlp_dim;
  const size_t tok_bytes = M * H * h->act_bytes;
  if (in != out) {
    const uint8_t* a = static_cast<const uint8_t*>(in);
    const uint8_t* b = static_cast<const uint8_t*>(out);
    if (a < b + tok_bytes && b < a + tok_bytes) return VIT_ERR_INVALID_ARG;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool b16 = c.dtype == VIT_BF16;
  uint8_t* y = static_cast<uint8_t*>(ws);                       // [M, H]: attention output (fp32 mode: also the LN output)
  uint8_t* wide = y + align_up(tok_bytes, 256);                 // [M, 3H] qkv, later [M, F] MLP hidden
  const size_t wide_cols = 3 * H > F ? 3 * H : F;
  float2* stats = reinterpret_cast<float2*>(wide + align_up(M * wide_cols * h->act_bytes, 256));   // [M] LayerNorm statistics

  for (int l = layer_begin; l < layer_end; ++l) {
    const LayerWeights& w = h->layers[l];
    const void* x_in = (l == layer_begin) ? in : out;
    LinearArgs a{};
    if (b16) {
      // LN1 folded into the QKV product: row statistics of x, then qkv = LN1(x) Wqkv^T + bqkv from the raw rows
      VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_rowstats_bf16((const bf16*)x_in, c.ln_eps, stats, (int)M, (int)H, s));
      a.M = (int)M; a.N = (int)(3 * H); a.K = (int)H;
      a.a = x_in; a.lda = (int)H; a.w = w.Wqkv; a.ldw = (int)H; a.bias = w.qkv_c0;
      a.epilogue = EPI_LN_BIAS; a.ln_stats = stats; a.ln_c1 = w.qkv_c1; a.out = wide; a.ldo = (int)(3 * H);
    } else {
      // y = LN1(x); qkv = y Wqkv^T + bqkv
      VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_layernorm_f32((const float*)x_in, w.ln1_g, w.ln1_b, c.ln_eps, (float*)y, (int)M, (int)H, s));
      a.M = (int)M; a.N = (int)(3 * H); a.K = (int)H;
      a.a = y; a.lda = (int)H; a.w = w.Wqkv; a.ldw = (int)H; a.bias = w.bqkv;
      a.epilogue = EPI_BIAS; a.out = wide; a.ldo = (int)(3 * H);
    }
    if ((st = linear(h, VIT_PROF_QKV, a, s)) != VIT_OK) return st;
    // y = attention(qkv)
    if (b16) VIT_LAUNCH(h, VIT_PROF_ATTENTION, launch_attention_bf16((const bf16*)wide, (bf16*)y, mb, h->T, c.heads, h->d, h->dev_status, s, &h->tmaps));
    else VIT_LAUNCH(h, VIT_PROF_ATTENTION, launch_attention_f32((const float*)wide, (float*)y, mb, h->T, c.heads, h->d, s));
    // x = x + y Wo^T + bo
    a = LinearArgs{};
    a.M = (int)M; a.N = (int)H; a.K = (int)H;
    a.a = y; a.lda = (int)H; a.w = w.Wo; a.ldw = (int)H; a.bias = w.bo;
    a.epilogue = EPI_BIAS_RESIDUAL; a.residual = x_in; a.out = out; a.ldo = (int)H;
    if ((st = linear(h, VIT_PROF_OUTPROJ, a, s)) != VIT_OK) return st;
    // u = gelu(LN2(x) W1^T + b1)
    a = LinearArgs{};
    if (b16) {
      VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_rowstats_bf16((const bf16*)out, c.ln_eps, stats, (int)M, (int)H, s));
      a.M = (int)M; a.N = (int)F; a.K = (int)H;
      a.a = out; a.lda = (int)H; a.w = w.W1; a.ldw = (int)H; a.bias = w.fc1_c0;
      a.epilogue = EPI_LN_BIAS_GELU; a.ln_stats = stats; a.ln_c1 = w.fc1_c1; a.out = wide; a.ldo = (int)F;
    } else {
      VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_layernorm_f32((const float*)out, w.ln2_g, w.ln2_b, c.ln_eps, (float*)y, (int)M, (int)H, s));
      a.M = (int)M; a.N = (int)F; a.K = (int)H;
      a.a = y; a.lda = (int)H; a.w = w.W1; a.ldw = (int)H; a.bias = w.b1;
      a.epilogue = EPI_BIAS_GELU; a.out = wide; a.ldo = (int)F;
    }
    if ((st = linear(h, VIT_PROF_FC1, a, s)) != VIT_OK) return st;
    // x = x + u W2^T + b2
    a = LinearArgs{};
    a.M = (int)M; a.N = (int)H; a.K = (int)F;
    a.a = wide; a.lda = (int)F; a.w = w.W2; a.ldw = (int)F; a.bias = w.b2;
    a.epilogue = EPI_BIAS_RESIDUAL; a.residual = out; a.out = out; a.ldo = (int)H;
    if ((st = linear(h, VIT_PROF_FC2, a, s)) != VIT_OK) return st;
  }
  return VIT_OK;
}

int vit_head(vit_handle* h, int mb, const void* tokens, float* logits, void* ws, size_t ws_bytes,
             void* stream) {
  int st = check_call(h, mb, ws, ws_bytes, h ? head_ws_bytes(h->cfg, mb) : 0);
  if (st != VIT_OK) return st;
  if (!tokens || !logits || misaligned(tokens) || misaligned(logits)) return VIT_ERR_INVALID_ARG;
  const vit_config& c = h->cfg;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  VIT_LAUNCH(h, VIT_PROF_HEAD, launch_head(tokens, h->lnf_g, h->lnf_b, c.ln_eps, h->head_W, h->head_b,
                                           h->head_dist_W, h->head_dist_b, static_cast<float*>(ws), logits, mb, h->T, c.hidden,
                                           c.num_classes, c.dtype == VIT_BF16, s));
  h->launches.fetch_add(1, std::memory_order_relaxed);   // the head is two kernels
  return VIT_OK;
}

int vit_head_static(vit_handle* h, int mb, const void* tokens, float* logits, void* stream) {
  if (!h || mb < 1 || mb > h->cfg.max_microbatch || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (!tokens || !logits || misaligned(tokens) || misaligned(logits)) return VIT_ERR_INVALID_ARG;
  const vit_config& c = h->cfg;
  if ((size_t)mb * (size_t)(1 + c.extra_tokens) * (size_t)c.hidden > (size_t)VIT_HEAD_STATIC_MAX_FLOATS) return VIT_ERR_TOO_LARGE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  VIT_LAUNCH(h, VIT_PROF_HEAD, launch_head_static(tokens, h->lnf_g, h->lnf_b, c.ln_eps, h->head_W,
                                                  h->head_b, h->head_dist_W, h->head_dist_b, logits, mb, h->T, c.hidden,
                                                  c.num_classes, c.dtype == VIT_BF16, s));
  h->launches.fetch_add(1, std::memory_order_relaxed);   // the head is two kernels
  return VIT_OK;
}

int vit_run_pipeline(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch, int mb,
                     const float* pixels, float* logits, void* const* ws_per_stream, size_t ws_bytes,
                     void* const* streams, int n_streams) {
  return run_pipeline(h, stage_layers, n_stages, batch, mb, pixels, logits, ws_per_stream, ws_bytes,
                      streams, n_streams, false);
}

int vit_run_pipeline_grouped(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch, int mb,
                             int group, const float* pixels, float* logits, void* const* ws_per_stream,
                             size_t ws_bytes, void* const* streams, int n_streams) {
  if (group < 1 || mb < 1 || (long long)group * mb > 0x7fffffffLL) return VIT_ERR_INVALID_ARG;
  // images are independent, so `group` microbatches carried through every launch together are the
  // same computation as one microbatch of group * mb images
  return run_pipeline(h, stage_layers, n_stages, batch, group * mb, pixels, logits, ws_per_stream, ws_bytes,
                      streams, n_streams, false);
}

int vit_run_pipeline_host(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch, int mb,
                          const float* host_pixels, float* host_logits, void* const* ws_per_stream,
                          size_t ws_bytes, void* const* streams, int n_streams) {
  return run_pipeline(h, stage_layers, n_stages, batch, mb, host_pixels, host_logits, ws_per_stream,
                      ws_bytes, streams, n_streams, true);
}

int vit_check_status(vit_handle* h, void* stream) {
  if (!h || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // The word is read and cleared in one atomic step on the device, so a timeout raised by a
  // kernel on another stream in the meantime is kept for the next check instead of being lost.
  std::lock_guard<std::mutex> lock(h->status_mutex);    // one snapshot slot per handle
  if (launch_status_take(h->dev_status, h->dev_status + 1, s) != cudaSuccess) return VIT_ERR_CUDA;
  int v = 0;
  if (cudaMemcpyAsync(&v, h->dev_status + 1, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return VIT_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return VIT_ERR_CUDA;
  return v;
}

int vit_profile_enable(vit_handle* h, int on) {
  if (!h) return VIT_ERR_INVALID_ARG;
  h->profiling = on != 0;
  return VIT_OK;
}

int vit_profile_collect(vit_handle* h, double* ms_by_class, uint64_t* launches_by_class) {
  if (!h || !ms_by_class || !launches_by_class) return VIT_ERR_INVALID_ARG;
  for (int i = 0; i < VIT_PROF_CLASSES; ++i) { ms_by_class[i] = 0.0; launches_by_class[i] = 0; }
  int st = VIT_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) st = VIT_ERR_CUDA;
  for (const ProfRecord& r : h->prof) {
    float ms = 0.f;
    if (st == VIT_OK && cudaEventElapsedTime(&ms, r.begin, r.end) == cudaSuccess) {
      ms_by_class[r.cls] += ms;
      launches_by_class[r.cls] += 1;
    }
    cudaEventDestroy(r.begin);
    cudaEventDestroy(r.end);
  }
  h->prof.clear();
  return st;
}

int vit_debug_wait_probe(vit_handle* h, int64_t limit_cycles, void* stream) {
  if (!h || limit_cycles < 1 || limit_cycles > (1ll << 31) || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  VIT_LAUNCH(h, VIT_PROF_OP, launch_wait_probe(limit_cycles, h->dev_status, s));
  return VIT_OK;
}

uint64_t vit_launch_count(const vit_handle* h) { return h ? h->launches.load() : 0; }

const char* vit_status_string(int status) {
  switch (status) {
    case VIT_OK: return "ok";
    case VIT_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, microbatch out of range)";
    case VIT_ERR_RANGE: return "layer range must satisfy 0 <= begin < end <= layers; stage counts must sum to layers";
    case VIT_ERR_CONFIG: return "inconsistent or unsupported model configuration";
    case VIT_ERR_WORKSPACE: return "workspace too small";
    case VIT_ERR_CUDA: return "CUDA call or kernel launch failed";
    case VIT_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
    case VIT_ERR_NO_DEVICE: return "no usable sm_100 device";
    case VIT_ERR_INFEASIBLE: return "no partition fits the devices' memory";
    case VIT_ERR_TOO_LARGE: return "problem larger than the fixed scratch of this allocation-free entry point";
  }
  return "unknown status";
}

int vit_op_layernorm(vit_handle* h, int dtype, int rows, int cols, const void* x, const float* gain,
                     const float* shift, float eps, void* y, void* stream) {
  if (!h || !x || !gain || !shift || !y || rows < 0 || cols < 1 || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (misaligned(x) || misaligned(y) || misaligned(gain) || misaligned(shift)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dtype == VIT_BF16) VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_layernorm_bf16((const bf16*)x, gain, shift, eps, (bf16*)y, rows, cols, s));
  else if (dtype == VIT_FP32) VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_layernorm_f32((const float*)x, gain, shift, eps, (float*)y, rows, cols, s));
  else return VIT_ERR_INVALID_ARG;
  return VIT_OK;
}

int vit_op_linear(vit_handle* h, int dtype, int M, int N, int K, const void* a, const void* w,
                  const float* bias, int epilogue, const void* residual, void* out, void* stream) {
  return vit_op_linear_tiled(h, dtype, M, N, K, a, w, bias, epilogue, residual, out, VIT_TILING_AUTO, stream);
}

int vit_op_linear_tiled(vit_handle* h, int dtype, int M, int N, int K, const void* a, const void* w,
                        const float* bias, int epilogue, const void* residual, void* out, int tiling,
                        void* stream) {
  if (!h || !a || !w || !bias || !out || M < 0 || N < 1 || K < 1 || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (tiling < VIT_TILING_AUTO || tiling > VIT_TILING_PAIR_256x256) return VIT_ERR_INVALID_ARG;
  if (dtype != VIT_BF16 && tiling != VIT_TILING_AUTO) return VIT_ERR_INVALID_ARG;
  if (epilogue < 0 || epilogue > 2 || (epilogue == 2 && !residual)) return VIT_ERR_INVALID_ARG;
  if (misaligned(a) || misaligned(w) || misaligned(out) || misaligned(bias) || misaligned(residual))
    return VIT_ERR_INVALID_ARG;
  LinearArgs p{};
  p.M = M; p.N = N; p.K = K; p.a = a; p.lda = K; p.w = w; p.ldw = K; p.bias = bias;
  p.epilogue = epilogue; p.residual = residual; p.out = out; p.ldo = N;
  p.tiling = tiling;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dtype == VIT_BF16) {
    if (K % 8 || N % 8) return VIT_ERR_INVALID_ARG;
    VIT_LAUNCH(h, VIT_PROF_OP, launch_linear_tc(p, h->dev_status, s, &h->tmaps));
  } else if (dtype == VIT_FP32) {
    VIT_LAUNCH(h, VIT_PROF_OP, launch_linear_f32(p, s));
  } else {
    return VIT_ERR_INVALID_ARG;
  }
  return VIT_OK;
}

int vit_op_rowstats(vit_handle* h, int rows, int cols, const void* x, float eps, float* stats, void* stream) {
  if (!h || !x || !stats || rows < 0 || cols < 1 || cols % 8 || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (misaligned(x) || misaligned(stats)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  VIT_LAUNCH(h, VIT_PROF_LAYERNORM, launch_rowstats_bf16((const bf16*)x, eps, reinterpret_cast<float2*>(stats), rows, cols, s));
  return VIT_OK;
}

int vit_op_linear_ln(vit_handle* h, int M, int N, int K, const void* a, const float* stats, const void* wg,
                     const float* c1, const float* c0, int gelu, void* out, int tiling, void* stream) {
  if (!h || !a || !stats || !wg || !c1 || !c0 || !out || M < 0 || N < 1 || K < 1 || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (K % 8 || N % 8 || tiling < VIT_TILING_AUTO || tiling > VIT_TILING_PAIR_256x256) return VIT_ERR_INVALID_ARG;
  if (misaligned(a) || misaligned(stats) || misaligned(wg) || misaligned(c1) || misaligned(c0) || misaligned(out))
    return VIT_ERR_INVALID_ARG;
  LinearArgs p{};
  p.M = M; p.N = N; p.K = K; p.a = a; p.lda = K; p.w = wg; p.ldw = K; p.bias = c0;
  p.epilogue = gelu ? EPI_LN_BIAS_GELU : EPI_LN_BIAS;
  p.ln_stats = reinterpret_cast<const float2*>(stats); p.ln_c1 = c1; p.out = out; p.ldo = N; p.tiling = tiling;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  VIT_LAUNCH(h, VIT_PROF_OP, launch_linear_tc(p, h->dev_status, s, &h->tmaps));
  return VIT_OK;
}

int vit_op_attention(vit_handle* h, int dtype, int images, int T, int heads, int d, const void* qkv,
                     void* out, void* stream) {
  if (!h || !qkv || !out || images < 0 || T < 1 || T > 512 || heads < 1 || d < 1 || !on_own_device(h)) return VIT_ERR_INVALID_ARG;
  if (misaligned(qkv) || misaligned(out)) return VIT_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dtype == VIT_BF16) {
    if (d % 16 || d > 128) return VIT_ERR_INVALID_ARG;
    VIT_LAUNCH(h, VIT_PROF_ATTENTION, launch_attention_bf16((const bf16*)qkv, (bf16*)out, images, T, heads, d, h->dev_status, s, &h->tmaps));
  } else if (dtype == VIT_FP32) {
    VIT_LAUNCH(h, VIT_PROF_ATTENTION, launch_attention_f32((const float*)qkv, (float*)out, images, T, heads, d, s));
  } else {
    return VIT_ERR_INVALID_ARG;
  }
  return VIT_OK;
}

}  // extern "C"
