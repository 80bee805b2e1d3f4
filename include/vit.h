/*
 * vit.h — C boundary of the ViT pipeline-stage forward library for NVIDIA B200 (sm_100a).
 *
 * The library computes the forward pass of one pipeline stage: a contiguous range of layers
 * [layer_begin, layer_end) of a pre-LN Vision Transformer encoder applied to one microbatch of
 * activations, plus the two book-ends (patch embedding before the first stage, classification
 * head after the last) and a stage runner that issues microbatches on CUDA streams.
 *
 * Conventions for every entry point
 *   - All functions return an int status: VIT_OK (0) or a negative VIT_ERR_* code.  Arguments
 *     are validated on the host before anything is launched; a failed call launches nothing.
 *   - "dev" pointers are device memory owned by the caller (for example the data_ptr() of a
 *     PyTorch tensor) and must stay alive until the stream has drained.  They must be 16-byte
 *     aligned.  "host" pointers are ordinary (preferably pinned) host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls are
 *     asynchronous on that stream, allocate no device memory and never synchronise the host,
 *     except where stated (while vit_profile_enable is on, every launch also creates a pair of
 *     CUDA events).
 *   - A handle belongs to the CUDA device that was current in vit_create; every call that takes
 *     the handle must be made with that device current (otherwise VIT_ERR_INVALID_ARG).
 *   - Activations are row-major [microbatch, T, H] (T = patches + 1 class token, H = hidden).
 *     Their element type is the model's activation type: bf16 when config.dtype == VIT_BF16
 *     (bf16 operands, fp32 accumulation), fp32 when config.dtype == VIT_FP32.
 *   - A workspace must not be shared by two calls that may overlap on the GPU.
 *   - A handle may be used from several host threads at once with distinct streams and
 *     workspaces; parameters are read-only after vit_create.
 */
#ifndef VIT_B200_H
#define VIT_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  VIT_OK = 0,
  VIT_ERR_INVALID_ARG = -1, /* null or misaligned pointer, microbatch < 1 or > max_microbatch */
  VIT_ERR_RANGE = -2,       /* not 0 <= layer_begin < layer_end <= layers (empty range is an error) */
  VIT_ERR_CONFIG = -3,      /* inconsistent or unsupported model shape */
  VIT_ERR_WORKSPACE = -4,   /* workspace smaller than the size query says */
  VIT_ERR_CUDA = -5,        /* a CUDA runtime/driver call or a launch failed */
  VIT_ERR_TIMEOUT = -6,     /* a bounded wait inside a kernel gave up (device status word) */
  VIT_ERR_NO_DEVICE = -7,   /* no sm_100 device / driver available */
  VIT_ERR_TOO_LARGE = -8,   /* problem exceeds the fixed scratch of an allocation-free entry point,
                               or the partitioner's tables do not fit in host memory */
  VIT_ERR_INFEASIBLE = -9   /* the partitioner found no assignment that fits the devices' memory */
};

enum { VIT_BF16 = 0, VIT_FP32 = 1 };

typedef struct vit_config {
  int32_t image_size;     /* pixels per side, e.g. 224 */
  int32_t patch_size;     /* 16 or 14; must divide image_size */
  int32_t channels;       /* 3 */
  int32_t hidden;         /* H, multiple of 64 */
  int32_t layers;         /* L */
  int32_t heads;          /* H / heads must be a multiple of 16 and <= 128 */
  int32_t mlp_dim;        /* F, multiple of 64 */
  int32_t num_classes;
  float   ln_eps;         /* LayerNorm epsilon (inside the square root) */
  int32_t dtype;          /* VIT_BF16 or VIT_FP32 */
  int32_t max_microbatch; /* largest microbatch any call will use */
  int32_t extra_tokens;   /* 0, or 1 for a distillation token after the class token (see below) */
} vit_config;

typedef struct vit_handle vit_handle; /* opaque */

/* Number of fp32 values in the host parameter blob for this configuration (0 if the
 * configuration is invalid).  Blob layout, tensors back to back, matrices [out, in] row-major:
 *   patch.W [H, C*P*P] (column = c*P*P + i*P + j), patch.b [H], cls [H], (dist [H]), pos [T, H],
 *   per layer: ln1.g ln1.b Wqkv[3H,H] bqkv[3H] Wo[H,H] bo[H] ln2.g ln2.b W1[F,H] b1[F] W2[H,F] b2[H],
 *   lnf.g [H], lnf.b [H], head.W [classes, H], head.b [classes], (head_dist.W, head_dist.b).
 * The entries in parentheses exist when extra_tokens == 1: the compressed models of the paper's
 * Section 5.5 are distilled transformers with a distillation token; then T = patches + 2, token 1
 * is dist + pos[1], patch tokens start at 2, and the head averages two classifiers.
 * Wqkv rows [0,H) produce Q, [H,2H) K, [2H,3H) V; head h owns rows h*d..(h+1)*d of each. */
size_t vit_param_count(const vit_config* cfg);

/* Bytes of scratch one call of vit_patch_embed / vit_run_stage / vit_head needs for
 * `microbatch` images (the maximum over the three).  0 if arguments are invalid. */
size_t vit_workspace_bytes(const vit_config* cfg, int microbatch);

/* Bytes of scratch one stream of vit_run_pipeline[_host] needs for `microbatch` images:
 * the stage scratch above plus the token buffer and pixel/logit staging. */
size_t vit_pipeline_workspace_bytes(const vit_config* cfg, int microbatch);

/* Creates a model instance on the current CUDA device.
 * The transformer to partition is given to the system as a configuration plus its weights
 * (paper Section 3.1: the model configuration is the partitioner's input; Section 4: the
 * models are standard ViT definitions).
 *   host_params: host, fp32 blob in the layout above, n_params == vit_param_count(cfg).
 *     In bf16 mode matrices are rounded to bf16 (nearest even) on upload; vectors stay fp32.
 * Allocates device memory for the parameters (freed by vit_destroy), synchronises.
 * Errors: INVALID_ARG, CONFIG, NO_DEVICE, CUDA. */
int vit_create(const vit_config* cfg, const float* host_params, size_t n_params, vit_handle** out);

/* Frees the handle and the device memory it allocated.  Synchronises the device. */
int vit_destroy(vit_handle* h);

/* Embedding book-end (paper Section 4: inputs pass an embedding layer that gives them the
 * uniform dimension the transformer layers expect).
 *   pixels: dev, fp32 [microbatch, C, S, S] (NCHW).
 *   tokens_out: dev, activations [microbatch, T, H].  Token 1 + extra_tokens + py*(S/P) + px is
 *     patch.W . vec(patch(py,px)) + patch.b + pos[token]; token 0 is cls + pos[0] (and token 1
 *     dist + pos[1] when extra_tokens == 1).
 *   ws: dev scratch of at least vit_workspace_bytes(cfg, microbatch). */
int vit_patch_embed(vit_handle* h, int microbatch, const float* pixels, void* tokens_out,
                    void* ws, size_t ws_bytes, void* stream);

/* One pipeline stage T_i (paper Section 3.1: the model is split into parts T_1..T_k of
 * consecutive layers, the output of stage i is the input of stage i+1, and
 * Y = T_k(...T_1(X))).  Applies layers [layer_begin, layer_end) to `in`, writes `out`.
 * Each layer is x += Wo.attention(LN1(x).Wqkv^T + bqkv) + bo;  x += W2.gelu(W1.LN2(x) + b1) + b2
 * (Section 2.1: self-attention, MLP, two layer normalisations, residual connections).  In bf16
 * mode the two layer normalisations are applied inside the QKV and fc1 products (row statistics
 * from a small kernel, gain and shift folded into the weights at vit_create).
 *   in, out: dev, activations [microbatch, T, H]; in == out is allowed (in place), any other
 *     overlap is INVALID_ARG.
 * Running [a,b) then [b,c) gives bit-identical results to one call on [a,c). */
int vit_run_stage(vit_handle* h, int layer_begin, int layer_end, int microbatch,
                  const void* in, void* out, void* ws, size_t ws_bytes, void* stream);

/* Classification book-end (paper Section 3.1: the device of the final stage produces the
 * final result; Section 4: the task is image classification).  Final LayerNorm of each image's
 * class token, then logits = f . head.W^T + head.b.  With extra_tokens == 1 the distillation
 * token (row 1) goes through the same LayerNorm and the classifier head_dist, and the logits are
 * the mean of the two classifiers' outputs.
 *   tokens: dev, activations [microbatch, T, H];  logits: dev, fp32 [microbatch, classes]. */
int vit_head(vit_handle* h, int microbatch, const void* tokens, float* logits,
             void* ws, size_t ws_bytes, void* stream);

/* vit_head for callers that cannot allocate device memory.  (The paper has no counterpart; this
 * is a convenience of the library.)  Some code that wants the classification result runs where
 * cudaMalloc is off limits: a real-time loop that must never enter the allocator (it can block
 * and synchronise the device), a plugin whose host application owns all device memory and hands
 * out only the input and output buffers, or a process whose memory pool was given away whole to
 * another framework at start-up.  vit_head needs a scratch buffer for
 * the normalised class-token features; this variant keeps that scratch in an array that is part
 * of the library itself, so the caller passes only tokens and logits.
 *   - Same arithmetic and same results as vit_head.
 *   - Limit: microbatch * (1 + extra_tokens) * hidden <= VIT_HEAD_STATIC_MAX_FLOATS (2 MiB of floats); anything
 *     larger returns VIT_ERR_TOO_LARGE and launches nothing.  Every GPU on which the library
 *     is loaded carries the array (2 MiB) until the process exits.
 *   - The first call on each device looks up the array's device address (a runtime query, not
 *     an allocation); make that first call before starting any stream capture.  It must be
 *     made with the handle's device current, like every other call.
 *   - There is ONE array per device, shared by all handles and streams, and it keeps whatever
 *     the last call left in it.  Nothing in it has to be cleared: a call overwrites every value
 *     before reading it.  Two calls that may run on the GPU at the same time (different
 *     streams, no dependency between them) would overwrite each other's features: order them.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine. */
#define VIT_HEAD_STATIC_MAX_FLOATS (512 * 1024)
int vit_head_static(vit_handle* h, int microbatch, const void* tokens, float* logits, void* stream);

/* Stage runner (paper Section 2.1/3.1: the minibatch is split into equal microbatches that
 * flow through the stages in order).  Splits `batch` images into microbatches of `microbatch`
 * (the last may be smaller), and for microbatch m issues, on streams[m % n_streams]:
 * patch embed, every stage in order (stage s covers stage_layers[s] layers; the counts must
 * sum to L), head.  A microbatch never changes stream, so stream order carries the
 * stage-to-stage dependency; different microbatches overlap across streams.
 *   pixels: dev fp32 [batch, C, S, S];  logits: dev fp32 [batch, classes].
 *   ws_per_stream[i]: dev scratch of at least vit_pipeline_workspace_bytes(cfg, microbatch).
 * Does not synchronise; the caller waits on the streams. */
int vit_run_pipeline(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch,
                     int microbatch, const float* pixels, float* logits,
                     void* const* ws_per_stream, size_t ws_bytes, void* const* streams,
                     int n_streams);

/* vit_run_pipeline with `group` consecutive microbatches carried through every kernel launch
 * together (paper Section 5.4 studies the microbatch size: small microbatches keep the memory
 * per stage low but leave a large GPU underused; images are independent, so several of them in
 * flight can share a launch without changing any result).  Microbatch m still consists of images
 * [m * microbatch, (m + 1) * microbatch); groups go round-robin over the streams.
 *   ws_per_stream[i]: at least vit_pipeline_workspace_bytes(cfg, group * microbatch);
 *   group * microbatch <= max_microbatch. */
int vit_run_pipeline_grouped(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch,
                             int microbatch, int group, const float* pixels, float* logits,
                             void* const* ws_per_stream, size_t ws_bytes, void* const* streams,
                             int n_streams);

/* Same as vit_run_pipeline with HOST pixels and logits: each microbatch's pixels are copied to
 * the device, and its logits back, on that microbatch's stream (copies are asynchronous only
 * if the host memory is pinned).  Does not synchronise. */
int vit_run_pipeline_host(vit_handle* h, const int32_t* stage_layers, int n_stages, int batch,
                          int microbatch, const float* host_pixels, float* host_logits,
                          void* const* ws_per_stream, size_t ws_bytes, void* const* streams,
                          int n_streams);

/* Returns and clears the device status word after everything queued on `stream` has finished
 * (synchronises that stream): VIT_OK, or VIT_ERR_TIMEOUT if a bounded wait in a kernel gave up
 * since the last check, or VIT_ERR_CUDA if the stream reported an error.  There is one word per
 * handle, shared by all its streams; it is read and cleared in one atomic step on the device, so
 * a timeout raised on another stream while this call runs is reported by the next check.  To
 * know that a multi-stream run was clean, check after each of its streams. */
int vit_check_status(vit_handle* h, void* stream);

/* Failure-detection self-test.  Every wait inside the tensor-core kernels is bounded: when it
 * expires the kernel raises the device status word and returns.  This call launches a one-warp
 * kernel whose wait can never be satisfied, with a limit of `limit_cycles` SM cycles (at most
 * 2^31, about a second), so that the path can be exercised without a stuck kernel: afterwards
 * vit_check_status returns VIT_ERR_TIMEOUT once and the handle keeps working. */
int vit_debug_wait_probe(vit_handle* h, int64_t limit_cycles, void* stream);

/* Number of kernels this handle has launched so far (host counter). */
uint64_t vit_launch_count(const vit_handle* h);

const char* vit_status_string(int status);

/* Per-kernel timing.  While enabled, every kernel launch of this handle is bracketed by a pair
 * of CUDA events on the stream it is launched on.  vit_profile_collect synchronises the device,
 * adds the elapsed milliseconds and launch counts per class into the two arrays of
 * VIT_PROF_CLASSES entries, and clears the records.  Use from one host thread only. */
enum {
  VIT_PROF_LAYERNORM = 0, VIT_PROF_QKV = 1, VIT_PROF_ATTENTION = 2, VIT_PROF_OUTPROJ = 3,
  VIT_PROF_FC1 = 4, VIT_PROF_FC2 = 5, VIT_PROF_EMBED = 6, VIT_PROF_HEAD = 7, VIT_PROF_OP = 8,
  VIT_PROF_CLASSES = 9
};
int vit_profile_enable(vit_handle* h, int on);
int vit_profile_collect(vit_handle* h, double* ms_by_class, uint64_t* launches_by_class);

/* ---- pipeline partitioner (host only, no GPU work) -------------------------------------------
 * Chooses which consecutive layers run on which device so that the slowest pipeline stage is as
 * fast as possible (paper Section 3.3: Eq. 1 T_comm = P_j / b(u,v); Eq. 2 T_period = max(T_comp,
 * T_comm); Eq. 3 the transition of the three-dimensional dynamic programme over layers done,
 * devices used and next device; Algorithm 1 with its memory check and precursor table).
 * All pointers are host memory. */
typedef struct vit_partition_problem {
  int32_t layers;            /* L */
  int32_t devices;           /* D (at most 16), or the number of categories (at most 8) */
  const double* layer_time;  /* [D][L] seconds layer j takes on device u; T_comp of a layer range is the sum */
  const double* out_bytes;   /* [L] P_j: bytes a stage ending with layer j sends to the next stage */
  const double* layer_mem;   /* [L] M_j: memory layer j needs */
  const double* device_mem;  /* [D] m_u */
  const double* bandwidth;   /* [D][D] bytes per second from device u to device v */
} vit_partition_problem;

/* t_opt: the slowest stage's period; n_stages, stage_layers[s] (layer counts in pipeline order,
 * summing to L) and stage_device[s] (device of stage s) describe one optimal mapping.  The two
 * output arrays need min(L, D) entries.  Every device is used at most once; not all need be used.
 * Errors: INVALID_ARG (null pointer, D > 16, a bandwidth that is not positive, a time, size or
 * memory that is negative or not a number), INFEASIBLE, TOO_LARGE (the tables of the dynamic
 * programme, about 8 * L * 2^D * D bytes, could not be allocated). */
int vit_partition(const vit_partition_problem* problem, double* t_opt, int32_t* n_stages,
                  int32_t* stage_layers, int32_t* stage_device);

/* The same problem with identical devices grouped (paper Section 3.3, last paragraph): `devices`
 * is the number of categories, category_count[c] the number of devices in category c, and
 * layer_time / device_mem / bandwidth are indexed by category (bandwidth[c][c] = between two
 * devices of category c).  stage_device receives category indices.  The state space shrinks from
 * 2^D to prod(count + 1).  Output arrays need min(L, total devices) entries. */
int vit_partition_categories(const vit_partition_problem* problem, const int32_t* category_count,
                             double* t_opt, int32_t* n_stages, int32_t* stage_layers,
                             int32_t* stage_device);

/* ---- single operations, exposed so that each kernel can be checked on its own ------------
 * All pointers dev; `dtype` selects the bf16 or fp32 kernel family as in vit_config.
 * They need a handle only for the device status word and the launch counter. */

/* y[r,:] = (x[r,:] - mean) / sqrt(var + eps) * gain + shift, biased variance, rows x cols.
 * x, y: activations; gain, shift: fp32 [cols]. */
int vit_op_layernorm(vit_handle* h, int dtype, int rows, int cols, const void* x,
                     const float* gain, const float* shift, float eps, void* y, void* stream);

/* out = epilogue(a[M,K] . w[N,K]^T + bias[N]); a, w, out, residual in the activation type,
 * bias fp32.  epilogue: 0 = none, 1 = erf-GELU, 2 = add residual[M,N] (residual may equal out).
 * bf16 family: K % 8 == 0 and N % 8 == 0. */
int vit_op_linear(vit_handle* h, int dtype, int M, int N, int K, const void* a, const void* w,
                  const float* bias, int epilogue, const void* residual, void* out, void* stream);

/* vit_op_linear with the tiling of the bf16 tensor-core kernel chosen by the caller instead of
 * by the library's shape-only cost model, so that every tiling can be checked on any shape.
 * VIT_TILING_PAIR_256x256 runs CTA pairs on 256 x 256 tiles.  fp32 family: AUTO only. */
enum { VIT_TILING_AUTO = 0, VIT_TILING_128x128 = 1, VIT_TILING_128x256 = 2, VIT_TILING_PAIR_256x256 = 3 };
int vit_op_linear_tiled(vit_handle* h, int dtype, int M, int N, int K, const void* a, const void* w,
                        const float* bias, int epilogue, const void* residual, void* out, int tiling,
                        void* stream);

/* The two halves of the LayerNorm that vit_run_stage folds into its QKV and fc1 products in bf16
 * mode (the normalised activations are never written to memory):
 *   vit_op_rowstats: stats[2 r] = mean of row r of x (bf16 [rows, cols]), stats[2 r + 1] =
 *     1 / sqrt(biased variance + eps); stats is fp32 [rows, 2].
 *   vit_op_linear_ln: out[m,n] = f(stats[m].rstd * (a[m,:] . wg[n,:] - stats[m].mean * c1[n]) + c0[n]),
 *     f = identity or erf-GELU.  With wg[n,k] = gain[k] w[n,k], c1[n] = sum_k wg[n,k] and
 *     c0[n] = bias[n] + sum_k shift[k] w[n,k] this equals f(LayerNorm(a)[m,:] . w[n,:] + bias[n]).
 *     a, wg, out bf16; c1, c0 fp32 [N]; `tiling` as in vit_op_linear_tiled. */
int vit_op_rowstats(vit_handle* h, int rows, int cols, const void* x, float eps, float* stats, void* stream);
int vit_op_linear_ln(vit_handle* h, int M, int N, int K, const void* a, const float* stats, const void* wg,
                     const float* c1, const float* c0, int gelu, void* out, int tiling, void* stream);

/* Multi-head self-attention for `images` sequences of T tokens: qkv [images*T, 3*heads*d]
 * (column blocks Q, K, V; head-major inside each), out [images*T, heads*d];
 * out_h = softmax_rows(Q_h K_h^T / sqrt(d)) V_h. */
int vit_op_attention(vit_handle* h, int dtype, int images, int T, int heads, int d,
                     const void* qkv, void* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VIT_B200_H */
