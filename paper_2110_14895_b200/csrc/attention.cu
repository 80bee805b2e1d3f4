// Fused multi-head self-attention for short sequences (T <= 512), bf16 in / bf16 out.
//
// One CTA per (image, head).  K and V of the head are staged once in shared memory; every warp
// owns 16-query tiles and walks the keys in chunks of 32 with an online softmax, so the score
// matrix only ever exists as 16 x 32 register fragments.  QK^T and PV run on the tensor cores
// through warp-level mma (m16n8k16, bf16 operands, fp32 accumulation); row statistics, the
// exponentials and the final normalisation are fp32.  P is rounded to bf16 before PV.
#include "vit_internal.h"

namespace vit {

namespace {

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
      "{%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <int D, int NT, int MINB>
__global__ void __launch_bounds__(NT, MINB)
attention_bf16_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out, int T, int heads) {
  constexpr int LD = D + 8;            // padded row (elements): keeps ldmatrix conflict-free
  constexpr int KS = D / 16;           // k-steps of QK^T
  constexpr int DN = D / 8;            // n-tiles of PV
  extern __shared__ __align__(16) uint8_t smem_raw[];
  bf16* Ks = reinterpret_cast<bf16*>(smem_raw);
  const int Tp = (T + 31) & ~31;
  bf16* Vs = Ks + (size_t)Tp * LD;

  const int img = blockIdx.x / heads, hd = blockIdx.x % heads;
  const int H = heads * D;
  const size_t ld = (size_t)3 * H;
  const bf16* base = qkv + (size_t)img * T * ld + (size_t)hd * D;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;

  // stage K and V (16-byte chunks), zero the padded rows
  constexpr int CPR = D / 8;           // chunks per row
  for (int i = threadIdx.x; i < Tp * CPR; i += blockDim.x) {
    const int t = i / CPR, c = i % CPR;
    uint4 k = make_uint4(0, 0, 0, 0), v = make_uint4(0, 0, 0, 0);
    if (t < T) {
      k = __ldg(reinterpret_cast<const uint4*>(base + (size_t)t * ld + H) + c);
      v = __ldg(reinterpret_cast<const uint4*>(base + (size_t)t * ld + 2 * H) + c);
    }
    *reinterpret_cast<uint4*>(Ks + (size_t)t * LD + c * 8) = k;
    *reinterpret_cast<uint4*>(Vs + (size_t)t * LD + c * 8) = v;
  }
  __syncthreads();

  const int g = lane >> 2, tq = lane & 3;
  const float sl2 = 1.4426950408889634f / sqrtf((float)D);   // log2(e) / sqrt(d)
  const uint32_t ks_base = (uint32_t)__cvta_generic_to_shared(Ks);
  const uint32_t vs_base = (uint32_t)__cvta_generic_to_shared(Vs);
  const int mi = lane >> 3, mr = lane & 7;                   // ldmatrix: matrix index, row in it
  const int ntiles = (T + 15) / 16;

  for (int tile = warp; tile < ntiles; tile += nwarps) {
    const int r0 = tile * 16;
    const int rowA = r0 + g, rowB = r0 + g + 8;
    // Q fragments straight from global memory
    uint32_t qf[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int c = ks * 16 + 2 * tq;
      qf[ks][0] = rowA < T ? __ldg(reinterpret_cast<const uint32_t*>(base + (size_t)rowA * ld + c)) : 0u;
      qf[ks][1] = rowB < T ? __ldg(reinterpret_cast<const uint32_t*>(base + (size_t)rowB * ld + c)) : 0u;
      qf[ks][2] = rowA < T ? __ldg(reinterpret_cast<const uint32_t*>(base + (size_t)rowA * ld + c + 8)) : 0u;
      qf[ks][3] = rowB < T ? __ldg(reinterpret_cast<const uint32_t*>(base + (size_t)rowB * ld + c + 8)) : 0u;
    }
    float o[DN][4];
#pragma unroll
    for (int n = 0; n < DN; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;

    for (int k0 = 0; k0 < Tp; k0 += 32) {
      float s[4][4];
#pragma unroll
      for (int n = 0; n < 4; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
        for (int np = 0; np < 2; ++np) {       // pairs of 8-key tiles
          uint32_t b[4];
          const int key = k0 + np * 16 + (mi >> 1) * 8 + mr;
          const int col = ks * 16 + (mi & 1) * 8;
          ldmatrix_x4(b, ks_base + (uint32_t)((key * LD + col) * 2));
          mma_bf16(s[2 * np], qf[ks], b[0], b[1]);
          mma_bf16(s[2 * np + 1], qf[ks], b[2], b[3]);
        }
      }
      // mask keys beyond T (only the last chunk can have any)
      if (k0 + 32 > T) {
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          const int key = k0 + n * 8 + 2 * tq;
          if (key >= T) { s[n][0] = -INFINITY; s[n][2] = -INFINITY; }
          if (key + 1 >= T) { s[n][1] = -INFINITY; s[n][3] = -INFINITY; }
        }
      }
      float cA = -INFINITY, cB = -INFINITY;
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        cA = fmaxf(cA, fmaxf(s[n][0], s[n][1]));
        cB = fmaxf(cB, fmaxf(s[n][2], s[n][3]));
      }
      cA = fmaxf(cA, __shfl_xor_sync(0xffffffffu, cA, 1));
      cA = fmaxf(cA, __shfl_xor_sync(0xffffffffu, cA, 2));
      cB = fmaxf(cB, __shfl_xor_sync(0xffffffffu, cB, 1));
      cB = fmaxf(cB, __shfl_xor_sync(0xffffffffu, cB, 2));
      const float nmA = fmaxf(mA, cA), nmB = fmaxf(mB, cB);    // finite: every chunk has a valid key
      const float fA = exp2f((mA - nmA) * sl2), fB = exp2f((mB - nmB) * sl2);
      mA = nmA; mB = nmB;
      float sA = 0.f, sB = 0.f;
      uint32_t pf[2][4];
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const float p0 = exp2f((s[n][0] - mA) * sl2), p1 = exp2f((s[n][1] - mA) * sl2);
        const float p2 = exp2f((s[n][2] - mB) * sl2), p3 = exp2f((s[n][3] - mB) * sl2);
        sA += p0 + p1;
        sB += p2 + p3;
        pf[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      lA = lA * fA + sA;
      lB = lB * fB + sB;
#pragma unroll
      for (int n = 0; n < DN; ++n) {
        o[n][0] *= fA; o[n][1] *= fA; o[n][2] *= fB; o[n][3] *= fB;
      }
#pragma unroll
      for (int kk = 0; kk < 2; ++kk) {         // two 16-key steps of PV
#pragma unroll
        for (int dn = 0; dn < DN; dn += 2) {
          uint32_t b[4];
          const int key = k0 + kk * 16 + (mi & 1) * 8 + mr;
          const int col = (dn + (mi >> 1)) * 8;
          ldmatrix_x4_trans(b, vs_base + (uint32_t)((key * LD + col) * 2));
          mma_bf16(o[dn], pf[kk], b[0], b[1]);
          mma_bf16(o[dn + 1], pf[kk], b[2], b[3]);
        }
      }
    }
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    const float iA = 1.0f / lA, iB = 1.0f / lB;
    bf16* oA = out + ((size_t)img * T + rowA) * H + (size_t)hd * D + 2 * tq;
    bf16* oB = out + ((size_t)img * T + rowB) * H + (size_t)hd * D + 2 * tq;
#pragma unroll
    for (int n = 0; n < DN; ++n) {
      if (rowA < T) *reinterpret_cast<uint32_t*>(oA + n * 8) = pack_bf16(o[n][0] * iA, o[n][1] * iA);
      if (rowB < T) *reinterpret_cast<uint32_t*>(oB + n * 8) = pack_bf16(o[n][2] * iB, o[n][3] * iB);
    }
  }
}

template <int D, int NT, int MINB>
cudaError_t launch_variant(const bf16* qkv, bf16* out, int images, int T, int heads, int nw, size_t smem,
                           cudaStream_t s) {
  static PerDeviceFlag configured;
  cudaError_t e = ensure_dynamic_smem(configured, attention_bf16_kernel<D, NT, MINB>, 227 * 1024);
  if (e != cudaSuccess) return e;
  attention_bf16_kernel<D, NT, MINB><<<images * heads, nw * 32, smem, s>>>(qkv, out, T, heads);
  return cudaGetLastError();
}

template <int D>
cudaError_t launch_d(const bf16* qkv, bf16* out, int images, int T, int heads, cudaStream_t s) {
  const int Tp = (T + 31) & ~31;
  const size_t smem = (size_t)2 * Tp * (D + 8) * sizeof(bf16);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  const int ntiles = (T + 15) / 16;
  int nw = (ntiles + 1) / 2;
  if (nw < 1) nw = 1;
  if (nw > 16) nw = 16;
  // up to 9 warps: registers capped so that two CTAs share an SM
  if (nw <= 9) return launch_variant<D, 288, 2>(qkv, out, images, T, heads, nw, smem, s);
  return launch_variant<D, 512, 1>(qkv, out, images, T, heads, nw, smem, s);
}

}  // namespace

cudaError_t launch_attention_bf16(const bf16* qkv, bf16* out, int images, int T, int heads, int d,
                                  int* dev_status, cudaStream_t s, TensorMapCache* cache) {
  if (images <= 0) return cudaSuccess;
  if (attention_tc_supported(T, d)) return launch_attention_tc(qkv, out, images, T, heads, d, dev_status, s, cache);
  switch (d) {
    case 16: return launch_d<16>(qkv, out, images, T, heads, s);
    case 32: return launch_d<32>(qkv, out, images, T, heads, s);
    case 48: return launch_d<48>(qkv, out, images, T, heads, s);
    case 64: return launch_d<64>(qkv, out, images, T, heads, s);
    case 80: return launch_d<80>(qkv, out, images, T, heads, s);
    case 96: return launch_d<96>(qkv, out, images, T, heads, s);
    case 112: return launch_d<112>(qkv, out, images, T, heads, s);
    case 128: return launch_d<128>(qkv, out, images, T, heads, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace vit
