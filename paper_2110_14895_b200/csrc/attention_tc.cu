// Fused multi-head self-attention on the 5th-generation tensor cores, for the sequence lengths
// of ViT (T = 197 or 257 tokens; any T in [193,208] or [241,260]) and head sizes 64 and 80.
//
// One CTA per (image, head), two CTAs per SM.  K, V and one 128-query tile of Q are brought into
// shared memory by TMA: columns [0,64) of the head as 128-byte-swizzled rows, columns [64,80)
// (d = 80 only) as 32-byte-swizzled rows.  The same tiles serve as K-major operands (Q, K in
// S = Q K^T) and as the N-major operand (V in O = P V).  Per query tile:
//   S = Q K^T        tcgen05.mma, 128 x NK x d, accumulator in tensor memory (NK fp32 columns)
//   softmax          8 warps, two threads per query row (each half of the keys): row max, exp2,
//                    row sum, halves combined through shared memory; P is written back over S
//                    as packed bf16 (tcgen05.st), so scores never leave the SM
//   O = P V          tcgen05.mma with A = P from tensor memory, B = V from shared memory (for
//                    d = 80, V is held as five 32-byte-swizzled blocks of 16 columns)
//   epilogue         O / rowsum -> bf16 -> global
// Keys beyond NK = 256 (the 257th token) are handled by the row's thread with plain FMAs on
// copies of those K/V rows in shared memory.
// Warps: 0-7 softmax/epilogue (warp w reads tensor-memory lanes 32 (w % 4) ...), 8 = TMA + MMA
// issue + tensor-memory allocation.
// The two resident CTAs overlap one's softmax with the other's loads and MMAs.
// Every mbarrier wait is bounded; on expiry the CTA raises the device status word and leaves.
#include "vit_internal.h"
#include "sm100_ptx.cuh"

#include <cuda.h>

namespace vit {

namespace {

using namespace ptx;

constexpr int QT = 128;          // queries per tile = tensor-memory lanes
constexpr int MAX_EXTRA = 4;     // keys beyond NK handled without the tensor cores
constexpr int SOFTMAX_THREADS = 8 * 32;
constexpr int NUM_THREADS = SOFTMAX_THREADS + 32;
constexpr int MMA_WARP = 8;
constexpr uint32_t TMEM_COLS = 256;

// Shared-memory matrix descriptors for TMA-written tiles whose rows are one swizzle span wide
// (128 or 32 bytes); groups of 8 rows are 8 spans apart.  The same descriptor form serves a
// K-major operand (rows = M/N index) and an N-major operand (rows = K index).
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t make_desc_sw32(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(256 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)6 << 61);
}
// N-major operand made of several 32-byte-wide swizzled column blocks `lbo` bytes apart
__device__ __forceinline__ uint64_t make_desc_sw32_blocks(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)(256 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)6 << 61);
}
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool b_n_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_n_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(QT >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 u;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "r"(a));
  return u;
}
__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
  const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* bh = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 x = __bfloat1622float2(ah[j]), y = __bfloat1622float2(bh[j]);
    acc = fmaf(x.x, y.x, acc);
    acc = fmaf(x.y, y.y, acc);
  }
  return acc;
}

struct AttnMaps { CUtensorMap q64, q16, kv64, kv16; };

// Tensor-memory columns (256 per CTA).  S occupies [0, NK).  The two threads of a row each own
// half of the keys and overwrite S with P (bf16 pairs) only inside columns they have already
// consumed themselves: half 0 walks its 32-key chunks upwards and packs P from column 0; half 1
// walks its chunks downwards and packs P downwards from column NK.  O sits in between.
template <int NK>
struct TmemMap {
  static constexpr int SPLIT = (NK / 64) * 32;              // keys [0, SPLIT) -> half 0, [SPLIT, NK) -> half 1
  static constexpr int END1 = SPLIT + ((NK - SPLIT + 31) / 32) * 32;   // end of half 1's last (maybe partial) chunk
  static constexpr uint32_t O_COL = SPLIT / 2;
  // first P column of the 32-key chunk that starts at key c0
  __host__ __device__ static constexpr uint32_t p_col(int c0) {
    return c0 < SPLIT ? (uint32_t)(c0 / 2) : (uint32_t)(NK - 16 * ((END1 - 32 - c0) / 32 + 1));
  }
  // P columns of the 16 keys of MMA step ks
  __host__ __device__ static constexpr uint32_t p_col_step(int ks) {
    return 16 * ks < SPLIT ? (uint32_t)(8 * ks)
                           : p_col(SPLIT + ((16 * ks - SPLIT) / 32) * 32) + (uint32_t)((((16 * ks - SPLIT) / 16) % 2) * 8);
  }
};

template <int D, int NK>
struct Smem {
  static constexpr bool TAIL = D > 64;                 // columns [64, D) live in the 32-byte part
  static constexpr uint32_t KA = NK * 128, QA = QT * 128;
  static constexpr uint32_t KB = TAIL ? NK * 32 : 0, QB = TAIL ? QT * 32 : 0;
  static constexpr uint32_t VBYTES = NK * D * 2;       // D = 64: one 128-byte-swizzled tile;
                                                       // D = 80: five 32-byte-swizzled 16-column blocks
  static constexpr uint32_t OFF_KA = 0, OFF_QA = KA, OFF_V = KA + QA;
  static constexpr uint32_t OFF_KB = OFF_V + VBYTES, OFF_QB = OFF_KB + KB;
  static constexpr uint32_t OFF_XK = OFF_QB + QB;      // extra K rows, plain [MAX_EXTRA][D]
  static constexpr uint32_t OFF_XV = OFF_XK + MAX_EXTRA * D * 2;
  static constexpr uint32_t OFF_RED = OFF_XV + MAX_EXTRA * D * 2;   // float [2 halves][QT] row max, then [2][QT] row sum
  static constexpr uint32_t OFF_SX = OFF_RED + 4 * QT * 4;          // float [2 tiles][MAX_EXTRA][QT] extra-key scores
  static constexpr uint32_t OFF_BARS = OFF_SX + 2 * MAX_EXTRA * QT * 4;
  static constexpr uint32_t BYTES = OFF_BARS + 128 + 1024 /*alignment slack*/;
  static constexpr uint32_t KV_TX = KA + KB + VBYTES, Q_TX = QA + QB;
};

template <int D, int NK>
__global__ void __launch_bounds__(NUM_THREADS, 2)
attention_tc_kernel(const __grid_constant__ AttnMaps maps, const bf16* __restrict__ qkv,
                    bf16* __restrict__ out, int T, int heads, int* dev_status) {
  using L = Smem<D, NK>;
  constexpr int CH = D / 8;                      // 16-byte chunks per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
  const uint32_t kv_full = smem_u32(&bars[0]);   // K, V landed                 (TMA bytes)
  const uint32_t q_full = smem_u32(&bars[1]);    // Q tile landed               (TMA bytes)
  const uint32_t s_ready = smem_u32(&bars[2]);   // S complete in tensor memory (MMA commit)
  const uint32_t p_ready = smem_u32(&bars[3]);   // P written                   (256 arrivals)
  const uint32_t o_ready = smem_u32(&bars[4]);   // O complete                  (MMA commit)
  const uint32_t t_free = smem_u32(&bars[5]);    // O read, tensor memory free  (256 arrivals)
  const uint32_t q_read = smem_u32(&bars[6]);    // Q rows read by their threads (128 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[7]);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int img = blockIdx.x / heads, hd = blockIdx.x % heads;
  const int H = heads * D;
  const size_t ld = (size_t)3 * H;
  const bf16* base = qkv + (size_t)img * T * ld + (size_t)hd * D;   // Q of token 0 of this head
  const int ntiles = (T + QT - 1) / QT;
  const int n_extra = T > NK ? T - NK : 0;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(kv_full, 1);
    mbar_init(q_full, 1);
    mbar_init(s_ready, 1);
    mbar_init(p_ready, SOFTMAX_THREADS);
    mbar_init(o_ready, 1);
    mbar_init(t_free, SOFTMAX_THREADS);
    mbar_init(q_read, QT);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == MMA_WARP) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  grid_dependency_wait();               // barrier set-up and allocation overlap the previous kernel's tail
  grid_launch_dependents();
  // copies of the K and V rows of the keys beyond NK, as plain rows
  for (int i = threadIdx.x; i < n_extra * CH * 2; i += NUM_THREADS) {
    const int which = i / (n_extra * CH), j = i % (n_extra * CH), e = j / CH, c = j % CH;
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (size_t)(NK + e) * ld + (which + 1) * H) + c);
    *reinterpret_cast<uint4*>(smem + (which ? L::OFF_XV : L::OFF_XK) + (e * CH + c) * 16) = v;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == MMA_WARP) {
    // ------------------------------------------------------------------ TMA + MMA issuer
    if (lane == 0) {
      const int row_g = img * T;                 // global row of token 0
      const int col_q = hd * D, col_k = H + hd * D, col_v = 2 * H + hd * D;
      mbar_arrive_expect_tx(kv_full, L::KV_TX);
      tma_load_2d(sb + L::OFF_KA, &maps.kv64, col_k, row_g, kv_full);
      if (L::TAIL) {
        tma_load_2d(sb + L::OFF_KB, &maps.kv16, col_k + 64, row_g, kv_full);
#pragma unroll
        for (int a = 0; a < D / 16; ++a)
          tma_load_2d(sb + L::OFF_V + (uint32_t)(a * NK * 32), &maps.kv16, col_v + 16 * a, row_g, kv_full);
      } else {
        tma_load_2d(sb + L::OFF_V, &maps.kv64, col_v, row_g, kv_full);
      }
      mbar_arrive_expect_tx(q_full, L::Q_TX);
      tma_load_2d(sb + L::OFF_QA, &maps.q64, col_q, row_g, q_full);
      if (L::TAIL) tma_load_2d(sb + L::OFF_QB, &maps.q16, col_q + 64, row_g, q_full);

      bool ok = mbar_wait(kv_full, 0, abort_flag);
      for (int t = 0; t < ntiles && ok; ++t) {
        const uint32_t ph = (uint32_t)(t & 1);
        if (!mbar_wait(q_full, ph, abort_flag)) break;
        if (t > 0 && !mbar_wait(t_free, ph ^ 1, abort_flag)) break;
        tc_fence_after();
        // S = Q K^T: 16 columns of the head per step, 32 bytes further along the swizzled row
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(tmem_base, make_desc_sw128(sb + L::OFF_QA) + (uint64_t)(2 * k),
                    make_desc_sw128(sb + L::OFF_KA) + (uint64_t)(2 * k), idesc_bf16(NK, false), k > 0 ? 1u : 0u);
        if (L::TAIL)
          umma_bf16(tmem_base, make_desc_sw32(sb + L::OFF_QB), make_desc_sw32(sb + L::OFF_KB),
                    idesc_bf16(NK, false), 1u);
        umma_commit(s_ready);
        if (t + 1 < ntiles) {
          // next Q tile: the buffer is free once these MMAs have read it (and, when rows are
          // also read by their threads for the extra keys, once they have)
          if (!mbar_wait(s_ready, ph, abort_flag)) break;
          if (n_extra > 0 && !mbar_wait(q_read, ph, abort_flag)) break;
          mbar_arrive_expect_tx(q_full, L::Q_TX);
          tma_load_2d(sb + L::OFF_QA, &maps.q64, col_q, row_g + (t + 1) * QT, q_full);
          if (L::TAIL) tma_load_2d(sb + L::OFF_QB, &maps.q16, col_q + 64, row_g + (t + 1) * QT, q_full);
        }
        if (!mbar_wait(p_ready, ph, abort_flag)) break;
        tc_fence_after();
        // O = P V: A = P in tensor memory (8 columns per 16 keys); B = V, 16 keys per step =
        // two 8-row groups of the tile
#pragma unroll
        for (int k = 0; k < NK / 16; ++k) {
          const uint64_t bdesc = L::TAIL ? make_desc_sw32_blocks(sb + L::OFF_V + (uint32_t)(k * 512), NK * 32)
                                         : make_desc_sw128(sb + L::OFF_V + (uint32_t)(k * 2048));
          umma_bf16_ts(tmem_base + TmemMap<NK>::O_COL, tmem_base + TmemMap<NK>::p_col_step(k), bdesc,
                       idesc_bf16(D, true), k > 0 ? 1u : 0u);
        }
        umma_commit(o_ready);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;                    // tensor-memory lane = query row of the tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = 1.4426950408889634f / sqrtf((float)D);   // log2(e) / sqrt(d)
    using TM = TmemMap<NK>;
    constexpr int SPLIT = TM::SPLIT;
    constexpr uint32_t O_COL = TM::O_COL;
    const int k_begin = half ? SPLIT : 0, k_end = half ? NK : SPLIT;
    float* red = reinterpret_cast<float*>(smem + L::OFF_RED);     // [0..1][QT] max, [2..3][QT] sum
    float* sx = reinterpret_cast<float*>(smem + L::OFF_SX);       // [tile & 1][MAX_EXTRA][QT]
    auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(1 + quarter) : "memory"); };
    bool ok = true;

    // Scores of the keys beyond NK for tile `tt` (half 0 only), by hand: the row of Q is read back
    // from the swizzled tile, the K rows are plain copies.  Results go to shared memory for both
    // halves; arrives on q_read.
    auto extra_scores = [&](int tt) -> bool {
      if (n_extra == 0 || half != 0) return true;
      if (!mbar_wait(q_full, (uint32_t)(tt & 1), abort_flag)) return false;
      if (tt * QT + quarter * 32 < T) {
        uint4 q[CH];
#pragma unroll
        for (int c = 0; c < 8; ++c) q[c] = lds128(sb + L::OFF_QA + (uint32_t)(row * 128 + ((c ^ (row & 7)) << 4)));
#pragma unroll
        for (int c = 8; c < CH; ++c)
          q[c] = lds128(sb + L::OFF_QB + (uint32_t)(row * 32 + (((c - 8) ^ ((row >> 2) & 1)) << 4)));
#pragma unroll
        for (int e = 0; e < MAX_EXTRA; ++e) {
          if (e < n_extra) {
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < CH; ++c) acc = dot8(q[c], lds128(sb + L::OFF_XK + (uint32_t)((e * CH + c) * 16)), acc);
            sx[((tt & 1) * MAX_EXTRA + e) * QT + row] = acc;
          }
        }
      }
      mbar_arrive(q_read);
      return true;
    };
    ok = extra_scores(0);

    for (int t = 0; t < ntiles && ok; ++t) {
      const uint32_t ph = (uint32_t)(t & 1);
      const bool warp_active = t * QT + quarter * 32 < T;   // any valid row in this warp
      const float* sxt = sx + (t & 1) * MAX_EXTRA * QT;
      if (!mbar_wait(s_ready, ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      float msl = 0.f;
      if (warp_active) {
        // pass 1: maximum over this half's keys
        float m = -INFINITY;
        if (half == 0) {
#pragma unroll
          for (int e = 0; e < MAX_EXTRA; ++e)
            if (e < n_extra) m = fmaxf(m, sxt[e * QT + row]);
        }
#pragma unroll 1
        for (int c0 = k_begin; c0 < k_end; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(lane_addr + (uint32_t)c0, r);      // the last chunk may run past NK: masked below
          tmem_ld_wait();
          if (c0 + 32 <= T && c0 + 32 <= NK) {
            float m2[2] = {m, m};
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              asm("max.f32 %0, %0, %1, %2;" : "+f"(m2[0]) : "f"(__uint_as_float(r[j])), "f"(__uint_as_float(r[j + 1])));
              asm("max.f32 %0, %0, %1, %2;" : "+f"(m2[1]) : "f"(__uint_as_float(r[j + 2])), "f"(__uint_as_float(r[j + 3])));
            }
            m = fmaxf(m2[0], m2[1]);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c0 + j < T && c0 + j < NK) m = fmaxf(m, __uint_as_float(r[j]));
          }
        }
        red[half * QT + row] = m;
      }
      pair_sync();
      float l = 0.f;
      if (warp_active) {
        msl = fmaxf(red[row], red[QT + row]) * sl2;
        // pass 2: p = exp2((s - m) * sl2), partial row sum, P (bf16) back into tensor memory
        // (half 0 upwards, half 1 downwards: see TmemMap)
        const int nchunks = (k_end - k_begin + 31) / 32;
#pragma unroll 1
        for (int i = 0; i < nchunks; ++i) {
          const int c0 = half ? k_begin + 32 * (nchunks - 1 - i) : k_begin + 32 * i;
          uint32_t r[32];
          tmem_ld32(lane_addr + (uint32_t)c0, r);
          tmem_ld_wait();
          uint32_t pk[16];
          if (c0 + 32 <= T && c0 + 32 <= NK) {
            float l2[2] = {0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(r[2 * j]), sl2, -msl));
              const float p1 = ex2_approx(fmaf(__uint_as_float(r[2 * j + 1]), sl2, -msl));
              l2[0] += p0;
              l2[1] += p1;
              pk[j] = pack_bf16(p0, p1);
            }
            l += l2[0] + l2[1];
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int k0 = c0 + 2 * j;
              const float p0 = (k0 < T && k0 < NK) ? ex2_approx(fmaf(__uint_as_float(r[2 * j]), sl2, -msl)) : 0.f;
              const float p1 = (k0 + 1 < T && k0 + 1 < NK) ? ex2_approx(fmaf(__uint_as_float(r[2 * j + 1]), sl2, -msl)) : 0.f;
              l += p0 + p1;
              pk[j] = pack_bf16(p0, p1);
            }
          }
          tmem_st16(lane_addr + TM::p_col(c0), pk);
        }
        red[(2 + half) * QT + row] = l;
        tmem_st_wait();
      }
      tc_fence_before();
      mbar_arrive(p_ready);
      // while the tensor core runs P V: the extra keys' scores of the next tile
      if (t + 1 < ntiles && !extra_scores(t + 1)) { ok = false; break; }
      // epilogue: O (+ the hand-computed keys' share) / l -> bf16 -> global; this half's columns
      if (!mbar_wait(o_ready, ph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      pair_sync();                                          // both partial sums are in shared memory
      constexpr int G0 = (D / 16 + 1) / 2;                  // 16-column groups [0, G0) -> half 0, the rest -> half 1
      const int g_begin = half ? G0 : 0, g_end = half ? D / 16 : G0;
      uint32_t oreg[G0 * 16];
      if (warp_active) {
#pragma unroll
        for (int g = 0; g < G0; ++g)
          if (g_begin + g < g_end)
            tmem_ld16(lane_addr + O_COL + (uint32_t)((g_begin + g) * 16), *reinterpret_cast<uint32_t(*)[16]>(&oreg[g * 16]));
        tmem_ld_wait();
      }
      tc_fence_before();
      mbar_arrive(t_free);               // the next tile's S may overwrite tensor memory now
      const int tok = t * QT + row;
      if (warp_active && tok < T) {
        l = red[2 * QT + row] + red[3 * QT + row];
        float p_ex[MAX_EXTRA];
#pragma unroll
        for (int e = 0; e < MAX_EXTRA; ++e) {
          p_ex[e] = e < n_extra ? ex2_approx(fmaf(sxt[e * QT + row], sl2, -msl)) : 0.f;
          l += p_ex[e];
        }
        const float inv = 1.0f / l;
        uint4* orow = reinterpret_cast<uint4*>(out + ((size_t)img * T + tok) * H + (size_t)hd * D);
#pragma unroll
        for (int g = 0; g < G0; ++g) {
          if (g_begin + g < g_end) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int c = (g_begin + g) * 2 + q;         // 16-byte chunk of the row
              float o[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) o[j] = __uint_as_float(oreg[g * 16 + q * 8 + j]);
              if (n_extra > 0) {
#pragma unroll
                for (int e = 0; e < MAX_EXTRA; ++e) {
                  if (e < n_extra) {
                    const uint4 va = lds128(sb + L::OFF_XV + (uint32_t)((e * CH + c) * 16));
                    const __nv_bfloat162* vh = reinterpret_cast<const __nv_bfloat162*>(&va);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                      const float2 v2 = __bfloat1622float2(vh[j]);
                      o[2 * j] = fmaf(p_ex[e], v2.x, o[2 * j]);
                      o[2 * j + 1] = fmaf(p_ex[e], v2.y, o[2 * j + 1]);
                    }
                  }
                }
              }
              uint4 w;
              w.x = pack_bf16(o[0] * inv, o[1] * inv);
              w.y = pack_bf16(o[2] * inv, o[3] * inv);
              w.z = pack_bf16(o[4] * inv, o[5] * inv);
              w.w = pack_bf16(o[6] * inv, o[7] * inv);
              orow[c] = w;
            }
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  if (*abort_flag) __nanosleep(200000);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(dev_status, (int)VIT_ERR_TIMEOUT);
  if (warp == MMA_WARP) {
    __syncwarp();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

bool encode_map(CUtensorMap* tm, const void* base, size_t rows, size_t cols, int box_cols, int box_rows,
                CUtensorMapSwizzle sw) {
  const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int NK>
cudaError_t launch_variant(const bf16* qkv, bf16* out, int images, int T, int heads, int* dev_status,
                           cudaStream_t s) {
  using L = Smem<D, NK>;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
      return cudaErrorNotReady;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  static PerDeviceFlag configured;
  cudaError_t e = ensure_dynamic_smem(configured, attention_tc_kernel<D, NK>, (int)L::BYTES);
  if (e != cudaSuccess) return e;
  const size_t rows = (size_t)images * T, cols = (size_t)3 * heads * D;
  AttnMaps m;
  if (!encode_map(&m.q64, qkv, rows, cols, 64, QT, CU_TENSOR_MAP_SWIZZLE_128B)) return cudaErrorInvalidValue;
  if (!encode_map(&m.kv64, qkv, rows, cols, 64, NK, CU_TENSOR_MAP_SWIZZLE_128B)) return cudaErrorInvalidValue;
  if (D > 64) {
    if (!encode_map(&m.q16, qkv, rows, cols, D - 64, QT, CU_TENSOR_MAP_SWIZZLE_32B)) return cudaErrorInvalidValue;
    if (!encode_map(&m.kv16, qkv, rows, cols, D - 64, NK, CU_TENSOR_MAP_SWIZZLE_32B)) return cudaErrorInvalidValue;
  } else {
    m.q16 = m.q64;
    m.kv16 = m.kv64;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(images * heads));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = L::BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_tc_kernel<D, NK>, m, qkv, out, T, heads, dev_status);
}

}  // namespace

bool attention_tc_supported(int T, int d) {
  if (d != 64 && d != 80) return false;
  return (T >= 193 && T <= 208) || (T >= 241 && T <= 256 + MAX_EXTRA);
}

cudaError_t launch_attention_tc(const bf16* qkv, bf16* out, int images, int T, int heads, int d,
                                int* dev_status, cudaStream_t s) {
  if (images <= 0) return cudaSuccess;
  if (!attention_tc_supported(T, d)) return cudaErrorInvalidValue;
  const bool wide = T > 208;
  if (d == 64) return wide ? launch_variant<64, 256>(qkv, out, images, T, heads, dev_status, s)
                           : launch_variant<64, 208>(qkv, out, images, T, heads, dev_status, s);
  return wide ? launch_variant<80, 256>(qkv, out, images, T, heads, dev_status, s)
              : launch_variant<80, 208>(qkv, out, images, T, heads, dev_status, s);
}

}  // namespace vit
