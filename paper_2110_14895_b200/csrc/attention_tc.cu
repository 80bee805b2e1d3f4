// Fused multi-head self-attention on the 5th-generation tensor cores, for the sequence lengths
// of ViT (T = 197 or 257 tokens; any T in [193,208] or [241,260]) and head sizes 64 and 80.
//
// Persistent kernel, one CTA per SM, all 512 tensor-memory columns; a CTA walks over (image, head)
// pairs with a static schedule.  Per head the 256 queries that fit two 128-row tiles are handled
// by two softmax warpgroups side by side, one tile each, sharing one copy of K and V:
//   TMA warp     K, V of the next head into the other of two shared-memory stages while this
//                head is computed; Q (two tiles) as soon as the S products have read the old one.
//                Columns [0,64) of the head are 128-byte-swizzled rows, columns [64,80) (d = 80)
//                32-byte-swizzled rows; V for d = 80 is five 32-byte-swizzled 16-column blocks.
//   MMA warp     per tile: S = Q K^T (tcgen05.mma, 128 x NKP x d, fp32 in tensor memory), later
//                O = P V with A = P read from tensor memory and V as the N-major B operand
//   softmax      2 x 4 warps, one thread per query row: row max, exp2, row sum; P is written back
//                over S as packed bf16 (tcgen05.st), O lands in columns S no longer needs; then
//                O / rowsum -> bf16 -> global.  While one warpgroup is in its exp2 phase the
//                tensor core works for the other.
//   helper warps the 257th token (ViT-H) on warp-level MMAs: its score column joins the row max
//                and its probability is appended to P as one more 16-key step of P V (the rows
//                of V behind it are zeroed); the 257th query row is computed start to finish.
// Scores never leave the SM.  Every mbarrier wait is bounded; on expiry the CTA raises the device
// status word, waits (bounded) for its copies and MMAs in flight, frees tensor memory and leaves.
#include "vit_internal.h"
#include "sm100_ptx.cuh"

#include <cuda.h>

namespace vit {

namespace {

using namespace ptx;

constexpr int QT = 128;              // queries per tile = tensor-memory lanes
constexpr int MAX_EXTRA = 4;         // tokens beyond 256 handled outside the two tiles
constexpr int SOFTMAX_WARPS = 8;     // warps 0-3: tile 0, warps 4-7: tile 1
constexpr int MMA_WARP = 8, TMA_WARP = 9, AUX_WARP0 = 10, AUX_WARPS = 4;
constexpr int AUX_THREADS = AUX_WARPS * 32;
constexpr int NUM_THREADS = (SOFTMAX_WARPS + 2 + AUX_WARPS) * 32;
constexpr uint32_t TMEM_COLS = 512, TILE_COLS = 256;
constexpr long long DRAIN_LIMIT_CYCLES = 1ll << 24;   // teardown after a failed wait: ~10 ms

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

// warp-level tensor-core fragments for the helper warps (m16n8k16, bf16 operands, fp32 accumulate)
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(saddr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(saddr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
      "{%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct AttnMaps { CUtensorMap q64, q16, k64m, k64x, k16m, k16x; };

// Shared memory.  K and V hold NKP rows for the tensor core plus, for NKP = 256, 16 more rows
// (tokens 256 ... 271 of the image: the extra tokens, then rows that are zeroed or never read).
template <int D, int NKP>
struct Smem {
  static constexpr bool TAIL = D > 64;                 // columns [64, D) live in the 32-byte part
  static constexpr int XR = NKP == 256 ? 16 : 0;
  static constexpr int KR = NKP + XR;                  // rows of the K and V tiles
  static constexpr uint32_t KA = KR * 128, KB = TAIL ? KR * 32 : 0;
  static constexpr uint32_t VBLK = KR * 32;            // d = 80: one 16-column block of V
  static constexpr uint32_t VBYTES = TAIL ? (D / 16) * VBLK : KR * 128;
  static constexpr uint32_t OFF_KA = 0, OFF_KB = KA, OFF_V = KA + KB;
  static constexpr uint32_t STAGE = KA + KB + VBYTES;  // one head's K and V; two stages
  static constexpr uint32_t OFF_QA = 2 * STAGE;        // two tiles of 128 x 128 B
  static constexpr uint32_t OFF_QB = OFF_QA + 2 * QT * 128;
  static constexpr uint32_t OFF_SX = OFF_QB + (TAIL ? 2 * QT * 32 : 0);   // float [2][MAX_EXTRA][256]
  static constexpr uint32_t OFF_QX = OFF_SX + 2 * MAX_EXTRA * 256 * 4;    // bf16 [8][D]: Q rows 256 ... 263
  static constexpr uint32_t OFF_SC = OFF_QX + 8 * D * 2;                  // float [MAX_EXTRA][XS]: their scores, then probabilities
  static constexpr int XS = 272;
  static constexpr uint32_t OFF_INV = OFF_SC + MAX_EXTRA * XS * 4;        // float [MAX_EXTRA]: 1 / row sum
  static constexpr uint32_t OFF_BARS = OFF_INV + 16;
  static constexpr uint32_t BYTES = OFF_BARS + 256 + 1024 /*alignment slack*/;
  static constexpr uint32_t KV_TX = STAGE, Q_TX = 2 * QT * (TAIL ? 160 : 128);
  // Tensor memory of one tile (256 columns).  S occupies [0, NKP) and is consumed in 32-column
  // chunks.  P (bf16 pairs, 8 columns per 16 keys) overwrites columns that have been read: keys
  // 0 ... 191 go to [0, 96), the remaining keys to [192, 224), the extra keys to [224, 232).  O is
  // accumulated in [96, 96 + D).
  static constexpr int KLO = 12;                       // 16-key steps whose P sits below O
  static constexpr uint32_t P_HI_COL = 192, PX_COL = 224, O_COL = 96;
  __host__ __device__ static constexpr uint32_t p_col(int kstep) {
    return kstep < KLO ? (uint32_t)(8 * kstep) : P_HI_COL + (uint32_t)(8 * (kstep - KLO));
  }
  static_assert(O_COL + D <= P_HI_COL && NKP > 16 * KLO && NKP <= 256, "tensor-memory map");
  static_assert(BYTES <= 227 * 1024, "shared memory");
  static_assert(STAGE % 1024 == 0 && KA % 1024 == 0 && OFF_V % 256 == 0 && (TAIL || OFF_V % 1024 == 0), "alignment");
};

enum Bar : int {
  KV_FULL0 = 0, KV_FULL1, KV_FREE0, KV_FREE1, Q_FULL, Q_FREE, S_READY0, S_READY1,
  P_READY0, P_READY1, O_READY0, O_READY1, T_FREE0, T_FREE1, SX_READY0, SX_READY1, VZ_READY0, VZ_READY1, AUX_SYNC,
  DRAIN, NUM_BARS
};

template <int D, int NKP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
attention_tc_kernel(const __grid_constant__ AttnMaps maps, const bf16* __restrict__ qkv,
                    bf16* __restrict__ out, int T, int heads, int total_heads, int* dev_status) {
  using L = Smem<D, NKP>;
  constexpr int CH = D / 8;                      // 16-byte chunks per row
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);
  auto bar = [&](int i) { return smem_u32(&bars[i]); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(&bars[NUM_BARS]);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int H = heads * D;
  const size_t ld = (size_t)3 * H;
  const int n_x = T > 256 ? T - 256 : 0;         // tokens beyond the two tiles (NKP = 256 only)
  const int n_iter = total_heads > (int)blockIdx.x ? (total_heads - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(KV_FULL0), 1);
    mbar_init(bar(KV_FULL1), 1);
    mbar_init(bar(KV_FREE0), 1 + AUX_WARPS);     // PV products retired + helper warps done with K, V
    mbar_init(bar(KV_FREE1), 1 + AUX_WARPS);
    mbar_init(bar(Q_FULL), 1);
    mbar_init(bar(Q_FREE), 1 + AUX_WARPS);       // S products retired + helper warps done with Q
    for (int w = 0; w < 2; ++w) {
      mbar_init(bar(S_READY0 + w), 1);
      mbar_init(bar(P_READY0 + w), 4);           // one arrival per softmax warp of the tile
      mbar_init(bar(O_READY0 + w), 1);
      mbar_init(bar(T_FREE0 + w), 4);
      mbar_init(bar(VZ_READY0 + w), AUX_WARPS);
    }
    // the helper warps can be a head ahead of a softmax warpgroup: one barrier per head parity, so
    // that a warpgroup never finds its phase overtaken
    mbar_init(bar(SX_READY0), AUX_WARPS);
    mbar_init(bar(SX_READY1), AUX_WARPS);
    mbar_init(bar(AUX_SYNC), AUX_WARPS);
    mbar_init(bar(DRAIN), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == MMA_WARP) tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
  grid_dependency_wait();               // barrier set-up and allocation overlap the previous kernel's tail
  grid_launch_dependents();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == TMA_WARP) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int armed_kv[2] = {0, 0}, armed_q = 0;     // how often each "full" barrier has been armed
      bool ok = true;
      for (int it = 0; it < n_iter && ok; ++it) {
        const int work = (int)blockIdx.x + it * (int)gridDim.x;
        const int img = work / heads, hd = work % heads;
        const int row_g = img * T;               // global row of token 0
        const int col_q = hd * D, col_k = H + hd * D, col_v = 2 * H + hd * D;
        const int s = it & 1;
        const uint32_t st = sb + (uint32_t)s * L::STAGE;
        const uint32_t kf = bar(KV_FULL0 + s);
        if (!mbar_wait(bar(KV_FREE0 + s), (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag)) { ok = false; break; }
        mbar_arrive_expect_tx(kf, L::KV_TX);
        ++armed_kv[s];
        tma_load_2d(st + L::OFF_KA, &maps.k64m, col_k, row_g, kf);
        if (L::XR) tma_load_2d(st + L::OFF_KA + NKP * 128, &maps.k64x, col_k, row_g + NKP, kf);
        if (L::TAIL) {
          tma_load_2d(st + L::OFF_KB, &maps.k16m, col_k + 64, row_g, kf);
          if (L::XR) tma_load_2d(st + L::OFF_KB + NKP * 32, &maps.k16x, col_k + 64, row_g + NKP, kf);
#pragma unroll
          for (int a = 0; a < D / 16; ++a) {
            tma_load_2d(st + L::OFF_V + (uint32_t)a * L::VBLK, &maps.k16m, col_v + 16 * a, row_g, kf);
            if (L::XR)
              tma_load_2d(st + L::OFF_V + (uint32_t)a * L::VBLK + NKP * 32, &maps.k16x, col_v + 16 * a, row_g + NKP, kf);
          }
        } else {
          tma_load_2d(st + L::OFF_V, &maps.k64m, col_v, row_g, kf);
          if (L::XR) tma_load_2d(st + L::OFF_V + NKP * 128, &maps.k64x, col_v, row_g + NKP, kf);
        }
        if (!mbar_wait(bar(Q_FREE), (uint32_t)((it & 1) ^ 1), abort_flag)) { ok = false; break; }
        mbar_arrive_expect_tx(bar(Q_FULL), L::Q_TX);
        ++armed_q;
#pragma unroll
        for (int w = 0; w < 2; ++w) {
          tma_load_2d(sb + L::OFF_QA + (uint32_t)w * QT * 128, &maps.q64, col_q, row_g + w * QT, bar(Q_FULL));
          if (L::TAIL)
            tma_load_2d(sb + L::OFF_QB + (uint32_t)w * QT * 32, &maps.q16, col_q + 64, row_g + w * QT, bar(Q_FULL));
        }
      }
      if (*abort_flag) {
        // a wait gave up somewhere: let the copies that were started land before the CTA leaves
        volatile int never = 0;
        for (int s = 0; s < 2; ++s)
          if (armed_kv[s]) mbar_wait_limit(bar(KV_FULL0 + s), (uint32_t)((armed_kv[s] - 1) & 1), &never, DRAIN_LIMIT_CYCLES);
        if (armed_q) mbar_wait_limit(bar(Q_FULL), (uint32_t)((armed_q - 1) & 1), &never, DRAIN_LIMIT_CYCLES);
      }
    }
  } else if (warp == MMA_WARP) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      auto issue_s = [&](int w, uint32_t st) {
        const uint32_t d_tmem = tmem_base + (uint32_t)w * TILE_COLS;
        // S = Q K^T: 16 columns of the head per step, 32 bytes further along the swizzled row
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_bf16(d_tmem, make_desc_sw128(sb + L::OFF_QA + (uint32_t)w * QT * 128) + (uint64_t)(2 * k),
                    make_desc_sw128(st + L::OFF_KA) + (uint64_t)(2 * k), idesc_bf16(NKP, false), k > 0 ? 1u : 0u);
        if (L::TAIL)
          umma_bf16(d_tmem, make_desc_sw32(sb + L::OFF_QB + (uint32_t)w * QT * 32), make_desc_sw32(st + L::OFF_KB),
                    idesc_bf16(NKP, false), 1u);
        umma_commit(bar(S_READY0 + w));
      };
      const int ksteps = NKP / 16 + (n_x > 0 ? 1 : 0);
      // O = P V: A = P in tensor memory (8 columns per 16 keys); B = V, 16 keys per step = two
      // 8-row groups of the tile.
      auto issue_pv = [&](int w, uint32_t st, int k0, int k1) {
        const uint32_t t0 = tmem_base + (uint32_t)w * TILE_COLS;
#pragma unroll 1
        for (int k = k0; k < k1; ++k) {
          const uint64_t bdesc = L::TAIL ? make_desc_sw32_blocks(st + L::OFF_V + (uint32_t)(k * 512), L::VBLK)
                                         : make_desc_sw128(st + L::OFF_V + (uint32_t)(k * 2048));
          umma_bf16_ts(t0 + L::O_COL, t0 + L::p_col(k), bdesc, idesc_bf16(D, true), k > 0 ? 1u : 0u);
        }
      };
      // Issue order per head h: S_0(h), P V of tile 1 of head h - 1, S_1(h), P V of tile 0 of head h:
      // tile 1 runs behind tile 0, so that one warpgroup is in its exp2 phase while the tensor core
      // serves the other.  (Letting the two tiles advance independently by polling, and issuing P V
      // in two parts as P becomes ready, both measured slower.)
      for (int it = 0; it <= n_iter && ok && n_iter > 0; ++it) {
        const int s = it & 1;
        const uint32_t st = sb + (uint32_t)s * L::STAGE, st_prev = sb + (uint32_t)(s ^ 1) * L::STAGE;
        const uint32_t hph = (uint32_t)(it & 1), kph = (uint32_t)((it >> 1) & 1);
        const bool head = it < n_iter;
        if (head) {
          if (!mbar_wait(bar(KV_FULL0 + s), kph, abort_flag)) { ok = false; break; }
          if (!mbar_wait(bar(Q_FULL), hph, abort_flag)) { ok = false; break; }
          if (!mbar_wait(bar(T_FREE0), hph ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_s(0, st);
        }
        if (it > 0) {
          if (!mbar_wait(bar(P_READY1), hph ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_pv(1, st_prev, 0, ksteps);
          umma_commit(bar(O_READY1));
          umma_commit(bar(KV_FREE0 + (s ^ 1)));
        }
        if (head) {
          if (!mbar_wait(bar(T_FREE1), hph ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_s(1, st);
          umma_commit(bar(Q_FREE));
          if (!mbar_wait(bar(VZ_READY0 + s), kph, abort_flag)) { ok = false; break; }
          if (!mbar_wait(bar(P_READY0), hph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          issue_pv(0, st, 0, ksteps);
          umma_commit(bar(O_READY0));
        }
      }
      if (*abort_flag) {
        volatile int never = 0;
        umma_commit(bar(DRAIN));                 // products issued so far retire before tensor memory is freed
        mbar_wait_limit(bar(DRAIN), 0, &never, DRAIN_LIMIT_CYCLES);
      }
    }
  }
  else if (warp < SOFTMAX_WARPS) {
    // ------------------------------------------------------------------ softmax + epilogue
    const int wg = warp >> 2, quarter = warp & 3;
    const int tok = wg * QT + quarter * 32 + lane;          // token of this thread's query row
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)wg * TILE_COLS;
    const bool warp_active = wg * QT + quarter * 32 < T;    // any valid row in this warp
    const int kmax = T < NKP ? T : NKP;                     // keys the tensor core covers
    const float sl2 = 1.4426950408889634f / sqrtf((float)D);   // log2(e) / sqrt(d)
    constexpr int NCH = (NKP + 31) / 32;                    // 32-key chunks of S (the last may be partial)
    const float* sx_all = reinterpret_cast<const float*>(smem + L::OFF_SX);
    bool ok = true;
    for (int it = 0; it < n_iter && ok; ++it) {
      const int work = (int)blockIdx.x + it * (int)gridDim.x;
      const int img = work / heads, hd = work % heads;
      const uint32_t hph = (uint32_t)(it & 1);
      const float* sxh = sx_all + (it & 1) * MAX_EXTRA * 256;
      if (!mbar_wait(bar(S_READY0 + wg), hph, abort_flag)) { ok = false; break; }
      if (n_x > 0 && !mbar_wait(bar(SX_READY0 + (it & 1)), (uint32_t)((it >> 1) & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      float l = 0.f;
      if (warp_active) {
        // pass 1: row maximum, two 32-column loads per wait (the reduction is short; what counts
        // is the latency of the tensor-memory loads)
        float m = -INFINITY;
#pragma unroll
        for (int e = 0; e < MAX_EXTRA; ++e)
          if (e < n_x) m = fmaxf(m, sxh[e * 256 + tok]);
        uint32_t r[2][32];
#pragma unroll
        for (int i = 0; i < NCH; i += 2) {
          tmem_ld32(taddr + (uint32_t)(32 * i), r[0]);
          if (i + 1 < NCH) tmem_ld32(taddr + (uint32_t)(32 * (i + 1)), r[1]);
          tmem_ld_wait_for(r[0]);
          if (i + 1 < NCH) tmem_ld_wait_for(r[1]);
#pragma unroll
          for (int h2 = 0; h2 < 2; ++h2) {
            if (i + h2 >= NCH) continue;
            const uint32_t (&c)[32] = r[h2];
            const int c0 = 32 * (i + h2);
            if (c0 + 32 <= kmax) {
              float m2[2] = {m, m};
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                asm("max.f32 %0, %0, %1, %2;" : "+f"(m2[0]) : "f"(__uint_as_float(c[j])), "f"(__uint_as_float(c[j + 1])));
                asm("max.f32 %0, %0, %1, %2;" : "+f"(m2[1]) : "f"(__uint_as_float(c[j + 2])), "f"(__uint_as_float(c[j + 3])));
              }
              m = fmaxf(m2[0], m2[1]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c0 + j < kmax) m = fmaxf(m, __uint_as_float(c[j]));
            }
          }
        }
        const float msl = m * sl2;
        // pass 2: p = exp2((s - m) * sl2), row sum, P (bf16 pairs) back into tensor memory over
        // columns this thread has already read (see the tensor-memory map).  The load of chunk
        // i + 1 is in flight while chunk i is worked on.
        float2 l2 = make_float2(0.f, 0.f);
        const float2 sl2v = make_float2(sl2, sl2), nmsl = make_float2(-msl, -msl);
        tmem_ld32(taddr, r[0]);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          tmem_ld_wait_for(r[i & 1]);
          if (i + 1 < NCH) tmem_ld32(taddr + (uint32_t)(32 * (i + 1)), r[(i + 1) & 1]);
          const uint32_t (&c)[32] = r[i & 1];
          uint32_t pk[16];
          if (32 * i + 32 <= kmax) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float2 x = __ffma2_rn(make_float2(__uint_as_float(c[2 * j]), __uint_as_float(c[2 * j + 1])), sl2v, nmsl);
              const float2 pp = make_float2(ex2_approx(x.x), ex2_approx(x.y));
              l2 = __fadd2_rn(l2, pp);
              pk[j] = pack_bf16(pp.x, pp.y);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int k0 = 32 * i + 2 * j;
              const float p0 = k0 < kmax ? ex2_approx(fmaf(__uint_as_float(c[2 * j]), sl2, -msl)) : 0.f;
              const float p1 = k0 + 1 < kmax ? ex2_approx(fmaf(__uint_as_float(c[2 * j + 1]), sl2, -msl)) : 0.f;
              l2.x += p0;
              l2.y += p1;
              pk[j] = pack_bf16(p0, p1);
            }
          }
          if (32 * i + 32 <= NKP) {
            tmem_st16(taddr + L::p_col(2 * i), pk);
          } else {                                   // NKP = 208: the last chunk holds 16 keys
            uint32_t part[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) part[j] = pk[j];
            tmem_st8(taddr + L::p_col(2 * i), part);
          }
        }
        l = l2.x + l2.y;
        if (n_x > 0) {
          // the extra keys' probabilities: one more 16-key step of P (keys 256 ... 271)
          float px[MAX_EXTRA];
#pragma unroll
          for (int e = 0; e < MAX_EXTRA; ++e) {
            px[e] = e < n_x ? ex2_approx(fmaf(sxh[e * 256 + tok], sl2, -msl)) : 0.f;
            l += px[e];
          }
          const uint32_t xp[8] = {pack_bf16(px[0], px[1]), pack_bf16(px[2], px[3]), 0u, 0u, 0u, 0u, 0u, 0u};
          tmem_st8(taddr + L::PX_COL, xp);
        }
        tmem_st_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(P_READY0 + wg));
      // epilogue: O / l -> bf16 -> global
      if (!mbar_wait(bar(O_READY0 + wg), hph, abort_flag)) { ok = false; break; }
      tc_fence_after();
      uint32_t o[D];
      if (warp_active) {
#pragma unroll
        for (int g = 0; g < D / 16; ++g)
          tmem_ld16(taddr + L::O_COL + (uint32_t)(g * 16), *reinterpret_cast<uint32_t(*)[16]>(&o[g * 16]));
        tmem_ld_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(T_FREE0 + wg));   // the next head's S may overwrite this tile now
      if (warp_active && tok < T) {
        const float inv = 1.0f / l;
        // the row is 32-byte aligned (d is a multiple of 16): 32-byte stores, one sector each
        bf16* orow = out + ((size_t)img * T + tok) * H + (size_t)hd * D;
#pragma unroll
        for (int c = 0; c < D / 16; ++c) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            w[q] = pack_bf16(__uint_as_float(o[16 * c + 2 * q]) * inv, __uint_as_float(o[16 * c + 2 * q + 1]) * inv);
          asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(orow + 16 * c), "r"(w[0]),
                       "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                       : "memory");
        }
      }
    }
  }
  else if (warp >= AUX_WARP0) {
    // ------------------------------------------------------------------ helper warps
    const int j = threadIdx.x - AUX_WARP0 * 32;             // 0 ... AUX_THREADS - 1
    const int aw = warp - AUX_WARP0;
    const float sl2 = 1.4426950408889634f / sqrtf((float)D);
    float* sx_all = reinterpret_cast<float*>(smem + L::OFF_SX);
    float* sc = reinterpret_cast<float*>(smem + L::OFF_SC);
    float* inv_l = reinterpret_cast<float*>(smem + L::OFF_INV);
    const uint32_t qxb = sb + L::OFF_QX;
    // fragment coordinates of this lane: ldmatrix row / 16-byte chunk offsets, mma row and column pair
    const int lrow = (lane & 7) + 8 * ((lane >> 3) & 1), lchunk = lane >> 4;
    const int g = lane >> 2, t2 = 2 * (lane & 3);
    uint32_t aux_phase = 0;
    bool ok = true;
    // barrier among the helper warps (bounded like every other wait)
    auto aux_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(AUX_SYNC));
      const bool done = mbar_wait(bar(AUX_SYNC), aux_phase, abort_flag);
      aux_phase ^= 1;
      return done;
    };
    // shared-memory address of 16-byte chunk c of row r of V (st = stage base)
    auto v_chunk = [&](uint32_t st, int r, int c) -> uint32_t {
      return L::TAIL ? st + L::OFF_V + (uint32_t)((c >> 1) * L::VBLK + r * 32 + (((c & 1) ^ ((r >> 2) & 1)) << 4))
                     : st + L::OFF_V + (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
    };
    // Fragment addresses for the warp-level MMAs, k-step ks (16 head columns): this lane's row of a
    // 16-row A tile that starts at row0 (a multiple of 16), and of an 8-row B tile (brow0 a multiple
    // of 8).  main = the 128-byte-swizzled part (columns 0 ... 63), tail = the 32-byte part.
    const uint32_t a_main = (uint32_t)(lrow * 128), a_tail = (uint32_t)(lrow * 32 + ((lchunk ^ ((lrow >> 2) & 1)) << 4));
    const int hb = (lane >> 3) & 1, brow = lane & 7;
    const uint32_t b_main = (uint32_t)(brow * 128), b_tail = (uint32_t)(brow * 32 + ((hb ^ ((brow >> 2) & 1)) << 4));
    auto a_addr = [&](uint32_t main, uint32_t tail, int row0, int ks) -> uint32_t {
      if (ks < 4) return main + (uint32_t)(row0 * 128) + a_main + (uint32_t)((((2 * ks + lchunk) ^ (lrow & 7))) << 4);
      return tail + (uint32_t)(row0 * 32) + a_tail;
    };
    auto b_addr = [&](uint32_t main, uint32_t tail, int brow0, int ks) -> uint32_t {
      if (ks < 4) return main + (uint32_t)(brow0 * 128) + b_main + (uint32_t)((((2 * ks + hb) ^ brow)) << 4);
      return tail + (uint32_t)(brow0 * 32) + b_tail;
    };
    for (int it = 0; it < n_iter && ok; ++it) {
      const int work = (int)blockIdx.x + it * (int)gridDim.x;
      const int img = work / heads, hd = work % heads;
      const int s = it & 1;
      const uint32_t st = sb + (uint32_t)s * L::STAGE;
      const uint32_t hph = (uint32_t)(it & 1), kph = (uint32_t)((it >> 1) & 1);
      if (!mbar_wait(bar(KV_FULL0 + s), kph, abort_flag)) { ok = false; break; }
      // rows of V behind the last token are multiplied by zero probabilities: make them zero too,
      // so that whatever lies behind this image in memory cannot reach the result
      for (int i = j; i < (L::KR - T) * CH; i += AUX_THREADS) {
        const int r = T + i / CH, c = i % CH;
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(v_chunk(st, r, c)), "r"(0u) : "memory");
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(VZ_READY0 + s));
      if (!mbar_wait(bar(Q_FULL), hph, abort_flag)) { ok = false; break; }
      if (n_x > 0) {
        // scores of the extra keys for the 256 tile rows: [256 x d] . [d x 8] on warp-level MMAs,
        // A = 16 rows of Q, B = rows 256 ... 263 of K (columns beyond the extra keys are not used)
        float* sxh = sx_all + (it & 1) * MAX_EXTRA * 256;
        uint32_t bk[D / 16][2];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) ldmatrix_x2(bk[ks], b_addr(st + L::OFF_KA, st + L::OFF_KB, 256, ks));
#pragma unroll 1
        for (int mt = aw; mt < 16; mt += AUX_WARPS) {
          float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(a, a_addr(sb + L::OFF_QA, sb + L::OFF_QB, mt * 16, ks));
            mma_bf16(c, a, bk[ks][0], bk[ks][1]);
          }
          const int r0 = mt * 16 + g;
          if (t2 < n_x) { sxh[t2 * 256 + r0] = c[0]; sxh[t2 * 256 + r0 + 8] = c[2]; }
          if (t2 + 1 < n_x) { sxh[(t2 + 1) * 256 + r0] = c[1]; sxh[(t2 + 1) * 256 + r0 + 8] = c[3]; }
        }
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(SX_READY0 + (it & 1)));
        mbar_arrive(bar(Q_FREE));
      }
      if (n_x > 0) {
        // the extra query rows, start to finish, on warp-level MMAs.  Rows 256 ... 263 of Q as
        // plain rows in shared memory (rows that are not extra queries are zero).
        for (int i = j; i < 8 * CH; i += AUX_THREADS) {
          const int e = i / CH, c = i % CH;
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (e < n_x) v = __ldg(reinterpret_cast<const uint4*>(qkv + ((size_t)img * T + 256 + e) * ld + (size_t)hd * D) + c);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(qxb + (uint32_t)(i * 16)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
        if (!aux_sync()) { ok = false; break; }
        // scores[key][e] = K[key] . Q[256 + e]
        uint32_t bq[D / 16][2];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          ldmatrix_x2(bq[ks], qxb + (uint32_t)(((lane & 7) * CH + 2 * ks + ((lane >> 3) & 1)) * 16));
        const int n_kt = (T + 15) / 16;                      // 16-key tiles
#pragma unroll 1
        for (int mt = aw; mt < n_kt; mt += AUX_WARPS) {
          float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t a[4];
            ldmatrix_x4(a, a_addr(st + L::OFF_KA, st + L::OFF_KB, mt * 16, ks));
            mma_bf16(c, a, bq[ks][0], bq[ks][1]);
          }
          const int k0 = mt * 16 + g;
          if (t2 < n_x) { sc[t2 * L::XS + k0] = c[0]; sc[t2 * L::XS + k0 + 8] = c[2]; }
          if (t2 + 1 < n_x) { sc[(t2 + 1) * L::XS + k0] = c[1]; sc[(t2 + 1) * L::XS + k0 + 8] = c[3]; }
        }
        if (!aux_sync()) { ok = false; break; }
        // softmax of row e by one warp: probabilities (zero behind the last token) and 1 / row sum
        for (int e = aw; e < n_x; e += AUX_WARPS) {
          float* row = sc + e * L::XS;
          float m = -INFINITY;
          for (int key = lane; key < T; key += 32) m = fmaxf(m, row[key]);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
          const float msl = m * sl2;
          float lsum = 0.f;
          for (int key = lane; key < n_kt * 16; key += 32) {
            const float p = key < T ? ex2_approx(fmaf(row[key], sl2, -msl)) : 0.f;
            row[key] = p;
            lsum += p;
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
          if (lane == 0) inv_l[e] = 1.0f / lsum;
        }
        if (!aux_sync()) { ok = false; break; }
        // O[e][:] = P[e][:] V: A = probabilities (rows beyond the extra queries zero), B = V through
        // transposing fragment loads; a warp owns pairs of 8-column tiles of the head
#pragma unroll 1
        for (int pr = aw; pr < CH / 2; pr += AUX_WARPS) {
          float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
          for (int kt = 0; kt < n_kt; ++kt) {
            uint32_t a[4] = {0u, 0u, 0u, 0u};
            if (g < n_x) {
              const float2 p0 = *reinterpret_cast<const float2*>(sc + g * L::XS + kt * 16 + t2);
              const float2 p1 = *reinterpret_cast<const float2*>(sc + g * L::XS + kt * 16 + 8 + t2);
              a[0] = pack_bf16(p0.x, p0.y);
              a[2] = pack_bf16(p1.x, p1.y);
            }
            uint32_t b[4];
            ldmatrix_x4_trans(b, v_chunk(st, kt * 16 + lrow, 2 * pr + lchunk));
            mma_bf16(acc0, a, b[0], b[1]);
            mma_bf16(acc1, a, b[2], b[3]);
          }
          if (g < n_x) {
            const float inv = inv_l[g];
            bf16* orow = out + ((size_t)img * T + 256 + g) * H + (size_t)hd * D + 16 * pr + t2;
            *reinterpret_cast<uint32_t*>(orow) = pack_bf16(acc0[0] * inv, acc0[1] * inv);
            *reinterpret_cast<uint32_t*>(orow + 8) = pack_bf16(acc1[0] * inv, acc1[1] * inv);
          }
        }
      }
      if (!ok) break;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(KV_FREE0 + s));
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
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

bool encode_map_raw(CUtensorMap* tm, const void* base, size_t rows, size_t cols, int box_cols, int box_rows,
                    CUtensorMapSwizzle sw);
bool encode_map(TensorMapCache* cache, CUtensorMap* tm, const void* base, size_t rows, size_t cols, int box_cols,
                int box_rows, CUtensorMapSwizzle sw) {
  const TensorMapKey key{base, (uint64_t)rows, (uint64_t)cols, (uint64_t)cols, (uint32_t)box_rows, (uint32_t)box_cols,
                         (uint32_t)sw + 1000u};
  return TensorMapCache::get(cache, key, tm, [&](CUtensorMap* out) { return encode_map_raw(out, base, rows, cols, box_cols, box_rows, sw); });
}
bool encode_map_raw(CUtensorMap* tm, const void* base, size_t rows, size_t cols, int box_cols, int box_rows,
                    CUtensorMapSwizzle sw) {
  const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box,
                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int NKP>
cudaError_t launch_variant(const bf16* qkv, bf16* out, int images, int T, int heads, int* dev_status,
                           cudaStream_t s, TensorMapCache* cache) {
  using L = Smem<D, NKP>;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !fn)
      return cudaErrorNotReady;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  static PerDeviceFlag configured;
  cudaError_t e = ensure_dynamic_smem(configured, attention_tc_kernel<D, NKP>, (int)L::BYTES);
  if (e != cudaSuccess) return e;
  const int sms = current_device_sm_count();
  if (sms < 1) return cudaErrorInvalidDevice;
  const size_t rows = (size_t)images * T, cols = (size_t)3 * heads * D;
  const CUtensorMapSwizzle s128 = CU_TENSOR_MAP_SWIZZLE_128B, s32 = CU_TENSOR_MAP_SWIZZLE_32B;
  AttnMaps m;
  if (!encode_map(cache, &m.q64, qkv, rows, cols, 64, QT, s128)) return cudaErrorInvalidValue;
  if (!encode_map(cache, &m.k64m, qkv, rows, cols, 64, NKP, s128)) return cudaErrorInvalidValue;
  if (!encode_map(cache, &m.k64x, qkv, rows, cols, 64, 16, s128)) return cudaErrorInvalidValue;
  if (D > 64) {
    if (!encode_map(cache, &m.q16, qkv, rows, cols, 16, QT, s32)) return cudaErrorInvalidValue;
    if (!encode_map(cache, &m.k16m, qkv, rows, cols, 16, NKP, s32)) return cudaErrorInvalidValue;
    if (!encode_map(cache, &m.k16x, qkv, rows, cols, 16, 16, s32)) return cudaErrorInvalidValue;
  } else {
    m.q16 = m.q64;
    m.k16m = m.k64m;
    m.k16x = m.k64x;
  }
  const int total = images * heads;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(total < sms ? total : sms));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = L::BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_tc_kernel<D, NKP>, m, qkv, out, T, heads, total, dev_status);
}

}  // namespace

bool attention_tc_supported(int T, int d) {
  if (d != 64 && d != 80) return false;
  return (T >= 193 && T <= 208) || (T >= 241 && T <= 256 + MAX_EXTRA);
}

cudaError_t launch_attention_tc(const bf16* qkv, bf16* out, int images, int T, int heads, int d,
                                int* dev_status, cudaStream_t s, TensorMapCache* cache) {
  if (images <= 0) return cudaSuccess;
  if (!attention_tc_supported(T, d)) return cudaErrorInvalidValue;
  const bool wide = T > 208;
  if (d == 64) return wide ? launch_variant<64, 256>(qkv, out, images, T, heads, dev_status, s, cache)
                           : launch_variant<64, 208>(qkv, out, images, T, heads, dev_status, s, cache);
  return wide ? launch_variant<80, 256>(qkv, out, images, T, heads, dev_status, s, cache)
              : launch_variant<80, 208>(qkv, out, images, T, heads, dev_status, s, cache);
}

}  // namespace vit
