// Linear layers on the 5th-generation tensor cores:  out[M,N] = epi(a[M,K] . w[N,K]^T + bias).
//
// Persistent, warp-specialised kernel, one CTA per SM:
//   warp 0      TMA producer: 128 x 64 tile of a and BN x 64 tile of w per stage, 128-byte swizzle
//   warp 1      allocates tensor memory and issues tcgen05.mma (128 x BN x 16 per instruction)
//   warps 2..9  epilogue: tcgen05.ld the fp32 accumulator, bias / GELU / residual, bf16 rows staged
//               in swizzled shared memory and written with TMA stores (the residual tile arrives
//               the same way, by TMA load), so global traffic is coalesced and asynchronous
// Two accumulators live in tensor memory (2 x BN columns) so the epilogue of tile i overlaps the
// main loop of tile i+1.  Tiles are handed out statically (tile = blockIdx.x + i * gridDim.x).
// For large problems the kernel runs as CTA pairs (CTAS = 2, a cluster of two): one 256 x 256
// tile per pair, each CTA loads its own 128 rows of a and half of the w tile (no multicast), the
// even CTA issues tcgen05.mma.cta_group::2 for both, and each CTA drains its own 128 rows of the
// accumulator.  Shared-memory fill traffic per flop drops by a third, which leaves room for the
// output stores.
// Every mbarrier wait is bounded; on expiry the CTA raises the device status word and leaves.
#include "vit_internal.h"
#include "sm100_ptx.cuh"

#include <cuda.h>

namespace vit {

namespace {

using namespace ptx;

constexpr int BM = 128;
constexpr int BK = 64;        // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = (2 + NUM_EPI_WARPS) * 32;
constexpr long long DRAIN_LIMIT_CYCLES = 1ll << 24;   // teardown after a failed wait: ~10 ms per barrier

template <int BN, int CTAS> struct Cfg {
  static constexpr int B_ROWS = BN / CTAS;                 // rows of the w tile this CTA loads
  static constexpr int STAGES = (B_ROWS == 256) ? 4 : 6;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = B_ROWS * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;                 // 512 or 256: a power of two
  static constexpr int STAGING_BYTES = NUM_EPI_WARPS * 4096;   // 32 rows x 128 B per epilogue warp
  static constexpr int SMEM_BYTES =
      STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, groups
// of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)1 << 16;                          // leading-dimension byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                // stride-dimension byte offset: 8 rows x 128 B
  d |= (uint64_t)1 << 46;                          // descriptor version for this architecture
  d |= (uint64_t)2 << 61;                          // swizzle mode: 128 bytes
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulate, bf16 x bf16, both operands K-major.
template <int BN, int CTAS> __host__ __device__ constexpr uint32_t make_idesc() {
  return (1u << 4)                       // D format: f32
         | (1u << 7)                     // A format: bf16
         | (1u << 10)                    // B format: bf16
         | ((uint32_t)(BN >> 3) << 17)   // N / 8
         | ((uint32_t)((BM * CTAS) >> 4) << 24);  // M / 16 (256 rows across a CTA pair)
}

// gelu(v) = 0.5 v (1 + erf(v / sqrt 2)) = max(v, 0) - 0.5 |v| erfc(|v| / sqrt 2), with
// erfc(z) = (a1 t + ... + a5 t^5) exp(-z^2), t = 1 / (1 + p z), z >= 0 (Abramowitz & Stegun
// 7.1.26, |error| <= 1.5e-7), on the MUFU reciprocal and exp2.  The factor -0.5 is folded into
// the coefficients and 1/sqrt 2 into p and the exponent scale.  Two values per call: the
// polynomial and the products run as packed two-wide fp32 instructions (9 instructions and
// 2 MUFU operations per value).
__device__ __forceinline__ float2 gelu_erf2(float2 v) {
  const float2 a = make_float2(fabsf(v.x), fabsf(v.y));
  const float kp = 0.3275911f * 0.70710678118654752440f;
  const float2 den = __ffma2_rn(make_float2(kp, kp), a, make_float2(1.0f, 1.0f));
  float2 t, e;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.x) : "f"(den.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t.y) : "f"(den.y));
  const float ke = -0.5f * 1.4426950408889634f;
  const float2 arg = __fmul2_rn(__fmul2_rn(a, a), make_float2(ke, ke));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.x) : "f"(arg.x));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e.y) : "f"(arg.y));
  const float c5 = -0.5f * 1.061405429f, c4 = -0.5f * -1.453152027f, c3 = -0.5f * 1.421413741f,
              c2 = -0.5f * -0.284496736f, c1 = -0.5f * 0.254829592f;
  float2 q = __ffma2_rn(make_float2(c5, c5), t, make_float2(c4, c4));
  q = __ffma2_rn(q, t, make_float2(c3, c3));
  q = __ffma2_rn(q, t, make_float2(c2, c2));
  q = __ffma2_rn(q, t, make_float2(c1, c1));
  const float2 r = make_float2(fmaxf(v.x, 0.f), fmaxf(v.y, 0.f));
  return __ffma2_rn(__fmul2_rn(q, a), __fmul2_rn(t, e), r);
}

struct TcParams {
  int M, N, K;
  const float* bias;
  const bf16* residual;   // EPI_BIAS_RESIDUAL
  const float* pos;       // EPI_BIAS_POS
  const float2* ln_stats; // EPI_LN_*
  const float* ln_c1;     // EPI_LN_*
  int n_patches, first_patch_token;
  bf16* out;
  int ldo;
  int tiles_m, tiles_n;
  int* dev_status;
};

template <int BN, int EPI, int CTAS>
__global__ void __launch_bounds__(NUM_THREADS, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_out, const __grid_constant__ CUtensorMap tm_res,
                 const TcParams p) {
  using C = Cfg<BN, CTAS>;
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: the swizzle pattern and the descriptors assume it
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* tiles = smem;
  uint8_t* staging = smem + C::STAGES * C::STAGE_BYTES;   // 1024-aligned: 4 KB per epilogue warp
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + C::STAGING_BYTES);
  uint64_t* full_bar = bars;                       // [STAGES]
  uint64_t* empty_bar = bars + C::STAGES;          // [STAGES]
  uint64_t* tfull_bar = bars + 2 * C::STAGES;      // [2]
  uint64_t* tempty_bar = bars + 2 * C::STAGES + 2; // [2]
  uint64_t* res_bar = bars + 2 * C::STAGES + 4;    // [NUM_EPI_WARPS] residual tile landed
  uint64_t* drain_bar = bars + 2 * C::STAGES + 4 + NUM_EPI_WARPS;   // teardown after a failed wait
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 5 + NUM_EPI_WARPS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;
  const int total_tiles = p.tiles_m * p.tiles_n;
  // scheduling unit: a CTA, or a pair of CTAs working on one 256-row tile
  const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
  const int unit = blockIdx.x / CTAS, num_units = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < C::STAGES; ++i) {
      mbar_init(smem_u32(&full_bar[i]), 1);
      mbar_init(smem_u32(&empty_bar[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&tfull_bar[i]), 1);
      mbar_init(smem_u32(&tempty_bar[i]), NUM_EPI_WARPS * CTAS);
    }
    for (int i = 0; i < NUM_EPI_WARPS; ++i) mbar_init(smem_u32(&res_bar[i]), 1);
    mbar_init(smem_u32(drain_bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_out)) : "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) tmem_alloc_pair(smem_u32(tmem_slot), (uint32_t)C::TMEM_COLS);
    else tmem_alloc(smem_u32(tmem_slot), (uint32_t)C::TMEM_COLS);
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync();          // the peer's barriers are initialised before anyone signals them
  tc_fence_after();
  // set-up above overlaps the tail of the previous kernel on the stream; its results are read
  // (and its inputs overwritten) only from here on
  grid_dependency_wait();
  grid_launch_dependents();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long long fills = 0;                         // stages filled so far (this CTA's share)
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
        const int m0 = (tile / p.tiles_n) * (BM * CTAS) + (int)rank * BM;
        const int n0 = (tile % p.tiles_n) * BN + (int)rank * C::B_ROWS;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1, abort_flag)) { ok = false; break; }
          ++fills;
          const uint32_t fb = smem_u32(&full_bar[stage]);
          const uint32_t sa = smem_u32(tiles + stage * C::STAGE_BYTES);
          if (CTAS == 2) {
            // both CTAs' copies are counted on the even CTA's barrier, which expects all the bytes
            const uint32_t fb0 = map_to_cta(fb, 0);
            if (rank == 0) mbar_arrive_expect_tx(fb, 2 * C::STAGE_BYTES);
            tma_load_2d_pair(sa, &tm_a, kb * BK, m0, fb0);
            tma_load_2d_pair(sa + C::A_BYTES, &tm_w, kb * BK, n0, fb0);
          } else {
            mbar_arrive_expect_tx(fb, C::STAGE_BYTES);
            tma_load_2d(sa, &tm_a, kb * BK, m0, fb);
            tma_load_2d(sa + C::A_BYTES, &tm_w, kb * BK, n0, fb);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (*abort_flag) {
        // A wait gave up somewhere in this CTA (or its partner).  The copies of the last STAGES
        // fills may still be in flight: wait, bounded, until each of those stages has received its
        // bytes, so that nothing lands in shared memory after the CTA has left.  In a pair the
        // barriers live in the even CTA and count both CTAs' bytes; the odd CTA is kept alive by
        // the cluster barrier of the teardown until the even one is through here.
        if (rank == 0) {
          volatile int never = 0;
          const long long first = fills > C::STAGES ? fills - C::STAGES : 0;
          for (long long f = first; f < fills; ++f)
            mbar_wait_limit(smem_u32(&full_bar[(int)(f % C::STAGES)]), (uint32_t)((f / C::STAGES) & 1), &never,
                            DRAIN_LIMIT_CYCLES);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc<BN, CTAS>();
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t aphase = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
        if (!mbar_wait(smem_u32(&tempty_bar[buf]), aphase ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(tiles + stage * C::STAGE_BYTES);
          const uint64_t adesc = make_smem_desc(sa);
          const uint64_t bdesc = make_smem_desc(sa + C::A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 elements along K = 32 bytes = 2 units of the encoded start address
            if (CTAS == 2)
              umma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                             (kb > 0 || k > 0) ? 1u : 0u);
            else
              umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                        (kb > 0 || k > 0) ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) when these MMAs retire
          if (CTAS == 2) umma_commit_pair(smem_u32(&empty_bar[stage]));
          else umma_commit(smem_u32(&empty_bar[stage]));
          if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (CTAS == 2) umma_commit_pair(smem_u32(&tfull_bar[buf]));   // accumulator complete
        else umma_commit(smem_u32(&tfull_bar[buf]));
        if (++buf == 2) { buf = 0; aphase ^= 1; }
      }
      if (*abort_flag) {
        // products issued so far retire before tensor memory is freed
        volatile int never = 0;
        umma_commit(smem_u32(drain_bar));
        mbar_wait_limit(smem_u32(drain_bar), 0, &never, DRAIN_LIMIT_CYCLES);
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int ew = warp - 2;
    const int quarter = warp & 3;                 // tensor-memory lanes this warp may read
    const int half = ew >> 2;                     // which half of the BN columns
    constexpr int COLS_PER_WARP = BN / 2;
    int buf = 0;
    uint32_t aphase = 0;
    if (EPI == EPI_BIAS_POS) {
      // patch embedding: rows are scattered to token 1 + patch of their image, direct stores
      for (int tile = unit; tile < total_tiles; tile += num_units) {
        const int m0 = (tile / p.tiles_n) * (BM * CTAS) + (int)rank * BM, n0 = (tile % p.tiles_n) * BN;
        if (!mbar_wait(smem_u32(&tfull_bar[buf]), aphase, abort_flag)) break;
        tc_fence_after();
        const int row = m0 + quarter * 32 + lane;
        const bool row_ok = row < p.M;
        const int img = row / p.n_patches, pt = row - img * p.n_patches;
        const size_t orow = (size_t)img * (p.n_patches + p.first_patch_token) + p.first_patch_token + pt;
        const float* posrow = p.pos + (size_t)(p.first_patch_token + pt) * p.N;
#pragma unroll 1
        for (int ch = 0; ch < COLS_PER_WARP / 32; ++ch) {
          const int cl = half * COLS_PER_WARP + ch * 32;
          const int c0 = n0 + cl;
          if (c0 >= p.N) break;                            // uniform across the warp
          uint32_t r[32];
          tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cl), r);
          tmem_ld_wait();
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int c = c0 + g * 8;
            if (c >= p.N || !row_ok) continue;
            uint4 o;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float v0 = __uint_as_float(r[g * 8 + 2 * e]) + __ldg(p.bias + c + 2 * e) +
                               __ldg(posrow + c + 2 * e);
              const float v1 = __uint_as_float(r[g * 8 + 2 * e + 1]) + __ldg(p.bias + c + 2 * e + 1) +
                               __ldg(posrow + c + 2 * e + 1);
              h[e] = __floats2bfloat162_rn(v0, v1);
            }
            *reinterpret_cast<uint4*>(p.out + orow * p.ldo + c) = o;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          // the accumulator buffer is handed back to the MMA issuer (the even CTA of a pair)
          if (CTAS == 2) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty_bar[buf]), 0));
          else mbar_arrive(smem_u32(&tempty_bar[buf]));
        }
        if (++buf == 2) { buf = 0; aphase ^= 1; }
      }
    } else {
      uint8_t* stg = staging + ew * 4096;            // this warp's 32-row x 64-column bf16 tile
      const uint32_t stg_u32 = smem_u32(stg);
      const uint32_t my_row = stg_u32 + (uint32_t)lane * 128u;
      const uint32_t rb = smem_u32(&res_bar[ew]);
      uint32_t rphase = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += num_units) {
        const int m0 = (tile / p.tiles_n) * (BM * CTAS) + (int)rank * BM, n0 = (tile % p.tiles_n) * BN;
        const int row0 = m0 + quarter * 32;
#pragma unroll 1
        for (int cb = 0; cb < COLS_PER_WARP / 64; ++cb) {
          const int cl = half * COLS_PER_WARP + cb * 64;   // column inside the tile
          const int c0 = n0 + cl;
          if (c0 >= p.N) break;                            // uniform across the warp
          if (EPI == EPI_BIAS_RESIDUAL) {
            // bring the residual tile into the staging buffer while the accumulator is awaited
            if (lane == 0) {
              tma_store_wait_read();
              mbar_arrive_expect_tx(rb, 4096);
              tma_load_2d(stg_u32, &tm_res, c0, row0, rb);
            }
          }
          if (cb == 0) {
            if (!mbar_wait(smem_u32(&tfull_bar[buf]), aphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
          }
          uint32_t r[64];
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cl);
          tmem_ld32(taddr, *reinterpret_cast<uint32_t(*)[32]>(&r[0]));
          tmem_ld32(taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&r[32]));
          tmem_ld_wait();
          float v[64];
          constexpr bool LN = EPI == EPI_LN_BIAS || EPI == EPI_LN_BIAS_GELU;
          float2 nmean = make_float2(0.f, 0.f), rstd = make_float2(1.f, 1.f);
          if (LN) {                                  // this thread's row: lane = row of the accumulator
            const float2 st = (row0 + lane < p.M) ? __ldg(p.ln_stats + row0 + lane) : make_float2(0.f, 1.f);
            nmean = make_float2(-st.x, -st.x);
            rstd = make_float2(st.y, st.y);
          }
#pragma unroll
          for (int g = 0; g < 16; ++g) {
            const bool in = c0 + 4 * g < p.N;
            const float4 b = in ? __ldg(reinterpret_cast<const float4*>(p.bias + c0) + g) : make_float4(0.f, 0.f, 0.f, 0.f);
            float2 lo = make_float2(__uint_as_float(r[4 * g + 0]), __uint_as_float(r[4 * g + 1]));
            float2 hi = make_float2(__uint_as_float(r[4 * g + 2]), __uint_as_float(r[4 * g + 3]));
            if (LN) {
              const float4 c1 = in ? __ldg(reinterpret_cast<const float4*>(p.ln_c1 + c0) + g) : make_float4(0.f, 0.f, 0.f, 0.f);
              lo = __ffma2_rn(rstd, __ffma2_rn(nmean, make_float2(c1.x, c1.y), lo), make_float2(b.x, b.y));
              hi = __ffma2_rn(rstd, __ffma2_rn(nmean, make_float2(c1.z, c1.w), hi), make_float2(b.z, b.w));
            } else {
              lo = __fadd2_rn(lo, make_float2(b.x, b.y));
              hi = __fadd2_rn(hi, make_float2(b.z, b.w));
            }
            v[4 * g + 0] = lo.x;
            v[4 * g + 1] = lo.y;
            v[4 * g + 2] = hi.x;
            v[4 * g + 3] = hi.y;
          }
          if (EPI == EPI_BIAS_GELU || EPI == EPI_LN_BIAS_GELU) {
#pragma unroll
            for (int e = 0; e < 64; e += 2) {
              const float2 y = gelu_erf2(make_float2(v[e], v[e + 1]));
              v[e] = y.x;
              v[e + 1] = y.y;
            }
          }
          if (EPI == EPI_BIAS_RESIDUAL) {
            if (!mbar_wait(rb, rphase, abort_flag)) { ok = false; break; }
            rphase ^= 1;
#pragma unroll
            for (int ck = 0; ck < 8; ++ck) {
              uint4 u;
              const uint32_t a = my_row + (uint32_t)((ck ^ (lane & 7)) << 4);
              asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                           : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w)
                           : "r"(a));
              const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float2 y = __fadd2_rn(make_float2(v[ck * 8 + 2 * e], v[ck * 8 + 2 * e + 1]), __bfloat1622float2(h[e]));
                v[ck * 8 + 2 * e] = y.x;
                v[ck * 8 + 2 * e + 1] = y.y;
              }
            }
          } else {
            if (lane == 0) tma_store_wait_read();          // previous store has left the buffer
            __syncwarp();
          }
#pragma unroll
          for (int ck = 0; ck < 8; ++ck) {
            uint4 o;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
            for (int e = 0; e < 4; ++e) h[e] = __floats2bfloat162_rn(v[ck * 8 + 2 * e], v[ck * 8 + 2 * e + 1]);
            const uint32_t a = my_row + (uint32_t)((ck ^ (lane & 7)) << 4);   // 128-byte swizzle
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(o.x), "r"(o.y),
                         "r"(o.z), "r"(o.w)
                         : "memory");
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) tma_store_2d(&tm_out, stg_u32, c0, row0);   // rows >= M, columns >= N are clipped
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          // the accumulator buffer is handed back to the MMA issuer (the even CTA of a pair)
          if (CTAS == 2) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty_bar[buf]), 0));
          else mbar_arrive(smem_u32(&tempty_bar[buf]));
        }
        if (++buf == 2) { buf = 0; aphase ^= 1; }
      }
      if (lane == 0) tma_store_wait_all();
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (CTAS == 2 && *abort_flag) {
    // tell the partner, which may be in a wait of its own that nothing will satisfy any more
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(map_to_cta(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u)), "r"(1) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  if (CTAS == 2) cluster_sync();          // neither CTA leaves while the other may still touch it
  tc_fence_after();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.dev_status, (int)VIT_ERR_TIMEOUT);
  if (warp == 1) {
    __syncwarp();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, (uint32_t)C::TMEM_COLS);
    else tmem_dealloc(tmem_base, (uint32_t)C::TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

bool encode_2d_bf16_raw(CUtensorMap* tm, const void* base, int rows, int cols, int ld, int box_rows);
bool encode_2d_bf16(TensorMapCache* cache, CUtensorMap* tm, const void* base, int rows, int cols, int ld, int box_rows) {
  const TensorMapKey key{base, (uint64_t)rows, (uint64_t)cols, (uint64_t)ld, (uint32_t)box_rows, (uint32_t)BK, 128u};
  return TensorMapCache::get(cache, key, tm, [&](CUtensorMap* out) { return encode_2d_bf16_raw(out, base, rows, cols, ld, box_rows); });
}
bool encode_2d_bf16_raw(CUtensorMap* tm, const void* base, int rows, int cols, int ld, int box_rows) {
  if (base == nullptr) return false;
  const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride,
                  box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Maps { CUtensorMap a, w, out, res; };

template <int BN, int EPI, int CTAS>
cudaError_t launch_variant(const Maps& m, const TcParams& p, cudaStream_t s) {
  using C = Cfg<BN, CTAS>;
  static PerDeviceFlag configured;
  cudaError_t e = ensure_dynamic_smem(configured, linear_tc_kernel<BN, EPI, CTAS>, C::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int total = p.tiles_m * p.tiles_n;
  const int units = current_device_sm_count() / CTAS;
  const int grid = (total < units ? total : units) * CTAS;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, linear_tc_kernel<BN, EPI, CTAS>, m.a, m.w, m.out, m.res, p);
}

template <int BN, int CTAS>
cudaError_t launch_bn(int epi, const Maps& m, const TcParams& p, cudaStream_t s) {
  switch (epi) {
    case EPI_BIAS: return launch_variant<BN, EPI_BIAS, CTAS>(m, p, s);
    case EPI_BIAS_GELU: return launch_variant<BN, EPI_BIAS_GELU, CTAS>(m, p, s);
    case EPI_BIAS_RESIDUAL: return launch_variant<BN, EPI_BIAS_RESIDUAL, CTAS>(m, p, s);
    case EPI_BIAS_POS: return launch_variant<BN, EPI_BIAS_POS, CTAS>(m, p, s);
    case EPI_LN_BIAS: return launch_variant<BN, EPI_LN_BIAS, CTAS>(m, p, s);
    case EPI_LN_BIAS_GELU: return launch_variant<BN, EPI_LN_BIAS_GELU, CTAS>(m, p, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

// A wait that nothing ever satisfies, with a short limit: shows the path a stuck kernel takes
// (status word raised, kernel returns, context stays usable) without hanging anything.
namespace {
__global__ void wait_probe_kernel(long long limit_cycles, int* dev_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!ptx::mbar_wait_limit(ptx::smem_u32(&bar), 0, &abort_flag, limit_cycles))
      atomicExch(dev_status, (int)VIT_ERR_TIMEOUT);
  }
}
}  // namespace

namespace {
__global__ void status_take_kernel(int* status, int* snapshot) { *snapshot = atomicExch(status, 0); }
}  // namespace

cudaError_t launch_status_take(int* status, int* snapshot, cudaStream_t s) {
  status_take_kernel<<<1, 1, 0, s>>>(status, snapshot);
  return cudaGetLastError();
}

cudaError_t launch_wait_probe(long long limit_cycles, int* dev_status, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(limit_cycles, dev_status);
  return cudaGetLastError();
}

bool tc_gemm_init() {
  if (g_encode) return true;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || fn == nullptr)
    return false;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  return current_device_sm_count() > 0;
}

int current_device_sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  const bool tracked = dev >= 0 && dev < 64;
  int n = tracked ? cache[dev].load(std::memory_order_relaxed) : 0;
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (tracked) cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

cudaError_t launch_linear_tc(const LinearArgs& a, int* dev_status, cudaStream_t s, TensorMapCache* cache) {
  if (a.M <= 0 || a.N <= 0) return cudaSuccess;
  if (!g_encode) return cudaErrorNotReady;
  if (a.K % 8 || a.N % 8 || a.lda % 8 || a.ldw % 8 || a.ldo % 8 || a.K <= 0) return cudaErrorInvalidValue;
  if ((reinterpret_cast<uintptr_t>(a.a) | reinterpret_cast<uintptr_t>(a.w) |
       reinterpret_cast<uintptr_t>(a.out) | reinterpret_cast<uintptr_t>(a.residual)) & 15)
    return cudaErrorInvalidValue;
  // Shape-only choice of the tiling by a small cost model: rounds of the static schedule times
  // the per-SM work of one tile (128x256 = 1 for a pair or a single CTA, 128x128 = 0.5, measured nearer 0.75), with a
  // bonus for the pair tiling's lower load traffic and a penalty for the small tile's overheads.
  const long long nt256 = (a.N + 255) / 256, nt128 = (a.N + 127) / 128;
  const long long tm1 = (a.M + BM - 1) / BM, tm2 = (a.M + 2 * BM - 1) / (2 * BM);
  const int sms = current_device_sm_count();
  if (sms < 2) return cudaErrorInvalidDevice;
  const long long units1 = sms, units2 = sms / 2;
  auto rounds = [](long long tiles, long long units) { return (double)((tiles + units - 1) / units); };
  const bool pair_allowed = a.epilogue != EPI_BIAS_POS;    // the scatter epilogue has no pair variant
  const double cost_pair = pair_allowed ? 0.92 * rounds(tm2 * nt256, units2) : 1e30;
  const double cost_256 = 1.0 * rounds(tm1 * nt256, units1);
  const double cost_128 = 0.75 * rounds(tm1 * nt128, units1);
  bool pair = cost_pair <= cost_256 && cost_pair <= cost_128;
  bool wide = pair || cost_256 <= cost_128;
  switch (a.tiling) {
    case TILING_AUTO: break;
    case TILING_128x128: pair = false; wide = false; break;
    case TILING_128x256: pair = false; wide = true; break;
    case TILING_PAIR_256x256:
      if (!pair_allowed) return cudaErrorInvalidValue;
      pair = true; wide = true; break;
    default: return cudaErrorInvalidValue;
  }
  const int tiles_m = (int)(pair ? tm2 : tm1);
  const int bn = wide ? 256 : 128;
  TcParams p;
  p.M = a.M; p.N = a.N; p.K = a.K;
  p.bias = a.bias;
  p.residual = static_cast<const bf16*>(a.residual);
  p.pos = a.pos;
  p.ln_stats = a.ln_stats;
  p.ln_c1 = a.ln_c1;
  if ((a.epilogue == EPI_LN_BIAS || a.epilogue == EPI_LN_BIAS_GELU) && (!a.ln_stats || !a.ln_c1)) return cudaErrorInvalidValue;
  p.n_patches = a.n_patches > 0 ? a.n_patches : 1;
  p.first_patch_token = a.first_patch_token > 0 ? a.first_patch_token : 1;
  p.out = static_cast<bf16*>(a.out);
  p.ldo = a.ldo;
  p.tiles_m = tiles_m;
  p.tiles_n = (a.N + bn - 1) / bn;
  p.dev_status = dev_status;
  Maps m;
  if (!encode_2d_bf16(cache, &m.a, a.a, a.M, a.K, a.lda, BM)) return cudaErrorInvalidValue;
  if (!encode_2d_bf16(cache, &m.w, a.w, a.N, a.K, a.ldw, pair ? bn / 2 : bn)) return cudaErrorInvalidValue;
  // output (and residual) tiles move as 32-row x 64-column boxes through the epilogue's staging
  if (!encode_2d_bf16(cache, &m.out, a.out, a.M, a.N, a.ldo, 32)) return cudaErrorInvalidValue;
  if (a.epilogue == EPI_BIAS_RESIDUAL) {
    if (!encode_2d_bf16(cache, &m.res, a.residual, a.M, a.N, a.ldo, 32)) return cudaErrorInvalidValue;
  } else {
    m.res = m.out;
  }
  if (pair) return launch_bn<256, 2>(a.epilogue, m, p, s);
  return wide ? launch_bn<256, 1>(a.epilogue, m, p, s) : launch_bn<128, 1>(a.epilogue, m, p, s);
}

}  // namespace vit
