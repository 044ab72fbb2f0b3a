// Eq. 10 on the tensor cores (bf16 mode, F = 64 so D = 128, d = 64 or 128).
// One CTA scores 128 members of the eligible set:
//   U = K_E W           tcgen05.mma  M=128, N=64,  K=d     (accumulator in tensor memory)
//   phi = [softmax(U), softmax(-U)] in registers, one thread per row, rounded to bf16
//   P = phi H           tcgen05.mma  M=128, N=d,   K=128
//   score = || P / (phi . s) - v ||_2
#pragma once
#include "lola_generic.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kScTile = 128;

template <int DPL>
struct ScoreTcSmem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;                       // 64-wide K blocks of the key tile
  static constexpr uint32_t a_k = 0;                        // [kblk][128 rows][128 B]
  static constexpr uint32_t a_phi = 0;                      // [2][128 rows][128 B]; reuses the key tile once U is done
  static constexpr uint32_t b_w = 2 * 128 * 128;            // W^T: [kblk][64 rows (f)][128 B]
  static constexpr uint32_t b_h = b_w + kblk * 64 * 128;    // H^T: [2][d rows (c)][128 B]
  static constexpr uint32_t s_vec = b_h + 2 * d * 128;      // [128] fp32
  static constexpr uint32_t bars = s_vec + 128 * 4;         // 2 mbarriers + tmem slot
  static constexpr uint32_t total = bars + 64;
  static constexpr uint32_t bytes = total + 1024;           // slack to align the base to 1024
};

// phi of one row from its 64 pre-activations (thread-local), written as bf16-rounded floats.
__device__ __forceinline__ void phi_from_u64(const float (&u0)[32], const float (&u1)[32], int kind, float* f /*[128]*/) {
  if (kind == 1) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      f[i] = expf(u0[i]); f[32 + i] = expf(u1[i]);
      f[64 + i] = expf(-u0[i]); f[96 + i] = expf(-u1[i]);
    }
  } else {
    float mx = -CUDART_INF_F, mn = CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      mx = fmaxf(mx, fmaxf(u0[i], u1[i]));
      mn = fminf(mn, fminf(u0[i], u1[i]));
    }
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      f[i] = expf(u0[i] - mx); f[32 + i] = expf(u1[i] - mx);
      f[64 + i] = expf(mn - u0[i]); f[96 + i] = expf(mn - u1[i]);
    }
    // same summation order as a sequential pass over the 64 entries is not required: fp32 sums of
    // positive terms, relative error ~1e-7
#pragma unroll
    for (int i = 0; i < 64; ++i) { s1 += f[i]; s2 += f[64 + i]; }
#pragma unroll
    for (int i = 0; i < 64; ++i) { f[i] = f[i] / s1; f[64 + i] = f[64 + i] / s2; }
  }
#pragma unroll
  for (int i = 0; i < 128; ++i) f[i] = round_bf16f(f[i]);
}

template <int DPL>
__global__ void __launch_bounds__(128) k_score_tc(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  using S = ScoreTcSmem<DPL>;
  constexpr int d = DPL * 32;
  constexpr int F = 64, D = 128;
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  const int unit = blockIdx.y, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int nE = c.count_g + c.r;
  const int e0 = blockIdx.x * kScTile;
  float* s_vec = (float*)(sm + S::s_vec);
  uint64_t* bars = (uint64_t*)(sm + S::bars);
  uint32_t* tmem_slot = (uint32_t*)(sm + S::bars + 32);
  const uint32_t bar0 = sbase + S::bars, bar1 = bar0 + 8;

  if (tid == 0) { tc::mbar_init(bar0, 1); tc::mbar_init(bar1, 1); tc::mbar_init_fence(); }
  if (warp == 0) tc::tmem_alloc(tmem_slot, 256);

  // key tile -> K-major swizzled A operand (16-byte chunks)
  {
    constexpr int nch = d / 8;                                   // chunks per row
    for (int i = tid; i < kScTile * nch; i += 128) {
      int r = i / nch, ch = i % nch, e = e0 + r;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (e < nE) {
        const T *kp, *vp;
        locate_eligible<T>(L, c, unit, b, h, e, kp, vp);
        val = *reinterpret_cast<const uint4*>(kp + ch * 8);
      }
      *reinterpret_cast<uint4*>(sm + S::a_k + (ch >> 3) * (128 * 128) + tc::sw128_off(r, ch & 7)) = val;
    }
  }
  // W^T -> K-major B operand: row f, K index j
  {
    const T* Wh = (const T*)L.W + (size_t)h * d * F;
    for (int i = tid; i < d * F; i += 128) {
      int j = i / F, f = i % F;
      *reinterpret_cast<T*>(sm + S::b_w + (j >> 6) * (64 * 128) + tc::sw128_off(f, (j & 63) >> 3) + (j & 7) * 2) = Wh[i];
    }
  }
  // H^T (rounded to bf16) -> K-major B operand: row c, K index j
  {
    const float* Hu = L.H + (size_t)unit * D * d;
    for (int i = tid; i < D * d; i += 128) {
      int j = i / d, cc = i % d;
      *reinterpret_cast<T*>(sm + S::b_h + (j >> 6) * (d * 128) + tc::sw128_off(cc, (j & 63) >> 3) + (j & 7) * 2) =
          __float2bfloat16_rn(Hu[i]);
    }
  }
  if (tid < D) s_vec[tid] = L.s[(size_t)unit * D + tid];
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_u = tmem, tm_p = tmem + 64;

  if (tid == 0) {
    tc::mma_kmajor(tm_u, sbase + S::a_k, 128 * 128, sbase + S::b_w, 64 * 128, d, tc::make_idesc_bf16(128, 64, false, false), false);
    tc::mma_commit(bar0);
  }
  bool ok = tc::mbar_wait(bar0, 0);
  tc::fence_after_sync();

  // one thread per row: feature map, normaliser, A operand of the second product
  float den = 0.f;
  {
    float u0[32], u1[32];
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
    tc::tmem_ld32(tm_u + lane_addr, u0);
    tc::tmem_ld32(tm_u + lane_addr + 32, u1);
    float f[128];
    phi_from_u64(u0, u1, L.phi_kind, f);
#pragma unroll
    for (int j = 0; j < 128; ++j) den = fmaf(f[j], s_vec[j], den);
#pragma unroll
    for (int ch = 0; ch < 16; ++ch)
      *reinterpret_cast<uint4*>(sm + S::a_phi + (ch >> 3) * (128 * 128) + tc::sw128_off(tid, ch & 7)) = tc::pack8_bf16(f + ch * 8);
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    tc::mma_kmajor(tm_p, sbase + S::a_phi, 128 * 128, sbase + S::b_h, d * 128, D, tc::make_idesc_bf16(128, d, false, false), false);
    tc::mma_commit(bar1);
  }
  ok = tc::mbar_wait(bar1, 0) && ok;
  tc::fence_after_sync();

  {
    const int e = e0 + tid;
    const T *kp = nullptr, *vp = nullptr;
    if (e < nE) locate_eligible<T>(L, c, unit, b, h, e, kp, vp);
    const float inv = den > 0.f ? 1.0f / den : 0.f;
    float ss = 0.f;
    const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
#pragma unroll
    for (int c0 = 0; c0 < d; c0 += 32) {
      float p[32];
      tc::tmem_ld32(tm_p + lane_addr + c0, p);                   // warp-collective: outside the row guard
      if (e < nE) {
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8) {
          uint4 raw = *reinterpret_cast<const uint4*>(vp + c0 + q8 * 8);
          const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            float2 vv = __bfloat1622float2(v2[t]);
            float d0 = (den > 0.f ? p[q8 * 8 + 2 * t] / den : 0.f) - vv.x;
            float d1 = (den > 0.f ? p[q8 * 8 + 2 * t + 1] / den : 0.f) - vv.y;
            ss = fmaf(d0, d0, ss);
            ss = fmaf(d1, d1, ss);
          }
        }
      }
    }
    (void)inv;
    if (e < nE && ok) {
      size_t o = (size_t)unit * (L.lam + L.cmax) + (e < c.count_g ? e : L.lam + (e - c.count_g));
      L.score[o] = sqrtf(ss);
    }
  }
  if (!ok && tid == 0) atomicOr(L.status, 2);
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 256);
}

}  // namespace lola
