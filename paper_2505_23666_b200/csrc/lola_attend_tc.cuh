// Eq. 14 on the tensor cores (bf16 mode, F = 64, d = 64 or 128) for a tile of 128 query rows of one
// unit: S = Q K^T, online softmax with one thread per row, O += P V, then the linear term
// phi(Q) H and phi(Q) . s in the same denominator.  Accumulators S and O live in tensor memory.
#pragma once
#include "lola_generic.cuh"
#include "lola_score_tc.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kAtM = 128;   // query rows per CTA
constexpr int kAtN = 128;   // keys per tile

template <int DPL>
struct AttendTcSmem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;
  static constexpr uint32_t q = 0;                           // Q [kblk][128][128B]; later phi(Q) [2][128][128B]
  static constexpr uint32_t kp = 2 * 128 * 128;              // K tile [kblk][128 keys][128B]; then P [2][128][128B]; later W^T
  static constexpr uint32_t v = kp + 2 * 128 * 128;          // V tile [kblk][128 keys][128B]; later H^T [2][d][128B]
  static constexpr uint32_t s_vec = v + 2 * 128 * 128;       // [128] fp32
  static constexpr uint32_t bars = s_vec + 512;
  static constexpr uint32_t total = bars + 64;
  static constexpr uint32_t bytes = total + 1024;
};

template <int DPL>
__global__ void __launch_bounds__(128) k_attend_tc(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  using S = AttendTcSmem<DPL>;
  constexpr int d = DPL * 32;
  constexpr int F = 64, D = 128;
  constexpr int nch = d / 8;
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  const int unit = blockIdx.y, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int nrows = L.g * c.nq;
  const int row0 = blockIdx.x * kAtM;
  const int row = row0 + tid;
  const int rtok = row % c.nq;
  float* s_vec = (float*)(sm + S::s_vec);
  uint32_t* tmem_slot = (uint32_t*)(sm + S::bars + 32);
  const uint32_t bar = sbase + S::bars;
  uint32_t phase = 0;
  bool ok = true;

  if (tid == 0) { tc::mbar_init(bar, 1); tc::mbar_init_fence(); }
  if (warp == 0) tc::tmem_alloc(tmem_slot, 256);

  // query tile -> K-major A operand
  for (int i = tid; i < kAtM * nch; i += 128) {
    int r = i / nch, ch = i % nch, rr = row0 + r;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (rr < nrows) {
      int hl = rr / c.nq, tk = rr % c.nq;
      val = *reinterpret_cast<const uint4*>((const T*)c.q + (((size_t)b * c.nq + tk) * L.Hq + h * L.g + hl) * d + ch * 8);
    }
    *reinterpret_cast<uint4*>(sm + S::q + (ch >> 3) * (128 * 128) + tc::sw128_off(r, ch & 7)) = val;
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s = tmem, tm_o = tmem + 128;
  const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;

  const int NK = c.att_g + c.att_wn + c.att_chunk;
  const int chunk0 = c.att_g + c.att_wn;
  // a causal tile's upper bound for this CTA's rows: keys beyond the newest visible one are skipped
  const float sl2 = L.scale * 1.4426950408889634f;           // scores in log2 units
  float m = 0.f, l = 0.f;                                     // m in natural units of z (stabiliser max(0, .))
  bool have_o = false;

  for (int kt = 0; kt < NK; kt += kAtN) {
    // keys and values of this tile
    for (int i = tid; i < kAtN * nch; i += 128) {
      int r = i / nch, ch = i % nch, idx = kt + r;
      uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if (idx < NK) {
        const T *kp, *vp;
        locate_att_key<T>(L, c, unit, b, h, idx, kp, vp);
        kv = *reinterpret_cast<const uint4*>(kp + ch * 8);
        vv = *reinterpret_cast<const uint4*>(vp + ch * 8);
      }
      uint32_t off = (ch >> 3) * (128 * 128) + tc::sw128_off(r, ch & 7);
      *reinterpret_cast<uint4*>(sm + S::kp + off) = kv;
      *reinterpret_cast<uint4*>(sm + S::v + off) = vv;
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    if (tid == 0) {
      tc::mma_kmajor(tm_s, sbase + S::q, 128 * 128, sbase + S::kp, 128 * 128, d, tc::make_idesc_bf16(128, 128, false, false), false);
      tc::mma_commit(bar);
    }
    ok = tc::mbar_wait(bar, phase) && ok;
    phase ^= 1;
    tc::fence_after_sync();

    // row maximum of the visible scores
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int c0 = 0; c0 < kAtN; c0 += 32) {
      float sv[32];
      tc::tmem_ld32(tm_s + lane_addr + c0, sv);
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        int idx = kt + c0 + j, ci = idx - chunk0;
        bool valid = idx < NK && (ci < 0 || ci <= rtok);
        mx = fmaxf(mx, valid ? sv[j] : -CUDART_INF_F);
      }
    }
    const float m_new = fmaxf(m, mx * L.scale);
    const float alpha = __expf(m - m_new);
    const float mb = m_new * 1.4426950408889634f;
    float lsum = 0.f;
    // probabilities -> K-major A operand over the key tile (which S no longer needs)
#pragma unroll
    for (int c0 = 0; c0 < kAtN; c0 += 32) {
      float sv[32];
      tc::tmem_ld32(tm_s + lane_addr + c0, sv);
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        int idx = kt + c0 + j, ci = idx - chunk0;
        bool valid = idx < NK && (ci < 0 || ci <= rtok);
        float p = valid ? exp2f(fmaf(sv[j], sl2, -mb)) : 0.f;
        p = round_bf16f(p);                                   // the sum uses the weights the product uses
        lsum += p;
        sv[j] = p;
      }
#pragma unroll
      for (int q8 = 0; q8 < 4; ++q8) {
        int ch = (c0 >> 3) + q8;
        *reinterpret_cast<uint4*>(sm + S::kp + (ch >> 3) * (128 * 128) + tc::sw128_off(tid, ch & 7)) = tc::pack8_bf16(sv + q8 * 8);
      }
    }
    l = l * alpha + lsum;
    m = m_new;
    // rescale the running output where some row's maximum moved
    if (have_o && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
      for (int c0 = 0; c0 < d; c0 += 32) {
        float ov[32];
        tc::tmem_ld32(tm_o + lane_addr + c0, ov);
#pragma unroll
        for (int j = 0; j < 32; ++j) ov[j] *= alpha;
        tc::tmem_st32(tm_o + lane_addr + c0, ov);
      }
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    if (tid == 0) {
      tc::mma_a_kmajor_b_mnmajor(tm_o, sbase + S::kp, 128 * 128, sbase + S::v, 128 * 128, kAtN,
                                 tc::make_idesc_bf16(128, d, false, true), have_o);
      tc::mma_commit(bar);
    }
    ok = tc::mbar_wait(bar, phase) && ok;
    phase ^= 1;
    tc::fence_after_sync();
    have_o = true;
  }

  // ---- linear term: U = Q W, phi(Q), L = phi(Q) H
  {
    const T* Wh = (const T*)L.W + (size_t)h * d * F;
    for (int i = tid; i < d * F; i += 128) {
      int j = i / F, f = i % F;
      *reinterpret_cast<T*>(sm + S::kp + (j >> 6) * (64 * 128) + tc::sw128_off(f, (j & 63) >> 3) + (j & 7) * 2) = Wh[i];
    }
    const float* Hu = L.H + (size_t)unit * D * d;
    for (int i = tid; i < D * d; i += 128) {
      int j = i / d, cc = i % d;
      *reinterpret_cast<T*>(sm + S::v + (j >> 6) * (d * 128) + tc::sw128_off(cc, (j & 63) >> 3) + (j & 7) * 2) =
          __float2bfloat16_rn(Hu[i]);
    }
    if (tid < D) s_vec[tid] = L.s[(size_t)unit * D + tid];
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    tc::mma_kmajor(tm_s, sbase + S::q, 128 * 128, sbase + S::kp, 64 * 128, d, tc::make_idesc_bf16(128, 64, false, false), false);
    tc::mma_commit(bar);
  }
  ok = tc::mbar_wait(bar, phase) && ok;
  phase ^= 1;
  tc::fence_after_sync();
  float lden = 0.f;
  {
    float u0[32], u1[32];
    tc::tmem_ld32(tm_s + lane_addr, u0);
    tc::tmem_ld32(tm_s + lane_addr + 32, u1);
    float f[128];
    phi_from_u64(u0, u1, L.phi_kind, f);
#pragma unroll
    for (int j = 0; j < 128; ++j) lden = fmaf(f[j], s_vec[j], lden);
#pragma unroll
    for (int ch = 0; ch < 16; ++ch)
      *reinterpret_cast<uint4*>(sm + S::q + (ch >> 3) * (128 * 128) + tc::sw128_off(tid, ch & 7)) = tc::pack8_bf16(f + ch * 8);
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    tc::mma_kmajor(tm_s, sbase + S::q, 128 * 128, sbase + S::v, d * 128, D, tc::make_idesc_bf16(128, d, false, false), false);
    tc::mma_commit(bar);
  }
  ok = tc::mbar_wait(bar, phase) && ok;
  phase ^= 1;
  tc::fence_after_sync();

  {
    const float e = (c.att_flags & 1) ? 0.f : __expf(-m);       // (0: the queries do not see H, s)
    const float inv = 1.0f / fmaf(e, lden, l);
    T* op = nullptr;
    if (row < nrows) {
      int hl = row / c.nq;
      op = (T*)c.out + (((size_t)b * c.nq + rtok) * L.Hq + h * L.g + hl) * d;
    }
#pragma unroll
    for (int c0 = 0; c0 < d; c0 += 32) {
      float lv[32], ov[32];
      tc::tmem_ld32(tm_s + lane_addr + c0, lv);
      if (have_o) tc::tmem_ld32(tm_o + lane_addr + c0, ov);
#pragma unroll
      for (int j = 0; j < 32; ++j) lv[j] = (fmaf(e, lv[j], have_o ? ov[j] : 0.f)) * inv;
      if (op && ok) {
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8) *reinterpret_cast<uint4*>(op + c0 + q8 * 8) = tc::pack8_bf16(lv + q8 * 8);
      }
    }
  }
  if (!ok && tid == 0) atomicOr(L.status, 4);
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 256);
}

}  // namespace lola
