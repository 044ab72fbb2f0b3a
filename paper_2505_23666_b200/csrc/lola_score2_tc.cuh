// Eq. 10 for the chunkwise update (bf16 layer, F = 64): the self-recall error of every member of the
// sparse cache and of every pair leaving the window, against the H, s before the fold.
//
// Rows are streamed by TMA in tiles of 128: sparse-cache slots 0..count_g-1 (count_g a multiple of
// 64), then the window ring slots 0..eta-1.  One CTA takes `tiles_per_cta` consecutive tiles of one
// unit; its two row groups of 256 threads (two threads per row) work on alternate tiles:
//     U = K_tile W                        tcgen05.mma  M=128, N=64,   K=d
//     phi = feature map of U, rounded to bf16, kept in tensor memory (A operand of the next product)
//     [P | den] = phi [H | s_hi s_lo]      tcgen05.mma  M=128, N=d+16, K=128
//     score = || P / den - v ||
// Ring rows whose pair stays in the window are computed and dropped.
// Every wait on an mbarrier is bounded; a wait that runs out sets bit 16 of the status word.
#pragma once
#include <cuda.h>

#include "lola_decode_tc.cuh"
#include "lola_update2_tc.cuh"
#include "lola_generic.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kSc2Threads = 512;

template <int DPL>
struct Score2Smem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;
  static constexpr uint32_t b1 = 0;                                  // W^T, K-major: [kblk][64][128B]
  static constexpr uint32_t ht_blk = (d + 16) * 128;
  static constexpr uint32_t ht = 16384;                              // [2 j blocks][d + 16 rows][128B]
  static constexpr uint32_t stage0 = ht + 2 * (128 + 16) * 128;
  static constexpr uint32_t st_k = 0, st_v = 32768;
  static constexpr uint32_t stage_bytes = 65536;
  static constexpr uint32_t misc = stage0 + 2 * stage_bytes;
  static constexpr uint32_t total = misc + 2048;
  static constexpr uint32_t bytes = total + 1024;
};

struct Score2Misc {
  float ssp[2][128];
  uint64_t bars[8];
  uint32_t tmem_slot;
};

template <int DPL>
__global__ void __launch_bounds__(kSc2Threads, 1)
k_score2_tc(Layer L, Call c, const __grid_constant__ CUtensorMap tm_gk, const __grid_constant__ CUtensorMap tm_gv,
            const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv, const uint4* wt_image,
            int tiles_per_cta, int beside_attention) {
  using S = Score2Smem<DPL>;
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  constexpr int d = DPL * 32;
  constexpr int kblk = d / 64;
  constexpr int D = 128;
  constexpr int HC = d / 2;
  constexpr float kLog2e = 1.4426950408889634f;
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  Score2Misc& X = *reinterpret_cast<Score2Misc*>(sm + S::misc);

  const int unit = blockIdx.y, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wg = tid >> 8, wq = warp & 3, hf = (warp >> 2) & 1;
  const int t = wq * 32 + lane;
  const bool lead = (tid & 255) == 0;
  const int lam = L.lam, eta = L.eta;
  const int cg = c.count_g;                                // multiple of 64
  const int nGB = cg / 64, nRB = (eta + 63) / 64, NT = (nGB + nRB + 1) / 2;
  const int tile0 = blockIdx.x * tiles_per_cta;
  const int tile1 = min(NT, tile0 + tiles_per_cta);
  const int cw = min(eta, c.n_seen);                       // pairs in the window before this call
  const int w0 = c.n_seen - cw;                            // oldest position in the window
  float* scu = L.score + (size_t)unit * (lam + L.cmax);

  const uint32_t bar_k = sbase + S::misc + (uint32_t)offsetof(Score2Misc, bars) + (uint32_t)wg * 24u;
  const uint32_t bar_v = bar_k + 8, bar_mma = bar_k + 16;
  const uint32_t bar_u = sbase + S::misc + (uint32_t)offsetof(Score2Misc, bars) + 48u + (uint32_t)wg * 8u;
  const uint32_t stage = sbase + S::stage0 + (uint32_t)wg * S::stage_bytes;
  uint8_t* stage_p = sm + S::stage0 + (size_t)wg * S::stage_bytes;
  uint32_t pk = 0, pv = 0, pm = 0, pu = 0;
  bool ok = true;

  if (tid == 0) {
    for (int i = 0; i < 8; ++i) tc::mbar_init(sbase + S::misc + (uint32_t)offsetof(Score2Misc, bars) + 8u * i, 1);
    tc::mbar_init_fence();
  }
  if (warp == 0) tc::tmem_alloc(&X.tmem_slot, 512);
  __syncthreads();
  // Launched as a programmatic dependent, this kernel may be resident while the kernel before it still runs.
  // beside_attention: that kernel is the attention kernel of the same call, which only reads the memories and has
  // let this one start after seeing everything before it complete: nothing to wait for here; every block waits
  // for it at its end instead, so that whatever follows this kernel follows both.
  if (!beside_attention) tc::grid_dep_wait();
  if (tid == 0) tc::grid_dep_launch_dependents();
  if (lead && tile0 + wg < tile1) {
    decode_issue_tile<DPL>(stage + S::st_k, &tm_gk, &tm_wk, tile0 + wg, nGB, nRB, unit, bar_k);
    decode_issue_tile<DPL>(stage + S::st_v, &tm_gv, &tm_wv, tile0 + wg, nGB, nRB, unit, bar_v);
  }
  // ---- operands: H^T operand image (from H through registers: thread x gathers, for DPL items (column c, 8
  //      consecutive j), the eight values H[j][c]; lanes = consecutive columns, so every load of a warp is one
  //      128-byte line), the two parts of s as rows d, d+1, W^T image
  {
    float pre_h[DPL][8];
    const float* Hg = L.H + (size_t)unit * D * d;
#pragma unroll
    for (int n = 0; n < DPL; ++n) {
      const int it = tid + kSc2Threads * n, cc = it % d, jc = it / d;
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) pre_h[n][jj] = Hg[(size_t)(jc * 8 + jj) * d + cc];
    }
    const uint4* img = wt_image + (size_t)h * kblk * 512;
    for (int i = tid; i < kblk * 512; i += kSc2Threads)
      *reinterpret_cast<uint4*>(sm + S::b1 + i * 16) = img[i];
    if (tid < D) {
      const float sv = L.s[(size_t)unit * D + tid];
      const __nv_bfloat16 hi = __float2bfloat16_rn(sv);
      const __nv_bfloat16 lo = __float2bfloat16_rn(sv - __bfloat162float(hi));
      const int ch = (tid & 63) >> 3;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d, ch) + (tid & 7) * 2) = hi;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d + 1, ch) + (tid & 7) * 2) = lo;
    }
    for (int i = tid; i < 2 * 14 * 8; i += kSc2Threads) {
      const int jb = i / (14 * 8), r = (i / 8) % 14, ch = i % 8;
      *reinterpret_cast<uint4*>(sm + S::ht + jb * S::ht_blk + tc::sw128_off(d + 2 + r, ch)) = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int n = 0; n < DPL; ++n) {
      const int it = tid + kSc2Threads * n, cc = it % d, jc = it / d;
      *reinterpret_cast<uint4*>(sm + S::ht + (jc >> 3) * S::ht_blk + tc::sw128_off(cc, jc & 7)) = tc::pack8_bf16(pre_h[n]);
    }
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = X.tmem_slot;
  const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
  const uint32_t tm_a = tmem + (uint32_t)wg * 256u;            // [P | den]
  const uint32_t tm_phi = tm_a + 192u;                         // U = K W of a tile, then its feature map in place (bf16 pairs)
  const uint32_t idesc1 = tc::make_idesc_bf16(128, 64, false, false);
  const uint32_t idesc2 = tc::make_idesc_bf16(128, d + 16, false, false);
  // operand descriptors once; a K step adds its byte offset / 16 to the address field
  const uint64_t dk = tc::make_desc_sw128(stage + S::st_k, 16, 1024), db1 = tc::make_desc_sw128(sbase + S::b1, 16, 1024),
                 dht = tc::make_desc_sw128(sbase + S::ht, 16, 1024);

  // U = K W of a tile is issued one tile ahead: right behind [P | den] of the tile before (the tensor pipe runs
  // in order, so the feature map there is consumed first), and runs while the row group works on Eq. 10
  auto issue_u = [&]() {
    ok = tc::mbar_wait(bar_k, pk) && ok; pk ^= 1;
    tc::fence_after_sync();
#pragma unroll
    for (int ks = 0; ks < d / 16; ++ks)
      tc::mma_bf16_ss(tm_phi, dk + (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                      db1 + (uint64_t)(((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), idesc1, ks > 0);
    tc::mma_commit(bar_u);
  };
  if (lead && tile0 + wg < tile1) issue_u();
  if (wg == 1) asm volatile("bar.arrive 3, 512;" ::: "memory");   // row group 0 takes the first turn

  for (int tile = tile0 + wg; tile < tile1; tile += 2) {
    const int R = tile * 128 + t;
    const bool is_g = R < cg;
    const int slot = R - cg;
    // ring slot -> position it holds; it is scored if that pair leaves the window in this call
    int e_idx = -1;
    if (is_g) e_idx = R;
    else if (slot < eta) {
      int off = slot - (w0 % eta);
      if (off < 0) off += eta;
      const int p = w0 + off;
      if (off < cw && p < c.r_pos0 + c.r && p >= c.r_pos0) e_idx = lam + (p - c.r_pos0);
    }

    ok = tc::mbar_wait(bar_u, pu) && ok; pu ^= 1;     // U of this tile is complete (and the key tile is read)
    tc::fence_after_sync();
    if (lead && tile + 2 < tile1) decode_issue_tile<DPL>(stage + S::st_k, &tm_gk, &tm_wk, tile + 2, nGB, nRB, unit, bar_k);
    {
      tc::named_bar_sync(3 + wg, 512);
      uint32_t u[64], pk2[32];
      tc::tmem_ld64u(tm_phi + lane_addr, u);
      tc::phi_half(u, hf != 0, L.phi_kind == 1, pk2);
      tc::fence_before_sync();
      tc::named_bar_sync(1 + wg, 256);               // both threads of a row have read U: its columns take the feature map
      tc::tmem_st32u(tm_phi + lane_addr + hf * 32, pk2);
      if (wg == 0) asm volatile("bar.arrive 4, 512;" ::: "memory"); else asm volatile("bar.arrive 3, 512;" ::: "memory");
    }
    tc::fence_before_sync();
    tc::named_bar_sync(1 + wg, 256);
    tc::fence_after_sync();
    if (lead) {
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ts(tm_a, tm_phi + ks * 8, dht + (uint64_t)(((ks >> 2) * S::ht_blk + (ks & 3) * 32) >> 4), idesc2, ks > 0);
      tc::mma_commit(bar_mma);
      if (tile + 2 < tile1) issue_u();               // U of this row group's next tile
    }
    ok = tc::mbar_wait(bar_v, pv) && ok; pv ^= 1;
    ok = tc::mbar_wait(bar_mma, pm) && ok; pm ^= 1;
    tc::fence_after_sync();
    {
      float dn[2];
      tc::tmem_ld2(tm_a + lane_addr + d, dn);
      const float den = dn[0] + dn[1];
      const float inv = den > 0.f ? 1.0f / den : 0.f;
      // packed pairs: d = v - P / den, four running sums of squares (columns 4k, 4k+1 | 4k+2, 4k+3)
      const uint64_t ninv2 = tc::pack_f2(-inv, -inv);
      uint64_t accA = tc::pack_f2(0.f, 0.f), accB = accA;
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        uint32_t p[32];
        tc::tmem_ld32u(tm_a + lane_addr + hf * HC + c0, p);
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8) {
          const int cc = hf * HC + c0 + q8 * 8;
          const uint4 raw = *reinterpret_cast<const uint4*>(stage_p + S::st_v + (cc >> 6) * 16384 + tc::sw128_off(t, (cc & 63) >> 3));
          const uint64_t d01 = tc::fma2(tc::pack_u2(p[q8 * 8 + 0], p[q8 * 8 + 1]), ninv2, tc::pack_u2(raw.x << 16, raw.x & 0xffff0000u));
          const uint64_t d23 = tc::fma2(tc::pack_u2(p[q8 * 8 + 2], p[q8 * 8 + 3]), ninv2, tc::pack_u2(raw.y << 16, raw.y & 0xffff0000u));
          const uint64_t d45 = tc::fma2(tc::pack_u2(p[q8 * 8 + 4], p[q8 * 8 + 5]), ninv2, tc::pack_u2(raw.z << 16, raw.z & 0xffff0000u));
          const uint64_t d67 = tc::fma2(tc::pack_u2(p[q8 * 8 + 6], p[q8 * 8 + 7]), ninv2, tc::pack_u2(raw.w << 16, raw.w & 0xffff0000u));
          accA = tc::fma2(d01, d01, accA);
          accB = tc::fma2(d23, d23, accB);
          accA = tc::fma2(d45, d45, accA);
          accB = tc::fma2(d67, d67, accB);
        }
      }
      float a0, a1, a2, a3;
      tc::unpack_f2(accA, a0, a1);
      tc::unpack_f2(accB, a2, a3);
      const float ss = (a0 + a1) + (a2 + a3);
      if (hf == 1) X.ssp[wg][t] = ss;
      tc::fence_async_smem();
      tc::fence_before_sync();
      tc::named_bar_sync(1 + wg, 256);          // both halves are done with the value tile and with P
      tc::fence_after_sync();
      if (hf == 0 && e_idx >= 0 && ok) scu[e_idx] = sqrtf(ss + X.ssp[wg][t]);
    }
    if (lead && tile + 2 < tile1) decode_issue_tile<DPL>(stage + S::st_v, &tm_gv, &tm_wv, tile + 2, nGB, nRB, unit, bar_v);
  }
  if (!ok && (tid & 255) == 0) atomicOr(L.status, 16);
  tc::fence_before_sync();
  __threadfence();                                   // this block's scores are visible before it counts itself
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
  // ---- the last block of a unit to finish selects the pairs to fold (Eq. 12) from all the unit's scores
  __shared__ int is_last;
  if (gridDim.x == 1) {                              // one block per unit: it has all the unit's scores
    update2_body<DPL, 1>(L, c, wt_image, nullptr, sm, unit);
    if (beside_attention) tc::grid_dep_wait();
    return;
  }
  if (tid == 0) {
    int* arrived = L.counts + (size_t)unit * 4 + 2;
    const int prev = atomicAdd(arrived, 1);
    is_last = prev == (int)gridDim.x - 1;
    if (is_last) *arrived = 0;                       // ready for the next call
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    update2_body<DPL, 1>(L, c, wt_image, nullptr, sm, unit);
  }
  if (beside_attention) tc::grid_dep_wait();
}

}  // namespace lola
