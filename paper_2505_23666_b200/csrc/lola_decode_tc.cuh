// The generation step (Eq. 11-14) as ONE kernel for the steady state of a bf16 layer with F = 64:
// caches full, exactly one pair leaves the window per step.  One CTA per (batch row, KV head) unit;
// the unit's memories are streamed once from HBM by TMA and everything that depends on them is
// computed on the way:
//
//   rows of the stream = sparse-cache slots 0..lambda-1, then the window ring slots 0..eta-1, in
//   tiles of 128 rows.  Two row groups of 256 threads work on alternate tiles (two threads per row:
//   one per half of the feature map / half of the value columns), so that one group's arithmetic
//   overlaps the other's loads and MMAs.  Per tile:
//     [U | Z] = K_tile [W | Q^T]          tcgen05.mma  M=128, N=80,   K=d   (pre-activations, q.k)
//     phi = feature map of U, rounded to bf16
//     [P | den] = phi [H | s_hi s_lo]      tcgen05.mma  M=128, N=d+16, K=128 (s split in two bf16 parts)
//     score = || P / den - v ||            for sparse-cache rows and the evicted pair (Eq. 10)
//     O^T += V_tile^T Pr^T                 tcgen05.mma  M=d(128), N=16, K=128 (Eq. 14 numerator),
//                                          Pr = exp(z - m) with a running maximum per query row
//   The pair to fold (Eq. 12: lowest score, ties: the younger pair) is only known after the last
//   tile, and it must not be attended.  So every tile leaves its own lowest-scored row out of O^T and
//   keeps that row's q.k, value and feature row in a small list; at the end the overall lowest is
//   folded (Eq. 13: H += phi v^T, s += phi) and the other list entries are added back.
//   The linear term uses the state after the fold: phi(q)^T H_old (an MMA that initialises O^T with
//   weight exp(0 - m), the m = max(0, .) stabiliser) plus (phi(q) . phi_fold) v_fold.
//
// Every wait on an mbarrier is bounded; a wait that runs out sets bit 8 of the status word.
#pragma once
#include <cuda.h>

#include "lola_generic.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kDecQ = 8;          // query rows per unit the kernel carries (group size g <= 8)
constexpr int kDecMaxTiles = 16;  // (lambda + eta rounded up to 64) / 128 <= 16
constexpr int kDecThreads = 512;  // two row groups of 256

template <int DPL>
struct DecodeSmem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;
  static constexpr uint32_t b1_blk = 80 * 128;                       // one K block of [W^T ; Q]: 80 rows
  static constexpr uint32_t b1 = 0;                                  // [kblk][80][128B]
  static constexpr uint32_t ht_blk = (d + 16) * 128;                 // one j block of [H^T ; s_hi ; s_lo ; ...]
  static constexpr uint32_t ht = 2 * b1_blk;                         // K-major: [2 j blocks][d + 16 rows][128B]
  static constexpr uint32_t phiq = ht + 2 * (128 + 16) * 128;        // phi(Q), K-major: [2 j blocks][16][128B]
  static constexpr uint32_t stage0 = phiq + 4096;
  static constexpr uint32_t st_k = 0;                                // K tile [kblk][128][128B]
  static constexpr uint32_t st_v = 32768;                            // V tile [kblk][128 keys][128B]; at the end O^T partials
  static constexpr uint32_t st_pt = 65536;                           // Pr^T, K-major: [2 key blocks][16][128B]
  static constexpr uint32_t stage_bytes = 65536 + 4096;
  static constexpr uint32_t misc = stage0 + 2 * stage_bytes;         // small arrays, see DecodeMisc
  static constexpr uint32_t total = misc + 28672;
  static constexpr uint32_t bytes = total + 1024;                    // slack to align the base to 1024
};

// small shared arrays
struct DecodeMisc {
  float qf[kDecQ][128];          // query rows, fp32
  float phiq_f[kDecQ][128];      // phi(q) rounded to bf16, as fp32
  float u_s[kDecQ][64];
  float knew[128], vnew[128];
  float zn[kDecQ], lden[kDecQ], dotL[kDecQ];
  float redmax[2][4][kDecQ];
  unsigned long long redkey[2][4];
  float red12[2][4][2];
  float ssp[2][128];             // partial squared errors of the second half of the value columns
  float wg_m[2][kDecQ];
  float wg_l[2][8][kDecQ];
  // per-tile list of the rows left out of O^T
  unsigned long long cand_key[kDecMaxTiles];
  float cand_score[kDecMaxTiles], cand_min2[kDecMaxTiles];
  int cand_row[kDecMaxTiles];
  float cand_z[kDecMaxTiles][kDecQ];
  uint4 cand_v[kDecMaxTiles][16];    // value row, bf16
  uint4 cand_phi[kDecMaxTiles][16];  // feature row, bf16
  uint64_t bars[12];
  uint32_t tmem_slot;
};
static_assert(sizeof(DecodeMisc) <= 28672, "misc region too small");

__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long x, int o) {
  unsigned lo = __shfl_xor_sync(0xffffffffu, (unsigned)x, o);
  unsigned hi = __shfl_xor_sync(0xffffffffu, (unsigned)(x >> 32), o);
  return ((unsigned long long)hi << 32) | lo;
}

// warp-wide maximum / minimum of fp32 values through the integer reduction instruction
__device__ __forceinline__ int f2ord(float x) { int i = __float_as_int(x); return i ^ ((i >> 31) & 0x7fffffff); }
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }
__device__ __forceinline__ float warp_max_redux(float x) { return ord2f(__reduce_max_sync(0xffffffffu, f2ord(x))); }

// two fp32 -> packed bf16x2 (a in the low half), and the rounded values back as fp32 by bit moves
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float bf16lo_f(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16hi_f(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// Loads of one tile: two half tiles of 64 rows; a half tile is a block of sparse-cache slots, a block
// of ring slots, or nothing (a box that lies entirely outside the ring tensor reads as zeros).
template <int DPL>
__device__ __forceinline__ void decode_issue_tile(uint32_t dst, const CUtensorMap* tm_g, const CUtensorMap* tm_w, int tile,
                                                  int nGB, int nRB, int unit, uint32_t bar) {
  constexpr int kblk = DPL / 2;
  tc::mbar_expect_tx(bar, (uint32_t)kblk * 16384u);
#pragma unroll
  for (int hb = 0; hb < 2; ++hb) {
    const int blk = tile * 2 + hb;
    const bool from_g = blk < nGB;
    const CUtensorMap* tm = from_g ? tm_g : tm_w;
    const int row = from_g ? blk * 64 : min(blk - nGB, nRB) * 64;
#pragma unroll
    for (int cb = 0; cb < kblk; ++cb)
      tc::tma_load_3d(dst + (uint32_t)cb * 16384u + (uint32_t)hb * 8192u, tm, cb * 64, row, unit, bar);
  }
}

template <int DPL, int QR>
__global__ void __launch_bounds__(kDecThreads, 1)
k_decode_tc(Layer L, Call c, const __grid_constant__ CUtensorMap tm_gk, const __grid_constant__ CUtensorMap tm_gv,
            const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv, const uint4* wt_image) {
  using S = DecodeSmem<DPL>;
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  constexpr int d = DPL * 32;
  constexpr int kblk = d / 64;
  constexpr int F = 64, D = 128;
  constexpr int HC = d / 2;                  // value columns per thread of a row pair
  constexpr float kLog2e = 1.4426950408889634f;
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  DecodeMisc& X = *reinterpret_cast<DecodeMisc*>(sm + S::misc);

  const int unit = blockIdx.x, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wg = tid >> 8;                   // row group
  const int wq = warp & 3;                   // tensor-memory lane quadrant of this warp
  const int hf = (warp >> 2) & 1;            // which half of the row's work this thread does
  const int t = wq * 32 + lane;              // row of the tile = tensor-memory lane
  const bool lead = (tid & 255) == 0;        // issues the row group's TMA and MMAs
  const int lam = L.lam, eta = L.eta, g = L.g;
  const int nGB = lam / 64, nRB = (eta + 63) / 64, NT = (nGB + nRB + 1) / 2;
  const int s_ev = c.n_seen % eta;           // ring slot of the pair that leaves = slot the new pair takes
  const int pos_ev = c.n_seen - eta;
  const float sl2 = L.scale * kLog2e;        // q.k in log2 units
  float* scu = L.score + (size_t)unit * (lam + L.cmax);

  const uint32_t bar_k = sbase + S::misc + (uint32_t)offsetof(DecodeMisc, bars) + (uint32_t)wg * 32u;
  const uint32_t bar_v = bar_k + 8, bar_mma = bar_k + 16, bar_mma3 = bar_k + 24;
  const uint32_t stage = sbase + S::stage0 + (uint32_t)wg * S::stage_bytes;
  uint8_t* stage_p = sm + S::stage0 + (size_t)wg * S::stage_bytes;
  uint32_t pk = 0, pv = 0, pm = 0, pm3 = 0;
  bool ok = true;

  if (tid == 0) {
    for (int i = 0; i < 10; ++i) tc::mbar_init(sbase + S::misc + (uint32_t)offsetof(DecodeMisc, bars) + 8u * i, 1);
    tc::mbar_init_fence();
  }
  if (warp == 0) tc::tmem_alloc(&X.tmem_slot, 512);
  __syncthreads();
  // first tile of each row group starts to stream while the operands below are prepared
  // H (fp32, 64 KB at d = 128) comes in by two bulk copies into the two value buffers, which the first
  // value tiles only need later; W^T by bulk copies straight into the operand rows
  const uint32_t bar_h = sbase + S::misc + (uint32_t)offsetof(DecodeMisc, bars) + 64u;
  const uint32_t bar_w = bar_h + 8u;
  if (tid == 0) {
    const float* Hg = L.H + (size_t)unit * D * d;
    tc::mbar_expect_tx(bar_h, (uint32_t)(D * d * 4));
    tc::bulk_copy_g2s(sbase + S::stage0 + S::st_v, Hg, 64u * d * 4u, bar_h);
    tc::bulk_copy_g2s(sbase + S::stage0 + S::stage_bytes + S::st_v, Hg + 64 * d, 64u * d * 4u, bar_h);
    tc::mbar_expect_tx(bar_w, (uint32_t)kblk * 8192u);
    for (int kb = 0; kb < kblk; ++kb)
      tc::bulk_copy_g2s(sbase + S::b1 + (uint32_t)kb * S::b1_blk, wt_image + ((size_t)h * kblk + kb) * 512, 8192u, bar_w);
  }
  if (lead && wg < NT) decode_issue_tile<DPL>(stage + S::st_k, &tm_gk, &tm_wk, wg, nGB, nRB, unit, bar_k);

  // ---- operands that stay for the whole unit
  {
    // rows d, d+1: s as the sum of two bf16 parts (phi . s_hi + phi . s_lo keeps the fp32 normaliser)
    if (tid < D) {
      const float sv = L.s[(size_t)unit * D + tid];
      const __nv_bfloat16 hi = __float2bfloat16_rn(sv);
      const __nv_bfloat16 lo = __float2bfloat16_rn(sv - __bfloat162float(hi));
      const int ch = (tid & 63) >> 3;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d, ch) + (tid & 7) * 2) = hi;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d + 1, ch) + (tid & 7) * 2) = lo;
    }
    // rows d+2 .. d+15 of both j blocks: zero
    for (int i = tid; i < 2 * 14 * 8; i += kDecThreads) {
      const int jb = i / (14 * 8), r = (i / 8) % 14, ch = i % 8;
      *reinterpret_cast<uint4*>(sm + S::ht + jb * S::ht_blk + tc::sw128_off(d + 2 + r, ch)) = make_uint4(0, 0, 0, 0);
    }
    // query rows: B1 rows 64..79 (rows >= g are zero) and an fp32 copy
    constexpr int per_row = d / 8;
    for (int i = tid; i < 16 * per_row; i += kDecThreads) {
      const int r = i / per_row, ch = i % per_row;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (r < g) val = *reinterpret_cast<const uint4*>((const T*)c.q + ((size_t)b * L.Hq + h * g + r) * d + ch * 8);
      *reinterpret_cast<uint4*>(sm + S::b1 + (ch >> 3) * S::b1_blk + tc::sw128_off(64 + r, ch & 7)) = val;
      if (r < QR) {
        const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&val);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float2 ff = __bfloat1622float2(v2[q]);
          X.qf[r][ch * 8 + 2 * q] = ff.x;
          X.qf[r][ch * 8 + 2 * q + 1] = ff.y;
        }
      }
    }
    if (tid < d) {
      X.knew[tid] = ldf<T>((const T*)c.k + ((size_t)b * L.Hkv + h) * d + tid);
      X.vnew[tid] = ldf<T>((const T*)c.v + ((size_t)b * L.Hkv + h) * d + tid);
    }
    if (tid < kDecMaxTiles) { X.cand_key[tid] = ~0ull; X.cand_score[tid] = CUDART_INF_F; X.cand_min2[tid] = CUDART_INF_F; X.cand_row[tid] = 0; }
    // zero phi(Q) and both Pr^T tiles
    for (int i = tid; i < 256; i += kDecThreads) {
      *reinterpret_cast<uint4*>(sm + S::phiq + i * 16) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(sm + S::stage0 + S::st_pt + i * 16) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(sm + S::stage0 + S::stage_bytes + S::st_pt + i * 16) = make_uint4(0, 0, 0, 0);
    }
  }
  ok = tc::mbar_wait(bar_w, 0) && ok;
  __syncthreads();
  // u = q W on the CUDA cores (g rows only) from the W^T operand image
  for (int i = tid; i < g * F; i += kDecThreads) {
    const int r = i >> 6, f = i & 63;
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int ch = 0; ch < d / 8; ++ch) {
      uint4 raw = *reinterpret_cast<const uint4*>(sm + S::b1 + (ch >> 3) * S::b1_blk + tc::sw128_off(f, ch & 7));
      const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float2 ww = __bfloat1622float2(w2[q]);
        a0 = fmaf(X.qf[r][ch * 8 + 2 * q], ww.x, a0);
        a1 = fmaf(X.qf[r][ch * 8 + 2 * q + 1], ww.y, a1);
      }
    }
    X.u_s[r][f] = a0 + a1;
  }
  __syncthreads();
  // phi(q), its normaliser phi(q) . s and q . k_new
  if (warp < g) {
    const int r = warp;
    float u0 = X.u_s[r][lane], u1 = X.u_s[r][lane + 32];
    float p0, p1, n0, n1;
    if (L.phi_kind == 1) {
      p0 = expf(u0); p1 = expf(u1); n0 = expf(-u0); n1 = expf(-u1);
    } else {
      float mx = warp_max(fmaxf(u0, u1)), mn = warp_min(fminf(u0, u1));
      p0 = expf(u0 - mx); p1 = expf(u1 - mx); n0 = expf(mn - u0); n1 = expf(mn - u1);
      float s1 = warp_sum(p0 + p1), s2 = warp_sum(n0 + n1);
      p0 /= s1; p1 /= s1; n0 /= s2; n1 /= s2;
    }
    float vals[4] = {round_bf16f(p0), round_bf16f(p1), round_bf16f(n0), round_bf16f(n1)};
    int js[4] = {lane, lane + 32, 64 + lane, 96 + lane};
    float ld = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int j = js[q];
      X.phiq_f[r][j] = vals[q];
      *reinterpret_cast<T*>(sm + S::phiq + (j >> 6) * 2048 + tc::sw128_off(r, (j & 63) >> 3) + (j & 7) * 2) = __float2bfloat16_rn(vals[q]);
      ld = fmaf(vals[q], L.s[(size_t)unit * D + j], ld);
    }
    ld = warp_sum(ld);
    float zz = 0.f;
    for (int j = lane; j < d; j += 32) zz = fmaf(X.qf[r][j], X.knew[j], zz);
    zz = warp_sum(zz);
    if (lane == 0) { X.lden[r] = ld; X.zn[r] = zz * sl2; }
  }
  // H (fp32 [D][d], staged in the value buffers) -> bf16 H^T, K-major: row c, 64 j per 128-byte row, two
  // j blocks.  A thread gathers 8 consecutive j of one column c (lanes = consecutive columns: no conflicts).
  ok = tc::mbar_wait(bar_h, 0) && ok;
  for (int i = tid; i < d * (D / 8); i += kDecThreads) {
    const int cc = i % d, jc = i / d;
    const float* src = reinterpret_cast<const float*>(sm + S::stage0 + (jc >> 3) * S::stage_bytes + S::st_v) + ((jc & 7) * 8) * d + cc;
    float f8[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) f8[jj] = src[jj * d];
    *reinterpret_cast<uint4*>(sm + S::ht + (jc >> 3) * S::ht_blk + tc::sw128_off(cc, jc & 7)) = tc::pack8_bf16(f8);
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  // the value buffers are free now: the first value tiles start to stream
  if (lead && wg < NT) decode_issue_tile<DPL>(stage + S::st_v, &tm_gv, &tm_wv, wg, nGB, nRB, unit, bar_v);
  const uint32_t tmem = X.tmem_slot;
  const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
  const uint32_t tm_a = tmem + (uint32_t)wg * 256u;            // [U | Z], then [P | den]
  const uint32_t tm_o = tm_a + 160u;                            // O^T: lanes = value column, 16 columns = query rows
  const uint32_t tm_phi = tm_a + 192u;                          // phi tile, bf16 pairs: 64 columns
  const uint32_t idesc1 = tc::make_idesc_bf16(128, 80, false, false);
  const uint32_t idesc2 = tc::make_idesc_bf16(128, d + 16, false, false);
  const uint32_t idesc0 = tc::make_idesc_bf16(128, 16, false, false);
  const uint32_t idesc3 = tc::make_idesc_bf16(128, 16, true, false);

  bool have_o = false;
  if (wg == 0) {
    // O^T = H^T phi(Q)^T: the linear term enters the running sums with weight exp(0 - m), m = 0 so far
    if (lead) {
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ss(tm_o, tc::make_desc_sw128(sbase + S::ht + (ks >> 2) * S::ht_blk + (ks & 3) * 32, 16, 1024),
                        tc::make_desc_sw128(sbase + S::phiq + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024), idesc0, ks > 0);
    }
    have_o = true;
  }

  // running maxima (log2 units, uniform over the row group) and this thread's share of the sums
  // the two row groups take turns in the exponential-heavy feature-map phase (barriers 3 + wg):
  // group 1 lets group 0 go first
  if (wg == 1) asm volatile("bar.arrive 3, 512;" ::: "memory");
  float m_run[QR], lpart[QR];
#pragma unroll
  for (int r = 0; r < QR; ++r) { m_run[r] = 0.f; lpart[r] = 0.f; }

  for (int tile = wg; tile < NT; tile += 2) {
    const int R = tile * 128 + t;
    const bool is_g = R < lam;
    const int slot = R - lam;
    const bool valid = is_g || slot < eta;
    const bool scored = is_g || slot == s_ev;
    const int pos = is_g ? L.gpos[(size_t)unit * lam + R] : pos_ev;

    // ---- [U | Z] = K_tile [W | Q^T]
    ok = tc::mbar_wait(bar_k, pk) && ok; pk ^= 1;
    tc::fence_after_sync();
    if (lead) {
#pragma unroll
      for (int ks = 0; ks < d / 16; ++ks)
        tc::mma_bf16_ss(tm_a, tc::make_desc_sw128(stage + S::st_k + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                        tc::make_desc_sw128(sbase + S::b1 + (ks >> 2) * S::b1_blk + (ks & 3) * 32, 16, 1024), idesc1, ks > 0);
      tc::mma_commit(bar_mma);
    }
    ok = tc::mbar_wait(bar_mma, pm) && ok; pm ^= 1;
    tc::fence_after_sync();

    float z[QR];
    {
      float zraw[8];
      tc::tmem_ld8(tm_a + lane_addr + 64, zraw);   // 8 columns are loaded, the first QR are query rows
#pragma unroll
      for (int r = 0; r < QR; ++r) z[r] = valid ? zraw[r] * sl2 : -CUDART_INF_F;
      if (hf == 0) {
#pragma unroll
        for (int r = 0; r < QR; ++r) {
          float wm = warp_max_redux(z[r]);
          if (lane == 0) X.redmax[wg][wq][r] = wm;
        }
      }
      // this thread's half of the feature map: hf = 0: softmax(u), hf = 1: softmax(-u); in place
      tc::named_bar_sync(3 + wg, 512);
      float e[64];
      tc::tmem_ld64(tm_a + lane_addr, e);
      const float sgn = hf ? -kLog2e : kLog2e;
      if (L.phi_kind == 1) {
#pragma unroll
        for (int i = 0; i < 64; ++i) e[i] = tc::fast_exp2(e[i] * sgn);
      } else {
        float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, m2 = -CUDART_INF_F, m3 = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < 64; i += 4) {
          m0 = fmaxf(m0, e[i] * sgn); m1 = fmaxf(m1, e[i + 1] * sgn);
          m2 = fmaxf(m2, e[i + 2] * sgn); m3 = fmaxf(m3, e[i + 3] * sgn);
        }
        const float mm = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int i = 0; i < 64; i += 4) {
          e[i] = tc::fast_exp2(fmaf(e[i], sgn, -mm)); s0 += e[i];
          e[i + 1] = tc::fast_exp2(fmaf(e[i + 1], sgn, -mm)); s1 += e[i + 1];
          e[i + 2] = tc::fast_exp2(fmaf(e[i + 2], sgn, -mm)); s2 += e[i + 2];
          e[i + 3] = tc::fast_exp2(fmaf(e[i + 3], sgn, -mm)); s3 += e[i + 3];
        }
        const float inv = 1.0f / ((s0 + s1) + (s2 + s3));
#pragma unroll
        for (int i = 0; i < 64; ++i) e[i] *= inv;
      }
      // bf16 pairs into tensor memory: the A operand of the second product (K index = feature j)
      uint32_t pk2[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) pk2[i] = pack_bf16x2(e[2 * i], e[2 * i + 1]);
      tc::tmem_st32u(tm_phi + lane_addr + hf * 32, pk2);
      if (wg == 0) asm volatile("bar.arrive 4, 512;" ::: "memory"); else asm volatile("bar.arrive 3, 512;" ::: "memory");
    }
    // the key tile is consumed: the next tile of this row group starts to stream now
    if (lead && tile + 2 < NT) decode_issue_tile<DPL>(stage + S::st_k, &tm_gk, &tm_wk, tile + 2, nGB, nRB, unit, bar_k);
    tc::fence_async_smem();
    tc::fence_before_sync();
    tc::named_bar_sync(1 + wg, 256);
    tc::fence_after_sync();
    // ---- [P | den] = phi [H | s_hi s_lo]
    if (lead) {
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks)
        tc::mma_bf16_ts(tm_a, tm_phi + ks * 8,
                        tc::make_desc_sw128(sbase + S::ht + (ks >> 2) * S::ht_blk + (ks & 3) * 32, 16, 1024), idesc2, ks > 0);
      tc::mma_commit(bar_mma);
    }
    // running maximum of q.k per query row (every valid row counts, also the one that will be folded:
    // any m >= the true maximum leaves Eq. 14 unchanged)
    float m_new[QR];
#pragma unroll
    for (int r = 0; r < QR; ++r)
      m_new[r] = fmaxf(fmaxf(m_run[r], fmaxf(X.redmax[wg][0][r], X.redmax[wg][1][r])),
                       fmaxf(X.redmax[wg][2][r], X.redmax[wg][3][r]));
    // ---- softmax weights of the tile (bf16; the sums use the rounded weights): this thread's query rows.
    // Computed while the second product runs, for every valid row; the row that turns out to have the
    // tile's lowest score takes its weights back below.
    float pw[QR];
    {
      bool moved = false;
      float alpha[QR];
#pragma unroll
      for (int r = 0; r < QR; ++r) {
        alpha[r] = tc::fast_exp2(m_run[r] - m_new[r]);
        moved = moved || (m_new[r] != m_run[r]);
        lpart[r] *= alpha[r];
        m_run[r] = m_new[r];
        pw[r] = 0.f;
      }
#pragma unroll
      for (int r = 0; r < QR; ++r) {          // static indices keep z, m_new, lpart in registers
        if ((r / (QR / 2)) == hf) {
          const float p = valid ? tc::fast_exp2(z[r] - m_new[r]) : 0.f;
          const uint32_t pb = pack_bf16x2(p, 0.f);
          pw[r] = bf16lo_f(pb);
          lpart[r] += pw[r];
          *reinterpret_cast<unsigned short*>(stage_p + S::st_pt + (t >> 6) * 2048 + tc::sw128_off(r, (t & 63) >> 3) + (t & 7) * 2) = (unsigned short)pb;
        }
      }
      if (have_o && moved && hf == 0) {          // `moved` is uniform over the row group
        float ov[8];
        tc::tmem_ld8(tm_o + lane_addr, ov);
#pragma unroll
        for (int r = 0; r < QR; ++r) ov[r] *= alpha[r];
        tc::tmem_st8(tm_o + lane_addr, ov);
      }
    }

    ok = tc::mbar_wait(bar_v, pv) && ok; pv ^= 1;
    ok = tc::mbar_wait(bar_mma, pm) && ok; pm ^= 1;
    tc::fence_after_sync();
    // ---- Eq. 10: this thread's half of the value columns
    float score;
    {
      float dn[2];
      tc::tmem_ld2(tm_a + lane_addr + d, dn);
      const float den = dn[0] + dn[1];
      const float inv = den > 0.f ? 1.0f / den : 0.f;
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        float p[32];
        tc::tmem_ld32(tm_a + lane_addr + hf * HC + c0, p);
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8) {
          const int cc = hf * HC + c0 + q8 * 8;
          uint4 raw = *reinterpret_cast<const uint4*>(stage_p + S::st_v + (cc >> 6) * 16384 + tc::sw128_off(t, (cc & 63) >> 3));
          float d0 = fmaf(p[q8 * 8 + 0], inv, -bf16lo_f(raw.x)), d1 = fmaf(p[q8 * 8 + 1], inv, -bf16hi_f(raw.x));
          float d2 = fmaf(p[q8 * 8 + 2], inv, -bf16lo_f(raw.y)), d3 = fmaf(p[q8 * 8 + 3], inv, -bf16hi_f(raw.y));
          float d4 = fmaf(p[q8 * 8 + 4], inv, -bf16lo_f(raw.z)), d5 = fmaf(p[q8 * 8 + 5], inv, -bf16hi_f(raw.z));
          float d6 = fmaf(p[q8 * 8 + 6], inv, -bf16lo_f(raw.w)), d7 = fmaf(p[q8 * 8 + 7], inv, -bf16hi_f(raw.w));
          a0 = fmaf(d0, d0, a0); a1 = fmaf(d1, d1, a1); a2 = fmaf(d2, d2, a2); a3 = fmaf(d3, d3, a3);
          a0 = fmaf(d4, d4, a0); a1 = fmaf(d5, d5, a1); a2 = fmaf(d6, d6, a2); a3 = fmaf(d7, d7, a3);
        }
      }
      const float ss = (a0 + a1) + (a2 + a3);
      if (hf == 1) X.ssp[wg][t] = ss;
      tc::named_bar_sync(1 + wg, 256);
      score = sqrtf(ss + X.ssp[wg][t]);       // hf = 1 threads double their own half; they do not use the score
    }
    // lowest score of the tile (ties: the younger pair), and the two lowest values
    unsigned long long key = ~0ull;
    if (hf == 0) {
      if (scored && ok) scu[is_g ? R : lam] = score;
      if (scored) key = ((unsigned long long)__float_as_uint(score) << 32) | (unsigned)(0x7fffffff - pos);
      // scores are norms (>= 0): their bit patterns order like unsigned integers
      const unsigned sb = scored ? __float_as_uint(score) : 0xffffffffu;
      const unsigned smin = __reduce_min_sync(0xffffffffu, sb);
      const unsigned tb_ = (sb == smin && scored) ? (unsigned)(0x7fffffff - pos) : 0xffffffffu;
      const unsigned tmin = __reduce_min_sync(0xffffffffu, tb_);
      const unsigned long long k = scored || smin != 0xffffffffu ? (((unsigned long long)smin << 32) | tmin) : ~0ull;
      const bool is_min = scored && sb == smin && tb_ == tmin;
      const unsigned s2 = __reduce_min_sync(0xffffffffu, is_min ? 0xffffffffu : sb);
      const float a1 = smin == 0xffffffffu ? CUDART_INF_F : __uint_as_float(smin);
      const float a2 = s2 == 0xffffffffu ? CUDART_INF_F : __uint_as_float(s2);
      if (lane == 0) { X.redkey[wg][wq] = k; X.red12[wg][wq][0] = a1; X.red12[wg][wq][1] = a2; }
    }
    tc::named_bar_sync(1 + wg, 256);
    unsigned long long tkey = X.redkey[wg][0];
#pragma unroll
    for (int w = 1; w < 4; ++w) tkey = X.redkey[wg][w] < tkey ? X.redkey[wg][w] : tkey;
    // the row left out of O^T: both threads of the row know it from the row's position
    const unsigned long long rowkey_lo = (unsigned)(0x7fffffff - pos);
    const bool left_out = scored && (unsigned)tkey == (unsigned)rowkey_lo && tkey != ~0ull;
    if (left_out) {
      if (hf == 0) {
        float a1 = X.red12[wg][0][0], a2 = X.red12[wg][0][1];
#pragma unroll
        for (int w = 1; w < 4; ++w) {
          float b1 = X.red12[wg][w][0], b2 = X.red12[wg][w][1];
          float lo = fminf(a1, b1), hi = fmaxf(a1, b1);
          a2 = fminf(hi, fminf(a2, b2));
          a1 = lo;
        }
        X.cand_key[tile] = key;
        X.cand_score[tile] = score;
        X.cand_min2[tile] = a2;
        X.cand_row[tile] = R;
#pragma unroll
        for (int r = 0; r < QR; ++r) X.cand_z[tile][r] = z[r];
      } else {
#pragma unroll
        for (int ch = 0; ch < d / 8; ++ch)
          X.cand_v[tile][ch] = *reinterpret_cast<const uint4*>(stage_p + S::st_v + (ch >> 3) * 16384 + tc::sw128_off(t, ch & 7));
      }
    }
    if (__any_sync(0xffffffffu, left_out)) {       // its feature row, read back from tensor memory (this thread's half)
      uint32_t pr[32];
      tc::tmem_ld32u(tm_phi + lane_addr + hf * 32, pr);
      if (left_out) {
        uint32_t* dst = reinterpret_cast<uint32_t*>(&X.cand_phi[tile][0]) + hf * 32;
#pragma unroll
        for (int i = 0; i < 32; ++i) dst[i] = pr[i];
      }
    }
    // the row left out of O^T: take its weights back (they were written before the scores were known)
    if (left_out) {
#pragma unroll
      for (int r = 0; r < QR; ++r) {
        if ((r / (QR / 2)) == hf) {
          lpart[r] -= pw[r];
          *reinterpret_cast<unsigned short*>(stage_p + S::st_pt + (t >> 6) * 2048 + tc::sw128_off(r, (t & 63) >> 3) + (t & 7) * 2) = 0;
        }
      }
    }
    tc::fence_async_smem();
    tc::fence_before_sync();
    tc::named_bar_sync(1 + wg, 256);
    tc::fence_after_sync();
    // ---- O^T += V^T Pr^T
    if (lead) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        tc::mma_bf16_ss(tm_o, tc::make_desc_sw128(stage + S::st_v + ks * 2048, 16384, 1024),
                        tc::make_desc_sw128(stage + S::st_pt + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024), idesc3,
                        (have_o || ks > 0) ? 1u : 0u);
      tc::mma_commit(bar_mma3);
    }
    if ((tid & 255) == 32) {
      // a second thread waits for this product (the leader goes on to issue the next tile's first one):
      // the value buffer is free once it is done; everybody else meets this thread again at the next
      // barrier, before anything of this product's operands or O^T is touched
      ok = tc::mbar_wait(bar_mma3, pm3) && ok;
      tc::fence_after_sync();
      if (tile + 2 < NT) decode_issue_tile<DPL>(stage + S::st_v, &tm_gv, &tm_wv, tile + 2, nGB, nRB, unit, bar_v);
    }
    pm3 ^= 1;
    have_o = true;
  }

  // ---- per row group: maximum, sums, partial O^T (kept in the group's own value buffer)
  tc::fence_before_sync();
  tc::named_bar_sync(1 + wg, 256);              // the leader has seen the last O^T product complete
  tc::fence_after_sync();
#pragma unroll
  for (int r = 0; r < QR; ++r) {
    float ls = warp_sum(lpart[r]);
    if (lane == 0) X.wg_l[wg][warp & 7][r] = ls;
    if (t == r && hf == 0) X.wg_m[wg][r] = m_run[r];
  }
  float* opart = reinterpret_cast<float*>(stage_p + S::st_v);   // [128][QR]
  if (hf == 0) {
    float ov[8];
#pragma unroll
    for (int r = 0; r < QR; ++r) ov[r] = 0.f;
    if (have_o) tc::tmem_ld8(tm_o + lane_addr, ov);
#pragma unroll
    for (int r = 0; r < QR; ++r) opart[t * QR + r] = ov[r];
  }
  tc::fence_before_sync();
  __syncthreads();

  // ---- the pair to fold: lowest (score, then youngest) over the tiles' left-out rows
  int lt = 0;
  {
    unsigned long long best = X.cand_key[0];
    for (int i = 1; i < NT; ++i)
      if (X.cand_key[i] < best) { best = X.cand_key[i]; lt = i; }
  }
  if (warp < g) {                                 // phi(q) . phi_fold
    const int r = warp;
    const __nv_bfloat16* pf = reinterpret_cast<const __nv_bfloat16*>(&X.cand_phi[lt][0]);
    float a = 0.f;
    for (int j = lane; j < D; j += 32) a = fmaf(X.phiq_f[r][j], __bfloat162float(pf[j]), a);
    a = warp_sum(a);
    if (lane == 0) X.dotL[r] = a;
  }
  __syncthreads();
  const __nv_bfloat16* phiL = reinterpret_cast<const __nv_bfloat16*>(&X.cand_phi[lt][0]);
  const __nv_bfloat16* vL = reinterpret_cast<const __nv_bfloat16*>(&X.cand_v[lt][0]);

  // ---- Eq. 13: H += phi_fold v_fold^T, s += phi_fold (fp32 additions performed at the L2, no read-back)
  if (ok) {
    float* Hgw = L.H + (size_t)unit * D * d;
    constexpr int per_row = d / 4;
#pragma unroll 4
    for (int i = tid; i < D * per_row; i += kDecThreads) {
      const int j = i / per_row, c4 = (i % per_row) * 4;
      const float pj = __bfloat162float(phiL[j]);
      const uint2 vv = *reinterpret_cast<const uint2*>(vL + c4);
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(Hgw + (size_t)i * 4), "f"(pj * bf16lo_f(vv.x)),
                   "f"(pj * bf16hi_f(vv.x)), "f"(pj * bf16lo_f(vv.y)), "f"(pj * bf16hi_f(vv.y))
                   : "memory");
    }
    if (tid < D) atomicAdd(L.s + (size_t)unit * D + tid, __bfloat162float(phiL[tid]));
  }

  // ---- Eq. 14: thread (query row r, value column cc)
  if (ok) {
    const float* op0 = reinterpret_cast<const float*>(sm + S::stage0 + S::st_v);
    const float* op1 = reinterpret_cast<const float*>(sm + S::stage0 + S::stage_bytes + S::st_v);
    for (int i = tid; i < g * d; i += kDecThreads) {
      const int r = i / d, cc = i % d;
      const float m0 = X.wg_m[0][r], m1 = X.wg_m[1][r];
      const float mf = fmaxf(fmaxf(m0, m1), X.zn[r]);
      const float a0 = tc::fast_exp2(m0 - mf), a1 = tc::fast_exp2(m1 - mf);
      float l0 = 0.f, l1 = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) { l0 += X.wg_l[0][w][r]; l1 += X.wg_l[1][w][r]; }
      float num = a0 * op0[cc * QR + r] + a1 * op1[cc * QR + r];
      float den = a0 * l0 + a1 * l1;
      for (int ti = 0; ti < NT; ++ti) {
        if (ti == lt || X.cand_key[ti] == ~0ull) continue;
        const float p = round_bf16f(tc::fast_exp2(X.cand_z[ti][r] - mf));
        num = fmaf(p, __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(&X.cand_v[ti][0])[cc]), num);
        den += p;
      }
      const float pn = tc::fast_exp2(X.zn[r] - mf);
      num = fmaf(pn, X.vnew[cc], num);
      den += pn;
      const float e = tc::fast_exp2(-mf);
      num = fmaf(e * X.dotL[r], __bfloat162float(vL[cc]), num);
      den = fmaf(e, X.lden[r] + X.dotL[r], den);
      ((T*)c.out)[((size_t)b * L.Hq + h * g + r) * d + cc] = __float2bfloat16_rn(num / den);
    }
  }

  // ---- the evicted pair takes the folded member's slot (nothing moves when it is folded itself)
  const int rowL = X.cand_row[lt];
  const T* ring_k = (const T*)L.wk + ((size_t)unit * eta + s_ev) * d;
  const T* ring_v = (const T*)L.wv + ((size_t)unit * eta + s_ev) * d;
  if (ok && rowL < lam) {
    constexpr int nch = d / 8;
    if (tid < 2 * nch) {
      const T* src = tid < nch ? ring_k : ring_v;
      T* dst = (tid < nch ? (T*)L.gk : (T*)L.gv) + ((size_t)unit * lam + rowL) * d;
      const int ch = tid % nch;
      *reinterpret_cast<uint4*>(dst + ch * 8) = *reinterpret_cast<const uint4*>(src + ch * 8);
    }
    if (tid == 64) {
      L.gpos[(size_t)unit * lam + rowL] = pos_ev;
      scu[rowL] = scu[lam];
    }
  }
  if (tid == 96 && ok) {
    // lowest kept / highest folded score of this update
    float second = X.cand_min2[lt];
    for (int i = 0; i < NT; ++i)
      if (i != lt) second = fminf(second, X.cand_score[i]);
    L.thr[(size_t)unit * 2 + 0] = second;
    L.thr[(size_t)unit * 2 + 1] = X.cand_score[lt];
  }
  __syncthreads();
  // ---- the new pair enters the window ring
  if (ok) {
    constexpr int nch = d / 8;
    if (tid < 2 * nch) {
      const T* src = (tid < nch ? (const T*)c.k : (const T*)c.v) + ((size_t)b * L.Hkv + h) * d;
      T* dst = (tid < nch ? (T*)L.wk : (T*)L.wv) + ((size_t)unit * eta + s_ev) * d;
      const int ch = tid % nch;
      *reinterpret_cast<uint4*>(dst + ch * 8) = *reinterpret_cast<const uint4*>(src + ch * 8);
    }
  }
  if (!ok && (tid & 255) == 0) atomicOr(L.status, 8);
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

// Writes, once per layer, W^T of every KV head as the K-major 128-byte-swizzled operand image the
// decode kernel copies into shared memory: per head [d/64 K blocks][64 rows f][128 bytes = 64 i].
template <int DPL>
__global__ void k_prep_wt_image(const __nv_bfloat16* W, __nv_bfloat16* image, int Hkv) {
  constexpr int d = DPL * 32, F = 64;
  const int h = blockIdx.x;
  for (int i = threadIdx.x; i < d * F; i += blockDim.x) {
    const int j = i / F, f = i % F;
    const size_t off = (size_t)h * (d / 64) * 8192 + (size_t)(j >> 6) * 8192 + tc::sw128_off(f, (j & 63) >> 3) + (j & 7) * 2;
    image[off / 2] = W[(size_t)h * d * F + i];
  }
}

}  // namespace lola
