// Eq. 14 for a prefill chunk (bf16 layer, F = 64, at most 64 tokens per call): softmax attention of
// the chunk's queries over the sparse cache, the resident window and the chunk itself (causal), with
// the linear term phi(q)^T H and its normaliser phi(q)^T s in the same denominator.
//
// One CTA serves up to two query tiles of one unit.  A query tile is 128 rows = two query heads x
// 64 token slots.  Keys and values stream through two shared-memory stages in tiles of 128 rows
// (64-row blocks of sparse-cache slots, ring slots, then the incoming chunk), loaded once for both
// query tiles by TMA.  Warp roles:
//   warps 0-7 / 8-15 softmax of query tile 0 / 1, two threads per row (64 keys each): S from tensor memory, masked
//                    maximum (the stabiliser only moves when it must grow by more than 2^8), weights
//                    exp(z - m) rounded to bf16 and written back over S as the A operand of PV
//   warp 16          issues every tcgen05.mma:  S_w = Q_w K^T,  O_w += P_w V  (P_w in tensor memory)
//   warp 17          TMA producer
// Before the first tile the feature map of the queries is computed (U_w = Q_w W on the tensor cores into the
// score columns, two threads per row) and fed as a tensor-memory A operand into O_w = phi H (H from its bf16
// operand image, made from H at the start): the linear term is the first thing in the accumulator, with the
// weight exp(0 - m) of a key whose score is 0 (m = 0 at that point), and follows the stabiliser like every
// other summand; its normaliser phi . s starts the row's denominator.  This runs while the first tiles load.
// Every wait on an mbarrier is bounded; a wait that runs out sets bit 64 of the status word and makes
// the other waits of the CTA return at once.
#pragma once
#include <cuda.h>

#include "lola_decode_tc.cuh"
#include "lola_generic.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kAt2Threads = 576;

template <int DPL>
struct Attend2Smem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;
  static constexpr uint32_t q = 0;                                   // 2 x [kblk][128][128B]
  static constexpr uint32_t stage0 = 65536;                          // 2 x (K 32 KB + V 32 KB)
  static constexpr uint32_t st_k = 0, st_v = 32768, stage_bytes = 65536;
  static constexpr uint32_t ht = stage0 + 2 * stage_bytes;           // H^T operand image [2 j blocks][d][128B]
  static constexpr uint32_t ht_blk = d * 128;
  static constexpr uint32_t misc = ht + 32768;
  static constexpr uint32_t total = misc + 2816;
  static constexpr uint32_t bytes = 232448;                          // all of an SM's shared memory; the base is aligned at run time
};

struct Attend2Misc {
  uint64_t bars[24];
  float s_vec[128];
  float hx[2][2][128];           // [query tile][half][row]: row maxima of the two halves of a key tile; at the end
                                 // the two halves of the row's denominator
  uint32_t tmem_slot;
  int abort_word;
};
// barrier indices
enum { A2_QFULL = 0, A2_KFULL = 1, A2_VFULL = 3, A2_KEMPTY = 5, A2_VEMPTY = 7, A2_SFULL = 9, A2_PREADY = 11, A2_ODONE = 13, A2_WFULL = 15, A2_HFULL = 16 };

template <int DPL>
__global__ void __launch_bounds__(kAt2Threads, 1)
k_attend2_tc(Layer L, Call c, const __grid_constant__ CUtensorMap tm_gk, const __grid_constant__ CUtensorMap tm_gv,
             const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
             const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_ck,
             const __grid_constant__ CUtensorMap tm_cv, const __grid_constant__ CUtensorMap tm_out, const uint4* wt_image,
             int before_scoring) {
  using S = Attend2Smem<DPL>;
  constexpr int d = DPL * 32;
  constexpr int kblk = d / 64;
  constexpr int D = 128;
  constexpr float kLog2e = 1.4426950408889634f;
  constexpr float kGrow = 8.0f;                       // the stabiliser moves only when it must grow by more than 2^8
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  Attend2Misc& X = *reinterpret_cast<Attend2Misc*>(sm + S::misc);
  const uint32_t bar0 = sbase + S::misc + (uint32_t)offsetof(Attend2Misc, bars);
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  volatile int* abortw = &X.abort_word;
  auto WAIT = [&](int i, uint32_t parity) { return tc::mbar_wait(BAR(i), parity, abortw); };

  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  if ((uint32_t)(sm - smem_raw) + S::total > S::bytes) {            // (cannot happen with a 1024-byte aligned window)
    if (threadIdx.x == 0) atomicOr(L.status, 64);
    return;
  }

  const int unit = blockIdx.y, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = L.g, n = c.nq;
  const int nqt = (g + 1) / 2;                        // query tiles of the unit
  const int qt0 = blockIdx.x * 2;
  const int nw = min(2, nqt - qt0);                   // query tiles of this CTA
  const int att_g = c.att_g, cw = c.att_wn;
  const int nGB = (att_g + 63) / 64, nRB = (cw + 63) / 64, NB = nGB + nRB + 1, NT = (NB + 1) / 2;
  const float sl2 = L.scale * kLog2e;
  bool ok = true;

  if (tid == 0) {
    X.abort_word = 0;
    for (int i = 0; i < 17; ++i) tc::mbar_init(BAR(i), i == A2_HFULL ? 512u : ((i == A2_PREADY || i == A2_PREADY + 1) ? 256u : 1u));
    tc::mbar_init_fence();
  }
  if (warp == 0) tc::tmem_alloc(&X.tmem_slot, 512);
  // the next kernel may set itself up beside this one.  before_scoring: the next kernel is the scoring kernel of
  // the same call, which only reads the memories and starts without waiting: it may only start once this block
  // has seen everything before it complete (below)
  if (tid == 0 && !before_scoring) tc::grid_dep_launch_dependents();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (warp == 17 && lane == 0) {
    // The queries are an input of the call, not something the kernels before this one in the stream produce (those
    // are this library's own, which write the memories and outputs only, or kernels that let nothing start before
    // they are complete): their load starts before the wait, so that U = Q W can begin as soon as W^T arrives.
    // queries: tile w, head slot hs -> rows hs * 64 .. hs * 64 + 63
    tc::mbar_expect_tx(BAR(A2_QFULL), (uint32_t)nw * kblk * 16384u);
    for (int w = 0; w < nw; ++w)
      for (int hs = 0; hs < 2; ++hs) {
        const int hl = (qt0 + w) * 2 + hs;
        const int head = hl < g ? h * g + hl : L.Hq;        // a head index outside the tensor reads as zeros
#pragma unroll
        for (int cb = 0; cb < kblk; ++cb)
          tc::tma_load_4d(sbase + S::q + (uint32_t)w * 32768u + (uint32_t)cb * 16384u + (uint32_t)hs * 8192u, &tm_q, cb * 64, head,
                          0, b, BAR(A2_QFULL));
      }
  }
  tc::grid_dep_wait();                               // everything before this kernel in the stream is complete
  if (tid == 0 && before_scoring) tc::grid_dep_launch_dependents();
  const uint32_t tmem = X.tmem_slot;
  // H (fp32 [D][d]) goes through registers into its bf16 operand image H^T (K-major: row c, 64 j per 128-byte row,
  // two j blocks): thread x of the 16 softmax warps gathers, for DPL items (column c, 8 consecutive j), the eight
  // values H[j][c]; lanes = consecutive columns, so every load of a warp is one 128-byte line
  float pre_h[DPL][8];
  if (tid < 512) {
    const float* Hg = L.H + (size_t)unit * D * d;
#pragma unroll
    for (int n = 0; n < DPL; ++n) {
      const int it = tid + 512 * n, cc = it % d, jc = it / d;
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) pre_h[n][jj] = Hg[(size_t)(jc * 8 + jj) * d + cc];
    }
  }
  if (tid < D) X.s_vec[tid] = L.s[(size_t)unit * D + tid];
  __syncthreads();
  if (tid < 512) {
#pragma unroll
    for (int n = 0; n < DPL; ++n) {
      const int it = tid + 512 * n, cc = it % d, jc = it / d;
      *reinterpret_cast<uint4*>(sm + S::ht + (jc >> 3) * S::ht_blk + tc::sw128_off(cc, jc & 7)) = tc::pack8_bf16(pre_h[n]);
    }
    tc::fence_async_smem();
    tc::mbar_arrive(BAR(A2_HFULL));
  }

  // block `blk` of the key stream -> TMA source
  auto issue_block = [&](uint32_t dst, int blk, bool is_v, uint32_t bar) {
#pragma unroll
    for (int cb = 0; cb < kblk; ++cb) {
      const uint32_t dd = dst + (uint32_t)cb * 16384u;
      if (blk < nGB) tc::tma_load_3d(dd, is_v ? &tm_gv : &tm_gk, cb * 64, blk * 64, unit, bar);
      else if (blk < nGB + nRB) tc::tma_load_3d(dd, is_v ? &tm_wv : &tm_wk, cb * 64, (blk - nGB) * 64, unit, bar);
      else if (blk == nGB + nRB) tc::tma_load_4d(dd, is_v ? &tm_cv : &tm_ck, cb * 64, h, 0, b, bar);
      else tc::tma_load_4d(dd, is_v ? &tm_cv : &tm_ck, cb * 64, h, 64, b, bar);   // beyond the chunk: zeros
    }
  };

  if (warp == 17) {
    // =============================== TMA producer ===============================
    if (lane == 0) {
      // W^T image into the key buffer of stage 1, which the second tile takes over once U = Q W has read it
      tc::mbar_expect_tx(BAR(A2_WFULL), (uint32_t)kblk * 8192u);
      tc::bulk_copy_g2s(sbase + S::stage0 + S::stage_bytes + S::st_k, wt_image + (size_t)h * kblk * 512, kblk * 8192u, BAR(A2_WFULL));
      for (int kt = 0; kt < NT; ++kt) {
        const int st = kt & 1;
        const uint32_t stage = sbase + S::stage0 + (uint32_t)st * S::stage_bytes;
        if (st == 1) ok = WAIT(A2_KEMPTY + 1, (kt >> 1) & 1) && ok;   // (its first completion is the read of W^T)
        else if (kt >= 2) ok = WAIT(A2_KEMPTY + 0, ((kt >> 1) - 1) & 1) && ok;
        tc::mbar_expect_tx(BAR(A2_KFULL + st), (uint32_t)kblk * 16384u);
        issue_block(stage + S::st_k, 2 * kt, false, BAR(A2_KFULL + st));
        issue_block(stage + S::st_k + 8192u, 2 * kt + 1, false, BAR(A2_KFULL + st));
        if (kt >= 2) ok = WAIT(A2_VEMPTY + st, ((kt >> 1) - 1) & 1) && ok;
        tc::mbar_expect_tx(BAR(A2_VFULL + st), (uint32_t)kblk * 16384u);
        issue_block(stage + S::st_v, 2 * kt, true, BAR(A2_VFULL + st));
        issue_block(stage + S::st_v + 8192u, 2 * kt + 1, true, BAR(A2_VFULL + st));
      }
      if (!ok) atomicOr(L.status, 64);
    }
  } else if (warp == 16) {
    // =============================== MMA issuer ===============================
    if (lane == 0) {
      const uint32_t idesc_s = tc::make_idesc_bf16(128, 128, false, false);
      const uint32_t idesc_pv = tc::make_idesc_bf16(128, d, false, true);
      // operand descriptors once; a K step adds its byte offset / 16 to the address field
      const uint64_t dq0 = tc::make_desc_sw128(sbase + S::q, 16, 1024), dq1 = tc::make_desc_sw128(sbase + S::q + 32768u, 16, 1024);
      const uint64_t dk0 = tc::make_desc_sw128(sbase + S::stage0 + S::st_k, 16, 1024);
      const uint64_t dk1 = tc::make_desc_sw128(sbase + S::stage0 + S::stage_bytes + S::st_k, 16, 1024);
      const uint64_t dv0 = tc::make_desc_sw128(sbase + S::stage0 + S::st_v, 16384, 1024);
      const uint64_t dv1 = tc::make_desc_sw128(sbase + S::stage0 + S::stage_bytes + S::st_v, 16384, 1024);
      auto issue_s = [&](int w, int kt) {
        const uint64_t dq = w ? dq1 : dq0, dk = (kt & 1) ? dk1 : dk0;
        const uint32_t ts = tmem + (uint32_t)w * 128u;
#pragma unroll
        for (int ks = 0; ks < d / 16; ++ks) {
          const uint64_t off = (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4);
          tc::mma_bf16_ss(ts, dq + off, dk + off, idesc_s, ks > 0);
        }
        tc::mma_commit(BAR(A2_SFULL + w));
      };
      auto issue_pv = [&](int w, int kt) {
        const uint64_t dv = (kt & 1) ? dv1 : dv0;
        const uint32_t to = tmem + 256u + (uint32_t)w * 128u, tp = tmem + (uint32_t)w * 128u;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)                                   // (the linear term is in O_w already)
          tc::mma_bf16_ts(to, tp + (uint32_t)(ks >> 2) * 64u + (ks & 3) * 8, dv + (uint64_t)((ks * 2048) >> 4), idesc_pv, 1u);
        tc::mma_commit(BAR(A2_ODONE + w));
      };
      // ---- linear term first: U_w = Q_w W into the score columns, then O_w = phi(Q_w) H
      ok = WAIT(A2_QFULL, 0) && ok;
      ok = WAIT(A2_WFULL, 0) && ok;
      tc::fence_after_sync();
      {
        const uint32_t wt = sbase + S::stage0 + S::stage_bytes + S::st_k;
        for (int w = 0; w < nw; ++w) {
#pragma unroll
          for (int ks = 0; ks < d / 16; ++ks)
            tc::mma_bf16_ss(tmem + (uint32_t)w * 128u,
                            tc::make_desc_sw128(sbase + S::q + (uint32_t)w * 32768u + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                            tc::make_desc_sw128(wt + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024),
                            tc::make_idesc_bf16(128, 64, false, false), ks > 0);
          tc::mma_commit(BAR(A2_SFULL + w));                              // completion 0 of S_w: U_w
        }
        tc::mma_commit(BAR(A2_KEMPTY + 1));                               // W^T is read: the second tile may load
      }
      ok = WAIT(A2_HFULL, 0) && ok;
      ok = WAIT(A2_KFULL + 0, 0) && ok;
      for (int w = 0; w < nw; ++w) {
        ok = WAIT(A2_PREADY + w, 0) && ok;                                // phi(Q_w) in tensor memory
        tc::fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ts(tmem + 256u + (uint32_t)w * 128u, tmem + (uint32_t)w * 128u + 64u + ks * 8,
                          tc::make_desc_sw128(sbase + S::ht + (ks >> 2) * S::ht_blk + (ks & 3) * 32, 16, 1024),
                          tc::make_idesc_bf16(128, d, false, false), ks > 0);
        tc::mma_commit(BAR(A2_ODONE + w));                                // completion 0 of O_w: the linear term
        issue_s(w, 0);                                                    // (the tensor pipe runs in order: phi is consumed first)
      }
      tc::mma_commit(BAR(A2_KEMPTY + 0));
      for (int kt = 0; kt < NT; ++kt) {
        const int st = kt & 1;
        ok = WAIT(A2_VFULL + st, (kt >> 1) & 1) && ok;
        if (kt + 1 < NT) ok = WAIT(A2_KFULL + (st ^ 1), ((kt + 1) >> 1) & 1) && ok;
        for (int w = 0; w < nw; ++w) {
          ok = WAIT(A2_PREADY + w, (kt + 1) & 1) && ok;
          tc::fence_after_sync();
          issue_pv(w, kt);
          if (kt + 1 < NT) issue_s(w, kt + 1);
        }
        tc::mma_commit(BAR(A2_VEMPTY + st));
        if (kt + 1 < NT) tc::mma_commit(BAR(A2_KEMPTY + (st ^ 1)));
      }
      if (!ok) atomicOr(L.status, 64);
    }
  } else if (warp < 8 * nw) {
    // =============================== softmax, two threads per query row ===============================
    // thread (query tile w, row t, half hf) owns the 64 keys [64 hf, 64 hf + 64) of every key tile, half of
    // the feature map in the linear term and half of the output columns
    const int w = warp >> 3, hf = (warp >> 2) & 1, wq = warp & 3;
    const int t = wq * 32 + lane;                      // row of the query tile = tensor-memory lane
    const int hl = (qt0 + w) * 2 + (t >> 6), tok = t & 63;
    const bool row_ok = hl < g && tok < n;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t tm_s = tmem + (uint32_t)w * 128u + lane_addr;
    const uint32_t tm_sb = tm_s + (uint32_t)hf * 64u;  // this thread's 64 score columns; its weights go to the first 32
    const uint32_t tm_o = tmem + 256u + (uint32_t)w * 128u + lane_addr;
    constexpr int HC = d / 2;
    const int pair_bar = 1 + w * 4 + wq;               // the two warps that share this row quadrant (64 threads)
    // ---- linear term first
    ok = WAIT(A2_SFULL + w, 0) && ok;                  // U = Q W is in the first 64 score columns
    tc::fence_after_sync();
    float m_used = 0.f, l;                             // log2 units; m >= 0 is the stabiliser max(0, max z)
    {
      // this thread's half of phi(q) (hf = 0: softmax(u), 1: softmax(-u)), with weight exp(0 - m), m = 0: bf16 pairs
      // into columns 64 + 32 hf .. of S_w (A operand of the linear product)
      float e[64];
      tc::tmem_ld64(tm_s, e);
      const float em = (c.att_flags & 1) ? 0.f : 1.0f;   // (0: the queries do not see H, s)
      const float sgn = hf ? -kLog2e : kLog2e;
      float scale;
      if (L.phi_kind == 1) {
#pragma unroll
        for (int i = 0; i < 64; ++i) e[i] = tc::fast_exp2(e[i] * sgn);
        scale = em;
      } else {
        float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < 64; i += 2) { m0 = fmaxf(m0, e[i] * sgn); m1 = fmaxf(m1, e[i + 1] * sgn); }
        const float mm = fmaxf(m0, m1);
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int i = 0; i < 64; i += 2) {
          e[i] = tc::fast_exp2(fmaf(e[i], sgn, -mm)); s0 += e[i];
          e[i + 1] = tc::fast_exp2(fmaf(e[i + 1], sgn, -mm)); s1 += e[i + 1];
        }
        scale = em / (s0 + s1);
      }
      float ld0 = 0.f, ld1 = 0.f;
#pragma unroll
      for (int i = 0; i < 64; i += 2) {
        e[i] *= scale;
        e[i + 1] *= scale;
        ld0 = fmaf(e[i], X.s_vec[hf * 64 + i], ld0);
        ld1 = fmaf(e[i + 1], X.s_vec[hf * 64 + i + 1], ld1);
      }
      l = ld0 + ld1;                                   // this half of the normaliser phi . s starts the sum of the weights
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) pk[j >> 1] = pack_bf16x2(e[c0 + j], e[c0 + j + 1]);
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n" ::"r"(
                tm_s + 64 + hf * 32 + (c0 >> 1)),
            "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]), "r"(pk[8]), "r"(pk[9]),
            "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15])
            : "memory");
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    tc::fence_before_sync();
    tc::mbar_arrive(BAR(A2_PREADY + w));               // completion 0: phi(Q_w) is in columns 64.. of S_w
    for (int kt = 0; kt < NT; ++kt) {
      // valid leading columns of this thread's 64-key block of the tile, for this row
      const int blk = 2 * kt + hf;
      int lim;
      if (blk < nGB) lim = att_g - blk * 64;
      else if (blk < nGB + nRB) lim = cw - (blk - nGB) * 64;
      else if (blk == nGB + nRB) lim = min(n, tok + 1);
      else lim = 0;
      lim = max(0, min(64, lim));
      ok = WAIT(A2_SFULL + w, (kt + 1) & 1) && ok;
      tc::fence_after_sync();
      float sv[64];
      tc::tmem_ld64(tm_sb, sv);
      float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
      if (lim == 64) {
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
          mx0 = fmaxf(mx0, fmaxf(sv[j], sv[j + 1]));
          mx1 = fmaxf(mx1, fmaxf(sv[j + 2], sv[j + 3]));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          sv[j] = j < lim ? sv[j] : -CUDART_INF_F;     // masked keys get weight 2^(-inf) = 0 below
          mx0 = fmaxf(mx0, sv[j]);
        }
      }
      X.hx[w][hf][t] = fmaxf(mx0, mx1);
      tc::named_bar_sync(pair_bar, 64);                    // (also: both halves hold their scores in registers now)
      const float m_tile = fmaxf(X.hx[w][0][t], X.hx[w][1][t]) * sl2;
      const bool grow = m_tile > m_used + kGrow;
      if (__any_sync(0xffffffffu, grow)) {             // rare; tensor-memory accesses are warp-wide: every lane takes part
        const float m_new = grow ? m_tile : m_used;
        const float alpha = tc::fast_exp2(m_used - m_new);
        l *= alpha;
        m_used = m_new;
        {
          ok = WAIT(A2_ODONE + w, kt & 1) && ok;         // the product of the tile before (or the linear term) is complete
          tc::fence_after_sync();
#pragma unroll
          for (int c0 = 0; c0 < HC; c0 += 8) {         // this thread's half of the row's output columns
            float ov[8];
            tc::tmem_ld8(tm_o + hf * HC + c0, ov);
#pragma unroll
            for (int j = 0; j < 8; ++j) ov[j] *= alpha;
            tc::tmem_st8(tm_o + hf * HC + c0, ov);
          }
        }
      }
      // weights 2^(z - m) <= 2^8 as bf16 pairs over the first half of this thread's S columns
      // (packed f32x2 arithmetic: the sums of the even and of the odd columns are the two lanes)
      const uint64_t sl22 = tc::pack_f2(sl2, sl2), nm2 = tc::pack_f2(-m_used, -m_used);
      uint64_t lacc = tc::pack_f2(0.f, 0.f);
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          float x0, x1;
          tc::unpack_f2(tc::fma2(tc::pack_f2(sv[c0 + j], sv[c0 + j + 1]), sl22, nm2), x0, x1);
          const float p0 = tc::fast_exp2(x0), p1 = tc::fast_exp2(x1);
          lacc = tc::add2(lacc, tc::pack_f2(p0, p1));
          pk[j >> 1] = pack_bf16x2(p0, p1);
        }
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};\n" ::"r"(
                tm_sb + (c0 >> 1)),
            "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7]), "r"(pk[8]), "r"(pk[9]),
            "r"(pk[10]), "r"(pk[11]), "r"(pk[12]), "r"(pk[13]), "r"(pk[14]), "r"(pk[15])
            : "memory");
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      float l0, l1;
      tc::unpack_f2(lacc, l0, l1);
      l += l0 + l1;
      tc::fence_before_sync();
      tc::mbar_arrive(BAR(A2_PREADY + w));
    }
    // ---- the two halves of the row's denominator meet (the extra barrier: the partner has read this row's last
    // maxima before the slot is reused)
    tc::named_bar_sync(pair_bar, 64);  
    X.hx[w][hf][t] = l;
    tc::named_bar_sync(pair_bar, 64);  
    const float lden = X.hx[w][hf ^ 1][t];
    ok = WAIT(A2_ODONE + w, NT & 1) && ok;
    tc::fence_after_sync();
    {
      // the tile's outputs are staged in the layout of a TMA box ([head slot][64-column block][64 tokens]
      // [128 bytes], 128-byte swizzle) and stored by one thread: 576 threads storing 16 bytes at a time would take
      // the load/store unit 2 us.  The staging buffers are the key (w = 0) and value (w = 1) buffers of the stage
      // the last tile did not use: the other query tile's last product may still be reading the last tile
      const float inv = 1.0f / (X.hx[w][hf][t] + lden);
      const uint32_t stg_off = S::stage0 + (uint32_t)(NT & 1) * S::stage_bytes + (w ? S::st_v : S::st_k);
      uint8_t* stg = sm + stg_off;
      const int hs = t >> 6;
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        float ov[32];
        tc::tmem_ld32(tm_o + hf * HC + c0, ov);
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8) {
          const int cc = hf * HC + c0 + q8 * 8;
          uint4 o;
          o.x = pack_bf16x2(ov[q8 * 8 + 0] * inv, ov[q8 * 8 + 1] * inv);
          o.y = pack_bf16x2(ov[q8 * 8 + 2] * inv, ov[q8 * 8 + 3] * inv);
          o.z = pack_bf16x2(ov[q8 * 8 + 4] * inv, ov[q8 * 8 + 5] * inv);
          o.w = pack_bf16x2(ov[q8 * 8 + 6] * inv, ov[q8 * 8 + 7] * inv);
          *reinterpret_cast<uint4*>(stg + (hs * kblk + (cc >> 6)) * 8192 + tc::sw128_off(tok, (cc & 63) >> 3)) = o;
        }
      }
      tc::fence_async_smem();
      tc::named_bar_sync(9 + w, 256);
      if (t == 0 && hf == 0 && ok) {
        const uint32_t sstg = sbase + stg_off;
        for (int s2 = 0; s2 < 2; ++s2) {
          const int hl2 = (qt0 + w) * 2 + s2;
          if (hl2 >= g) continue;                      // (rows of tokens >= n lie outside the tensor: not written)
#pragma unroll
          for (int cb = 0; cb < kblk; ++cb)
            tc::tma_store_4d(&tm_out, sstg + (uint32_t)(s2 * kblk + cb) * 8192u, cb * 64, h * g + hl2, 0, b);
        }
        tc::bulk_commit_group();
        tc::bulk_wait_group_read();                    // the staging buffer stays valid until it is read
      }
    }
    if (!ok && t == 0 && hf == 0) atomicOr(L.status, 64);
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

}  // namespace lola
