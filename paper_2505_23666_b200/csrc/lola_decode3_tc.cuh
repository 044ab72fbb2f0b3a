// The generation step (Eq. 11-14) as ONE PERSISTENT kernel: a thread block stays on its SM and works through
// several units, and the set-up of the next unit runs while the current one is still being scored, so that
// the memories stream from HBM without the gaps a block per unit leaves between its prologue, its tiles and
// its epilogue.  Same arithmetic and the same per-tile products as k_decode2_tc (steady state of a bf16 layer
// with F = 64, caches full, one pair leaving the window; at most 8 row tiles per unit, g <= 4).
//
//   feature group (warps 0-7)   per unit: fetches q, the new pair, the leaving pair, s and H (H straight into
//                               registers, 64 values per thread), computes phi(q) and its normaliser, writes the
//                               bf16 operand image of H^T; per tile: q.k columns and their warp maxima into shared
//                               memory, the feature map of U into tensor memory
//   score group   (warps 8-15)  per tile: running maxima and softmax weights (bf16) into the Pr^T operand,
//                               Eq. 10 from [P | den] and the value tile, the tile's lowest score, the row left
//                               out of O^T; per unit: the fold (Eq. 13) as vector reductions at the L2, the
//                               outputs (Eq. 14), the slot replacement
//   warp 16, one thread         issues [U | Z] = K [W | Q^T] (up to two tiles ahead, across unit boundaries),
//                               the linear term H^T phi(Q)^T and [P | den] = phi [H | s]; key-tile and W^T loads
//   warp 17, one thread         issues O^T += V^T Pr^T; value-tile loads
//
// All tile-level hand-overs are mbarriers whose phases run on over the units of a block (a tile's buffers and
// barrier parities follow its running index in the block), unit-level hand-overs have one barrier each.
// Every wait is bounded; a wait that runs out raises the block's abort word (bit 8 of the status word).
#pragma once
#include "lola_decode2_tc.cuh"

namespace lola {

constexpr int kDec3Q = 4;              // query rows per unit (g <= 4)

struct Decode3Misc {
  // written by the feature group in a unit's set-up and read only there
  float qf[kDec3Q][128];
  float u_s[kDec3Q][64];
  float knew[128], s_f[128];
  // written in a unit's set-up, read by the score group at the end of that unit: one copy per unit parity
  float phiq_f[2][kDec3Q][128];          // phi(q) rounded to bf16, as fp32
  float vnew[2][128];
  uint4 ring_kv[2][2 * 16];              // the pair that leaves the window (key chunks, then value chunks), bf16
  uint4 new_kv[2][2 * 16];               // the new pair, bf16
  float zn[2][kDec3Q], lden[2][kDec3Q];
  // per tile, feature group -> score group (tile parity)
  float redmax[2][4][kDec3Q];
  float z_s[2][kDec3Q][128];             // q.k of the tile's rows (log2 units)
  // score group
  float dotL[kDec3Q], m_s[kDec3Q], l_s[4][kDec3Q];
  unsigned long long redkey[4];
  float red12[4][2];
  float ssp[128];
  float opart[128][kDec3Q];              // O^T after the last tile: [value column][query row]
  unsigned long long cand_key[kDec2MaxTiles];
  float cand_score[kDec2MaxTiles], cand_min2[kDec2MaxTiles];
  int cand_row[kDec2MaxTiles];
  float cand_z[kDec2MaxTiles][kDec3Q];
  uint4 cand_v[kDec2MaxTiles][16];       // value row, bf16
  uint4 cand_phi[kDec2MaxTiles][16];     // feature row, bf16
  uint64_t bars[24];
  uint32_t tmem_slot;
  int abort_word;
};
static_assert(sizeof(Decode3Misc) <= 28672, "misc region too small");

// barrier indices
enum {
  D3_KFULL = 0, D3_VFULL = 2, D3_UFULL = 4, D3_PHIDONE = 6, D3_PTREADY = 8, D3_ODONE = 10,   // two each (tile parity)
  D3_PDONE = 12, D3_PFREE = 13,                                                               // one per tile
  D3_WFULL = 14, D3_QREADY = 15, D3_HTREADY = 16, D3_HTFREE = 17, D3_LINDONE = 18, D3_OREAD = 19, D3_EPIDONE = 20,   // one per unit
  D3_NBARS = 21
};

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int DPL>
__global__ void __launch_bounds__(kDec2Threads, 1)
k_decode3_tc(Layer L, Call c, const __grid_constant__ CUtensorMap tm_gk, const __grid_constant__ CUtensorMap tm_gv,
             const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv, const uint4* wt_image) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  using S = DecodeSmem<DPL>;
  constexpr int QR = kDec3Q;
  constexpr int d = DPL * 32;
  constexpr int kblk = d / 64;
  constexpr int F = 64, D = 128;
  constexpr int HC = d / 2;                  // value columns per thread of a row pair
  constexpr int QH = QR / 2;                 // query rows per thread of a row pair
  constexpr float kLog2e = 1.4426950408889634f;
  typedef __nv_bfloat16 T;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = tc::smem_u32(sm);
  Decode3Misc& X = *reinterpret_cast<Decode3Misc*>(sm + S::misc);

  const int U = L.B * L.Hkv;
  const int nU = (U - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // units of this block
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int role = warp < 8 ? 0 : (warp < 16 ? 1 : warp - 14);   // 0 feature, 1 score, 2 / 3 issuing threads
  const int gtid = tid & 255;                // index inside a compute group
  const int gw = warp & 7;
  const int wq = gw & 3;                     // tensor-memory lane quadrant of this warp (= warp % 4)
  const int hf = gw >> 2;                    // which half of the row's work this thread does
  const int t = wq * 32 + lane;              // row of the tile = tensor-memory lane
  const int lam = L.lam, eta = L.eta, g = L.g;
  const int nGB = lam / 64, nRB = (eta + 63) / 64, NT = (nGB + nRB + 1) / 2;
  const int TT = nU * NT;                    // tiles of this block, all units
  const int s_ev = c.n_seen % eta;           // ring slot of the pair that leaves = slot the new pair takes
  const int pos_ev = c.n_seen - eta;
  const float sl2 = L.scale * kLog2e;        // q.k in log2 units
  volatile int* abw = &X.abort_word;
  auto unit_of = [&](int n) { return (int)blockIdx.x + n * (int)gridDim.x; };

  const uint32_t bars = sbase + S::misc + (uint32_t)offsetof(Decode3Misc, bars);
  auto BAR = [&](int i) { return bars + 8u * (uint32_t)i; };
  auto WAIT = [&](int i, uint32_t parity) { return tc::mbar_wait(BAR(i), parity & 1u, abw); };
  auto stage_k = [&](int i) { return sbase + S::stage0 + (uint32_t)i * S::stage_bytes + S::st_k; };
  auto stage_v = [&](int i) { return sbase + S::stage0 + (uint32_t)i * S::stage_bytes + S::st_v; };
  auto stage_pt = [&](int i) { return S::stage0 + (uint32_t)i * S::stage_bytes + S::st_pt; };   // offset from sm

  if (tid == 0) {
    X.abort_word = 0;
    for (int i = 0; i < D3_NBARS; ++i) {
      const bool group = (i == D3_PHIDONE || i == D3_PHIDONE + 1 || i == D3_PTREADY || i == D3_PTREADY + 1 || i == D3_PFREE ||
                          i == D3_QREADY || i == D3_HTREADY || i == D3_OREAD || i == D3_EPIDONE);
      tc::mbar_init(BAR(i), group ? 256u : 1u);
    }
    tc::mbar_init_fence();
  }
  if (warp == 0) tc::tmem_alloc(&X.tmem_slot, 512);
  // operand rows that stay zero for the whole launch: rows d+2 .. d+15 of both j blocks of [H^T ; s], phi(Q),
  // both Pr^T tiles (rows of no query head)
  for (int i = tid; i < 2 * 14 * 8; i += kDec2Threads) {
    const int jb = i / (14 * 8), r = (i / 8) % 14, ch = i % 8;
    *reinterpret_cast<uint4*>(sm + S::ht + jb * S::ht_blk + tc::sw128_off(d + 2 + r, ch)) = make_uint4(0, 0, 0, 0);
  }
  for (int i = tid; i < 256; i += kDec2Threads) {
    *reinterpret_cast<uint4*>(sm + S::phiq + i * 16) = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(sm + stage_pt(0) + i * 16) = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(sm + stage_pt(1) + i * 16) = make_uint4(0, 0, 0, 0);
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();

  const uint32_t tmem = X.tmem_slot;
  const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
  auto tm_uz = [&](int i) { return tmem + (uint32_t)i * 96u; };          // [U | Z]: 80 columns, two buffers
  const uint32_t tm_o = tmem + 176u;                                       // O^T: lanes = value column, 16 columns = query rows
  auto tm_phi = [&](int i) { return tmem + 192u + (uint32_t)i * 64u; };   // phi tile, bf16 pairs: 64 columns, two buffers
  const uint32_t tm_p = tmem + 320u;                                       // [P | den]: d + 16 columns
  const uint32_t idesc1 = tc::make_idesc_bf16(128, 80, false, false);
  const uint32_t idesc2 = tc::make_idesc_bf16(128, d + 16, false, false);
  const uint32_t idesc0 = tc::make_idesc_bf16(128, 16, false, false);
  const uint32_t idesc3 = tc::make_idesc_bf16(128, 16, true, false);
  bool ok = true;

  if (role == 2) {
    // =================== products of the feature side, key tiles, W^T ===================
    if (lane == 0) {
      // operand descriptors: the address field (units of 16 bytes) takes the offset of a K step
      const uint64_t dk0 = tc::make_desc_sw128(stage_k(0), 16, 1024), dk1 = tc::make_desc_sw128(stage_k(1), 16, 1024);
      const uint64_t db1 = tc::make_desc_sw128(sbase + S::b1, 16, 1024), dht = tc::make_desc_sw128(sbase + S::ht, 16, 1024);
      auto issue_w = [&](int n) {                      // W^T of unit n's KV head into rows 0..63 of the operand
        const int h = unit_of(n) % L.Hkv;
        tc::mbar_expect_tx(BAR(D3_WFULL), (uint32_t)kblk * 8192u);
        for (int kb = 0; kb < kblk; ++kb)
          tc::bulk_copy_g2s(sbase + S::b1 + (uint32_t)kb * S::b1_blk, wt_image + ((size_t)h * kblk + kb) * 512, 8192u, BAR(D3_WFULL));
      };
      auto issue_k = [&](int G) {
        decode2_issue_tile<DPL>(stage_k(G & 1), &tm_gk, &tm_wk, G % NT, nGB, nRB, unit_of(G / NT), BAR(D3_KFULL + (G & 1)));
      };
      auto issue_mma1 = [&](int G) {
        const uint64_t dk = (G & 1) ? dk1 : dk0;
        const uint32_t tmu = tm_uz(G & 1);
#pragma unroll
        for (int ks = 0; ks < d / 16; ++ks)
          tc::mma_bf16_ss(tmu, dk + (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                          db1 + (uint64_t)(((ks >> 2) * S::b1_blk + (ks & 3) * 32) >> 4), idesc1, ks > 0);
        tc::mma_commit(BAR(D3_UFULL + (G & 1)));
      };
      int next_k = 0;                                  // next key tile to load (running index over the block's units)
      int next1 = 0;                                   // next first product to issue
      int w_issued = 1;                                // units whose W^T copy has been issued
      issue_w(0);
      for (; next_k < min(2, TT); ++next_k) issue_k(next_k);
      // Tries to issue the first product of tile `next1`.  Inside a unit every wait is short.  At the first tile
      // of a unit the operand [W | Q^T] changes: with `blocking` false the attempt is given up while the feature
      // group has not yet written the new unit's query rows (the products this thread owes the unit in progress
      // come first).
      auto advance_mma1 = [&](bool blocking) -> bool {
        const int G1 = next1, n1 = G1 / NT, t1 = G1 % NT;
        while (next_k <= G1) {                         // (its key tile must have been requested: the stage is free
          if (next_k >= 2) ok = WAIT(D3_UFULL + (next_k & 1), (uint32_t)((next_k - 2) >> 1)) && ok;   // once the product two tiles before is complete)
          issue_k(next_k);
          ++next_k;
        }
        if (t1 == 0) {
          if (n1 >= w_issued) {
            // every first product of the unit before is complete, and its set-up has read W^T
            ok = WAIT(D3_UFULL + ((G1 - 1) & 1), (uint32_t)((G1 - 1) >> 1)) && ok;
            ok = WAIT(D3_HTREADY, (uint32_t)(n1 - 1)) && ok;
            issue_w(n1);
            w_issued = n1 + 1;
          }
          if (blocking) {
            ok = WAIT(D3_WFULL, (uint32_t)n1) && ok;
            ok = WAIT(D3_QREADY, (uint32_t)n1) && ok;
          } else if (!mbar_test(BAR(D3_WFULL), (uint32_t)n1 & 1u) || !mbar_test(BAR(D3_QREADY), (uint32_t)n1 & 1u)) {
            return false;
          }
        }
        ok = WAIT(D3_KFULL + (G1 & 1), (uint32_t)(G1 >> 1)) && ok;
        tc::fence_after_sync();
        issue_mma1(G1);
        ++next1;
        return true;
      };
      for (int G = 0; G < TT; ++G) {
        while (next1 <= min(G + (G == 0 ? 1 : 0), TT - 1)) {   // (normally issued two tiles earlier; both [U | Z] buffers are free at the start)
          if (next1 <= G) advance_mma1(true);
          else if (!advance_mma1(false)) break;
        }
        const int i = G & 1, n = G / NT, tt = G % NT;
        ok = WAIT(D3_PHIDONE + i, (uint32_t)(G >> 1)) && ok;    // phi(G) written, [U | Z] of this tile read
        if (G > 0) ok = WAIT(D3_PFREE, (uint32_t)(G - 1)) && ok; // [P | den] of the tile before is read
        tc::fence_after_sync();
        if (tt == 0) {
          // H^T, s and phi(Q) of this unit are in place; O^T of the unit before has been read.  O^T starts as the
          // linear term H^T phi(Q)^T, with weight exp(0 - m), m = 0 so far
          ok = WAIT(D3_HTREADY, (uint32_t)n) && ok;
          if (n > 0) ok = WAIT(D3_OREAD, (uint32_t)(n - 1)) && ok;
          tc::fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tm_o, tc::make_desc_sw128(sbase + S::ht + (ks >> 2) * S::ht_blk + (ks & 3) * 32, 16, 1024),
                            tc::make_desc_sw128(sbase + S::phiq + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024), idesc0, ks > 0);
          tc::mma_commit(BAR(D3_LINDONE));
        }
        const uint32_t tph = tm_phi(i);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ts(tm_p, tph + ks * 8, dht + (uint64_t)(((ks >> 2) * S::ht_blk + (ks & 3) * 32) >> 4), idesc2, ks > 0);
        tc::mma_commit(BAR(D3_PDONE));
        if (tt == NT - 1) tc::mma_commit(BAR(D3_HTFREE));        // the unit's last reader of [H^T ; s]
        // first products run two tiles ahead of the feature group: the buffer a tile used is free once its
        // feature rows are written (seen above)
        const int upto = min(G + 2, TT - 1);
        while (next1 <= upto)
          if (!advance_mma1(false)) break;
        // key tiles whose buffer is free already (the product that read it is complete) start to stream now
        while (next_k < TT && next_k - 2 < next1 && mbar_test(BAR(D3_UFULL + (next_k & 1)), (uint32_t)((next_k - 2) >> 1) & 1u)) {
          issue_k(next_k);
          ++next_k;
        }
      }
    }
    __syncwarp();
  } else if (role == 3) {
    // =================== O^T products, value tiles ===================
    if (lane == 0) {
      const uint64_t dv0 = tc::make_desc_sw128(stage_v(0), 16384, 1024), dv1 = tc::make_desc_sw128(stage_v(1), 16384, 1024);
      const uint64_t dp0 = tc::make_desc_sw128(sbase + stage_pt(0), 16, 1024), dp1 = tc::make_desc_sw128(sbase + stage_pt(1), 16, 1024);
      auto issue_v = [&](int G) {
        decode2_issue_tile<DPL>(stage_v(G & 1), &tm_gv, &tm_wv, G % NT, nGB, nRB, unit_of(G / NT), BAR(D3_VFULL + (G & 1)));
      };
      for (int G = 0; G < min(2, TT); ++G) issue_v(G);
      for (int G = 0; G < TT; ++G) {
        const int i = G & 1;
        ok = WAIT(D3_PTREADY + i, (uint32_t)(G >> 1)) && ok;    // Pr^T of the tile written, its value tile read by the score group
        tc::fence_after_sync();
        const uint64_t dv = i ? dv1 : dv0, dp = i ? dp1 : dp0;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          tc::mma_bf16_ss(tm_o, dv + (uint64_t)((ks * 2048) >> 4), dp + (uint64_t)(((ks >> 2) * 2048 + (ks & 3) * 32) >> 4), idesc3, 1u);
        tc::mma_commit(BAR(D3_ODONE + i));
        ok = WAIT(D3_ODONE + i, (uint32_t)(G >> 1)) && ok;
        if (G + 2 < TT) issue_v(G + 2);
      }
    }
    __syncwarp();
  }
  else if (role == 0) {
    // =================== feature group ===================
    const bool exp_kind = L.phi_kind == 1;
    constexpr int NI = d / 16;                       // (column, block of 8 features) items of H per thread
    constexpr int per_row = d / 8;
    int G = 0;
    for (int n = 0; n < nU; ++n) {
      const int unit = unit_of(n), b = unit / L.Hkv, h = unit % L.Hkv, par = n & 1;
      // ---- set-up of unit n.  Everything it needs from global memory is requested first: H (this thread's
      // 8 NI values: column cc, features 8 jc .. 8 jc + 7), s, the query rows, the new pair, the leaving pair
      float hreg[NI * 8];
      {
        const float* Hg = L.H + (size_t)unit * D * d;
#pragma unroll
        for (int k = 0; k < NI; ++k) {
          const int i = gtid + k * 256, cc = i % d, jc = i / d;
#pragma unroll
          for (int jj = 0; jj < 8; ++jj) hreg[k * 8 + jj] = Hg[(size_t)(jc * 8 + jj) * d + cc];
        }
      }
      float pre_s = 0.f, pre_k = 0.f, pre_v = 0.f;
      uint4 pre_q = make_uint4(0, 0, 0, 0), pre_ring = pre_q, pre_new = pre_q;
      if (gtid < D) pre_s = L.s[(size_t)unit * D + gtid];
      if (gtid < 16 * per_row && gtid / per_row < g)
        pre_q = *reinterpret_cast<const uint4*>((const T*)c.q + ((size_t)b * L.Hq + h * g + gtid / per_row) * d + (gtid % per_row) * 8);
      if (gtid < 2 * per_row) {
        const int ch = gtid % per_row;
        const bool is_k = gtid < per_row;
        pre_ring = *reinterpret_cast<const uint4*>((is_k ? (const T*)L.wk : (const T*)L.wv) + ((size_t)unit * eta + s_ev) * d + ch * 8);
        pre_new = *reinterpret_cast<const uint4*>((is_k ? (const T*)c.k : (const T*)c.v) + ((size_t)b * L.Hkv + h) * d + ch * 8);
      }
      if (gtid < d) {
        pre_k = ldf<T>((const T*)c.k + ((size_t)b * L.Hkv + h) * d + gtid);
        pre_v = ldf<T>((const T*)c.v + ((size_t)b * L.Hkv + h) * d + gtid);
      }
      // the copies of the unit two before (same parity) are free once its end-of-unit work is complete
      if (n >= 2) ok = WAIT(D3_EPIDONE, (uint32_t)(n - 2)) && ok;
      // query rows: operand rows 64..79 (rows >= g are zero) and an fp32 copy.  Every first product of the unit
      // before is complete: this group has waited for each of them.
      if (gtid < 16 * per_row) {
        const int r = gtid / per_row, ch = gtid % per_row;
        *reinterpret_cast<uint4*>(sm + S::b1 + (ch >> 3) * S::b1_blk + tc::sw128_off(64 + r, ch & 7)) = pre_q;
        if (r < QR) {
          const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&pre_q);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float2 ff = __bfloat1622float2(v2[q]);
            X.qf[r][ch * 8 + 2 * q] = ff.x;
            X.qf[r][ch * 8 + 2 * q + 1] = ff.y;
          }
        }
      }
      if (gtid < 2 * per_row) { X.ring_kv[par][gtid] = pre_ring; X.new_kv[par][gtid] = pre_new; }
      if (gtid < d) { X.knew[gtid] = pre_k; X.vnew[par][gtid] = pre_v; }
      if (gtid < D) X.s_f[gtid] = pre_s;
      tc::fence_async_smem();
      tc::mbar_arrive(BAR(D3_QREADY));
      ok = WAIT(D3_WFULL, (uint32_t)n) && ok;          // W^T of this unit's KV head is in the operand rows
      tc::named_bar_sync(1, 256);
      // u = q W on the CUDA cores (g rows only) from the W^T operand rows
      for (int i = gtid; i < g * F; i += 256) {
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
      tc::named_bar_sync(1, 256);
      // phi(q), its normaliser phi(q) . s and q . k_new.  The linear product of the unit before has read phi(Q).
      if (n > 0) ok = WAIT(D3_LINDONE, (uint32_t)(n - 1)) && ok;
      if (gw < g) {
        const int r = gw;
        float u0 = X.u_s[r][lane], u1 = X.u_s[r][lane + 32];
        float p0, p1, n0, n1;
        if (exp_kind) {
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
          X.phiq_f[par][r][j] = vals[q];
          *reinterpret_cast<T*>(sm + S::phiq + (j >> 6) * 2048 + tc::sw128_off(r, (j & 63) >> 3) + (j & 7) * 2) = __float2bfloat16_rn(vals[q]);
          ld = fmaf(vals[q], X.s_f[j], ld);
        }
        ld = warp_sum(ld);
        float zz = 0.f;
        for (int j = lane; j < d; j += 32) zz = fmaf(X.qf[r][j], X.knew[j], zz);
        zz = warp_sum(zz);
        if (lane == 0) { X.lden[par][r] = ld; X.zn[par][r] = zz * sl2; }
      }
      // [H^T ; s_hi ; s_lo]: the unit before has issued its last product that reads it
      if (n > 0) ok = WAIT(D3_HTFREE, (uint32_t)(n - 1)) && ok;
      if (gtid < D) {
        // rows d, d+1: s as the sum of two bf16 parts (phi . s_hi + phi . s_lo keeps the fp32 normaliser)
        const __nv_bfloat16 hi = __float2bfloat16_rn(pre_s);
        const __nv_bfloat16 lo = __float2bfloat16_rn(pre_s - __bfloat162float(hi));
        const int ch = (gtid & 63) >> 3;
        *reinterpret_cast<T*>(sm + S::ht + (gtid >> 6) * S::ht_blk + tc::sw128_off(d, ch) + (gtid & 7) * 2) = hi;
        *reinterpret_cast<T*>(sm + S::ht + (gtid >> 6) * S::ht_blk + tc::sw128_off(d + 1, ch) + (gtid & 7) * 2) = lo;
      }
      // H (fp32 [D][d]) -> bf16 H^T, K-major: row c, 64 j per 128-byte row, two j blocks
#pragma unroll
      for (int k = 0; k < NI; ++k) {
        const int i = gtid + k * 256, cc = i % d, jc = i / d;
        *reinterpret_cast<uint4*>(sm + S::ht + (jc >> 3) * S::ht_blk + tc::sw128_off(cc, jc & 7)) = tc::pack8_bf16(&hreg[k * 8]);
      }
      tc::fence_async_smem();
      tc::mbar_arrive(BAR(D3_HTREADY));

      // ---- tiles of unit n
      for (int tile = 0; tile < NT; ++tile, ++G) {
        const int i = G & 1;
        const int R = tile * 128 + t;
        const bool valid = R < lam || R - lam < eta;
        ok = WAIT(D3_UFULL + i, (uint32_t)(G >> 1)) && ok;
        tc::fence_after_sync();
        // q.k of this row (log2 units) and the warp's maxima: the score group turns them into weights
        float z[QH], wm[QH];
        {
          float zraw[QH];
          tc::tmem_ld2(tm_uz(i) + lane_addr + 64 + hf * QH, reinterpret_cast<float(&)[2]>(zraw));
#pragma unroll
          for (int r = 0; r < QH; ++r) {
            z[r] = valid ? zraw[r] * sl2 : -CUDART_INF_F;
            wm[r] = warp_max_redux(z[r]);
          }
        }
        // this thread's half of the feature map: hf = 0: softmax(u), hf = 1: softmax(-u)
        uint32_t pk2[32];
        {
          uint32_t u[64];
          tc::tmem_ld64u(tm_uz(i) + lane_addr, u);
          tc::phi_half(u, hf != 0, exp_kind, pk2);
        }
        if (G >= 2) {                                  // the score group is done with the buffers of the tile two before
          ok = WAIT(D3_PTREADY + i, (uint32_t)((G - 2) >> 1)) && ok;
          tc::fence_after_sync();
        }
        // bf16 pairs into tensor memory: the A operand of the second product (K index = feature j)
        tc::tmem_st32u(tm_phi(i) + lane_addr + hf * 32, pk2);
#pragma unroll
        for (int r = 0; r < QH; ++r) {
          X.z_s[i][hf * QH + r][t] = z[r];
          if (lane == 0) X.redmax[i][wq][hf * QH + r] = wm[r];
        }
        tc::fence_before_sync();
        tc::mbar_arrive(BAR(D3_PHIDONE + i));          // (release: the shared-memory writes above are visible to whoever acquires it)
      }
    }
  }
  else {
    // =================== score group ===================
    int G = 0;
    for (int n = 0; n < nU; ++n) {
      const int unit = unit_of(n), b = unit / L.Hkv, h = unit % L.Hkv, par = n & 1;
      float* scu = L.score + (size_t)unit * (lam + L.cmax);
      if (gtid < kDec2MaxTiles) { X.cand_key[gtid] = ~0ull; X.cand_score[gtid] = CUDART_INF_F; X.cand_min2[gtid] = CUDART_INF_F; X.cand_row[gtid] = 0; }
      // running maxima of q.k per query row (log2 units; every valid row counts, also the one that will be
      // folded: any m >= the true maximum leaves Eq. 14 unchanged) and this thread's share of the sums
      float lpart[QH], m_run[QR];
#pragma unroll
      for (int r = 0; r < QR; ++r) m_run[r] = 0.f;
#pragma unroll
      for (int r = 0; r < QH; ++r) lpart[r] = 0.f;
      for (int tile = 0; tile < NT; ++tile, ++G) {
        const int i = G & 1;
        const int R = tile * 128 + t;
        const bool is_g = R < lam;
        const int slot = R - lam;
        const bool scored = is_g || slot == s_ev;
        const int pos = is_g ? L.gpos[(size_t)unit * lam + R] : pos_ev;
        const uint8_t* vtile = sm + S::stage0 + (size_t)i * S::stage_bytes + S::st_v;
        uint8_t* ptile = sm + stage_pt(i);

        ok = WAIT(D3_VFULL + i, (uint32_t)(G >> 1)) && ok;
        ok = WAIT(D3_PDONE, (uint32_t)G) && ok;       // (its commit follows the feature group's arrival: z_s, redmax are visible)
        if (tile == 0) ok = WAIT(D3_LINDONE, (uint32_t)n) && ok;   // O^T holds the unit's linear term
        if (G >= 2) ok = WAIT(D3_ODONE + i, (uint32_t)((G - 2) >> 1)) && ok;   // the Pr^T operand of the tile two before was consumed
        tc::fence_after_sync();
        // ---- softmax weights of the tile (bf16; the sums use the rounded weights) into the Pr^T operand
        float pw[QH];
        {
          const bool valid = is_g || slot < eta;
          float m_new[QR];
          bool moved = false;
#pragma unroll
          for (int r = 0; r < QR; ++r) {
            m_new[r] = fmaxf(fmaxf(m_run[r], fmaxf(X.redmax[i][0][r], X.redmax[i][1][r])),
                             fmaxf(X.redmax[i][2][r], X.redmax[i][3][r]));
            moved = moved || (m_new[r] != m_run[r]);
          }
          if (moved) {                                 // uniform over the group and rare after the first tiles
            float alpha[QR];
#pragma unroll
            for (int r = 0; r < QR; ++r) alpha[r] = tc::fast_exp2(m_run[r] - m_new[r]);
#pragma unroll
            for (int r = 0; r < QH; ++r) lpart[r] *= hf ? alpha[QH + r] : alpha[r];
            if (hf == 0) {
              // O^T so far (the products up to the tile before, or the linear term) moves to the new maximum
              if (tile > 0) ok = WAIT(D3_ODONE + ((G - 1) & 1), (uint32_t)((G - 1) >> 1)) && ok;
              tc::fence_after_sync();
              float ov[4];
              tc::tmem_ld4(tm_o + lane_addr, ov);
#pragma unroll
              for (int r = 0; r < QR; ++r) ov[r] *= alpha[r];
              asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};\n\ttcgen05.wait::st.sync.aligned;\n" ::"r"(tm_o + lane_addr),
                           "r"(__float_as_uint(ov[0])), "r"(__float_as_uint(ov[1])), "r"(__float_as_uint(ov[2])), "r"(__float_as_uint(ov[3]))
                           : "memory");
            }
          }
#pragma unroll
          for (int r = 0; r < QR; ++r) m_run[r] = m_new[r];
#pragma unroll
          for (int r = 0; r < QH; ++r) {
            const int rr = hf * QH + r;
            const float mr = hf ? m_run[QH + r] : m_run[r];
            const uint32_t pb = pack_bf16x2(valid ? tc::fast_exp2(X.z_s[i][rr][t] - mr) : 0.f, 0.f);
            pw[r] = bf16lo_f(pb);
            *reinterpret_cast<unsigned short*>(ptile + (t >> 6) * 2048 + tc::sw128_off(rr, (t & 63) >> 3) + (t & 7) * 2) = (unsigned short)pb;
          }
        }
        // ---- Eq. 10: this thread's half of the value columns
        float score;
        {
          float dn[2];
          tc::tmem_ld2(tm_p + lane_addr + d, dn);
          const float den = dn[0] + dn[1];
          const float inv = den > 0.f ? 1.0f / den : 0.f;
          // packed pairs: d = v - P / den, four running sums of squares (columns 4k, 4k+1 | 4k+2, 4k+3)
          const uint64_t ninv2 = tc::pack_f2(-inv, -inv);
          uint64_t accA = tc::pack_f2(0.f, 0.f), accB = accA;
#pragma unroll
          for (int c0 = 0; c0 < HC; c0 += 32) {
            uint32_t p[32];
            tc::tmem_ld32u(tm_p + lane_addr + hf * HC + c0, p);
            if (c0 + 32 >= HC) {                 // [P | den] is read: the next tile's product may overwrite it
              tc::fence_before_sync();
              tc::mbar_arrive(BAR(D3_PFREE));
            }
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              const int cc = hf * HC + c0 + q8 * 8;
              const uint4 raw = *reinterpret_cast<const uint4*>(vtile + (cc >> 6) * 16384 + tc::sw128_off(t, (cc & 63) >> 3));
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
          if (hf == 1) X.ssp[t] = ss;
          tc::named_bar_sync(2, 256);
          score = sqrtf(ss + X.ssp[t]);           // hf = 1 threads double their own half; they do not use the score
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
          if (lane == 0) { X.redkey[wq] = k; X.red12[wq][0] = a1; X.red12[wq][1] = a2; }
        }
        tc::named_bar_sync(2, 256);
        unsigned long long tkey = X.redkey[0];
#pragma unroll
        for (int w = 1; w < 4; ++w) tkey = X.redkey[w] < tkey ? X.redkey[w] : tkey;
        // the row left out of O^T: both threads of the row know it from the row's position
        const unsigned long long rowkey_lo = (unsigned)(0x7fffffff - pos);
        const bool left_out = scored && (unsigned)tkey == (unsigned)rowkey_lo && tkey != ~0ull;
        if (left_out) {
          if (hf == 0) {
            float a1 = X.red12[0][0], a2 = X.red12[0][1];
#pragma unroll
            for (int w = 1; w < 4; ++w) {
              float b1 = X.red12[w][0], b2 = X.red12[w][1];
              float lo = fminf(a1, b1), hi = fmaxf(a1, b1);
              a2 = fminf(hi, fminf(a2, b2));
              a1 = lo;
            }
            X.cand_key[tile] = key;
            X.cand_score[tile] = score;
            X.cand_min2[tile] = a2;
            X.cand_row[tile] = R;
#pragma unroll
            for (int r = 0; r < QR; ++r) X.cand_z[tile][r] = X.z_s[i][r][t];
          } else {
#pragma unroll
            for (int ch = 0; ch < d / 8; ++ch)
              X.cand_v[tile][ch] = *reinterpret_cast<const uint4*>(vtile + (ch >> 3) * 16384 + tc::sw128_off(t, ch & 7));
          }
        }
        if (__any_sync(0xffffffffu, left_out)) {       // its feature row, read back from tensor memory (this thread's half)
          uint32_t pr[32];
          tc::tmem_ld32u(tm_phi(i) + lane_addr + hf * 32, pr);
          if (left_out) {
            uint32_t* dst = reinterpret_cast<uint32_t*>(&X.cand_phi[tile][0]) + hf * 32;
#pragma unroll
            for (int q = 0; q < 32; ++q) dst[q] = pr[q];
          }
        }
        // sums of the weights (the row left out takes its weights back)
#pragma unroll
        for (int r = 0; r < QH; ++r) {
          if (left_out) {
            const int rr = hf * QH + r;
            *reinterpret_cast<unsigned short*>(ptile + (t >> 6) * 2048 + tc::sw128_off(rr, (t & 63) >> 3) + (t & 7) * 2) = 0;
          } else {
            lpart[r] += pw[r];
          }
        }
        tc::fence_async_smem();
        tc::fence_before_sync();
        tc::mbar_arrive(BAR(D3_PTREADY + i));
      }

      // ---- end of unit n (this group alone; the other roles are already at work on unit n + 1).
      // O^T is complete once the last PV product is; it is read first, so that the next unit's linear term may
      // take its place
      {
        const int Gl = G - 1;
        ok = WAIT(D3_ODONE + (Gl & 1), (uint32_t)(Gl >> 1)) && ok;
        tc::fence_after_sync();
        if (hf == 0) {
          float ov[4];
          tc::tmem_ld4(tm_o + lane_addr, ov);
#pragma unroll
          for (int r = 0; r < QR; ++r) X.opart[t][r] = ov[r];
        }
        tc::fence_before_sync();
        tc::mbar_arrive(BAR(D3_OREAD));
      }
#pragma unroll
      for (int r = 0; r < QH; ++r) {
        float ls = warp_sum(lpart[r]);
        if (lane == 0) X.l_s[wq][hf * QH + r] = ls;
      }
      if (gtid == 0) {
#pragma unroll
        for (int r = 0; r < QR; ++r) X.m_s[r] = m_run[r];
      }
      tc::named_bar_sync(2, 256);
      const bool okb = X.abort_word == 0;
      // the pair to fold: lowest (score, then youngest) over the tiles' left-out rows
      int lt = 0;
      {
        unsigned long long best = X.cand_key[0];
        for (int i = 1; i < NT; ++i)
          if (X.cand_key[i] < best) { best = X.cand_key[i]; lt = i; }
      }
      const __nv_bfloat16* phiL = reinterpret_cast<const __nv_bfloat16*>(&X.cand_phi[lt][0]);
      const __nv_bfloat16* vL = reinterpret_cast<const __nv_bfloat16*>(&X.cand_v[lt][0]);
      if (gw < g) {                                   // phi(q) . phi_fold
        float a = 0.f;
        for (int j = lane; j < D; j += 32) a = fmaf(X.phiq_f[par][gw][j], __bfloat162float(phiL[j]), a);
        a = warp_sum(a);
        if (lane == 0) X.dotL[gw] = a;
      }
      // Eq. 13: H += phi_fold v_fold^T, s += phi_fold, as reductions performed at the L2 (nothing is read back)
      if (okb) {
        float* Hgw = L.H + (size_t)unit * D * d;
        constexpr int per_row4 = d / 4;
#pragma unroll 4
        for (int i = gtid; i < D * per_row4; i += 256) {
          const int j = i / per_row4, c4 = (i % per_row4) * 4;
          const float pj = __bfloat162float(phiL[j]);
          const uint2 vv = *reinterpret_cast<const uint2*>(vL + c4);
          red_add_v4(Hgw + (size_t)j * d + c4, pj * bf16lo_f(vv.x), pj * bf16hi_f(vv.x), pj * bf16lo_f(vv.y), pj * bf16hi_f(vv.y));
        }
        if (gtid < D) atomicAdd(L.s + (size_t)unit * D + gtid, __bfloat162float(phiL[gtid]));
      }
      tc::named_bar_sync(2, 256);                     // dotL
      // Eq. 14: thread (query row r, value column cc)
      if (okb) {
        for (int i = gtid; i < g * d; i += 256) {
          const int r = i / d, cc = i % d;
          const float m0 = X.m_s[r];
          const float mf = fmaxf(m0, X.zn[par][r]);
          const float a0 = tc::fast_exp2(m0 - mf);
          float l0 = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) l0 += X.l_s[w][r];
          float num = a0 * X.opart[cc][r];
          float den = a0 * l0;
          for (int ti = 0; ti < NT; ++ti) {
            if (ti == lt || X.cand_key[ti] == ~0ull) continue;
            const float p = round_bf16f(tc::fast_exp2(X.cand_z[ti][r] - mf));
            num = fmaf(p, __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(&X.cand_v[ti][0])[cc]), num);
            den += p;
          }
          const float pn = tc::fast_exp2(X.zn[par][r] - mf);
          num = fmaf(pn, X.vnew[par][cc], num);
          den += pn;
          const float e = tc::fast_exp2(-mf);
          num = fmaf(e * X.dotL[r], __bfloat162float(vL[cc]), num);
          den = fmaf(e, X.lden[par][r] + X.dotL[r], den);
          ((T*)c.out)[((size_t)b * L.Hq + h * g + r) * d + cc] = __float2bfloat16_rn(num / den);
        }
        // the evicted pair takes the folded member's slot (nothing moves when it is folded itself) and the new
        // pair enters the window ring; both were fetched in the unit's set-up
        const int rowL = X.cand_row[lt];
        constexpr int nch = d / 8;
        if (gtid < 2 * nch && rowL < lam) {
          T* dst = (gtid < nch ? (T*)L.gk : (T*)L.gv) + ((size_t)unit * lam + rowL) * d;
          *reinterpret_cast<uint4*>(dst + (gtid % nch) * 8) = X.ring_kv[par][gtid];
        }
        if (gtid >= 32 && gtid < 32 + 2 * nch) {
          const int i = gtid - 32;
          T* dst = (i < nch ? (T*)L.wk : (T*)L.wv) + ((size_t)unit * eta + s_ev) * d;
          *reinterpret_cast<uint4*>(dst + (i % nch) * 8) = X.new_kv[par][i];
        }
        if (gtid == 64 && rowL < lam) {
          L.gpos[(size_t)unit * lam + rowL] = pos_ev;
          scu[rowL] = scu[lam];
        }
        if (gtid == 96) {
          // lowest kept / highest folded score of this update
          float second = X.cand_min2[lt];
          for (int i = 0; i < NT; ++i)
            if (i != lt) second = fminf(second, X.cand_score[i]);
          L.thr[(size_t)unit * 2 + 0] = second;
          L.thr[(size_t)unit * 2 + 1] = X.cand_score[lt];
        }
      }
      tc::named_bar_sync(2, 256);                     // the lists of this unit are read: the next unit may fill them
      tc::mbar_arrive(BAR(D3_EPIDONE));
    }
  }

  // ---- every role is through its units (the thread that issued the last product has seen it complete)
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (X.abort_word != 0 && tid == 0) atomicOr(L.status, 8);
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

}  // namespace lola
