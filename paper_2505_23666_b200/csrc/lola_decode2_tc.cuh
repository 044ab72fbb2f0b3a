// The generation step (Eq. 11-14) as ONE kernel, organised as a pipeline of roles (the steady state of
// a bf16 layer with F = 64, caches full, one pair leaving the window; at most 8 row tiles per unit).
// Same arithmetic and the same per-tile products as k_decode_tc; what differs is who does what:
//
//   feature group (warps 0-7)   per tile: q.k columns and their warp maxima into shared memory, the
//                               feature map of U into tensor memory; no barrier inside the group
//   score group   (warps 8-15)  per tile: running maxima and softmax weights (bf16) into the Pr^T operand,
//                               Eq. 10 from [P | den] and the value tile, the running sums of the weights,
//                               and per row quadrant (a pair of warps) the lowest-scored pair so far
//   warp 16, one thread         issues [P | den] = phi [H | s] (and the linear term H^T phi(Q)^T once)
//   warp 17, one thread         issues O^T += V^T Pr^T; value-tile loads
//   warp 18, one thread         issues [U | Z] = K [W | Q^T]; key-tile loads
//
// The two groups work on different tiles at the same time: [U | Z] and phi are double-buffered in
// tensor memory, so while the score group is busy with tile t the feature group already works on
// tile t + 1 and the tensor core on the products between them.  Every hand-over is an mbarrier; every
// wait is bounded, and a wait that runs out raises the block's abort word (bit 8 of the status word).
//
// The pair to fold is only known after the last tile.  Every row is therefore attended by the O^T products;
// each quadrant keeps (q.k, stabiliser, value row, feature row) of its lowest-scored pair, and the epilogue
// takes the overall lowest out of O^T and the weight sums again (its bf16 weight times its bf16 value row is
// exact in fp32, so what is subtracted is what the product added, up to the rounding of the running sum).
// The score group's warps only meet their quadrant partner inside a tile (a 64-thread barrier); a slow warp
// holds up its partner and the hand-over to the O^T product, not the other quadrants.
#pragma once
#include "lola_decode_tc.cuh"

namespace lola {

constexpr int kDec2MaxTiles = 8;
constexpr int kDec2Threads = 608;      // 16 compute warps + 3 issuing warps
constexpr float kDec2Lazy = 8.0f;      // log2 units the running maximum may lag behind before O^T is rescaled

__device__ __forceinline__ int ld_global_i32(const int* p) {
  int v;
  asm volatile("ld.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

struct Decode2Misc {
  float qf[kDecQ][128];          // query rows, fp32
  float phiq_f[kDecQ][128];      // phi(q) rounded to bf16, as fp32
  float u_s[kDecQ][64];
  float knew[128], vnew[128];
  float s_f[128];                // the normaliser state s, fp32
  uint4 ring_kv[2 * 16];         // the pair that leaves the window (key chunks, then value chunks), bf16
  uint4 new_kv[2 * 16];          // the new pair, bf16
  float zn[kDecQ], lden[kDecQ], dotL[kDecQ];
  float redmax[2][4][kDecQ];
  float m_s[1][kDecQ];           // running maxima after the last tile (log2 units)
  float z_s[2][kDecQ][128];      // q.k of the tile's rows (log2 units)
  float ssp[2][128];             // partial squared errors of the second half of the value columns (by tile parity)
  float l_s[4][kDecQ];
  // the lowest-scored pair each of the four row quadrants has seen (its warp keeps the key in registers)
  unsigned long long wb_key[4];
  float wb_a1[4], wb_a2[4];      // the two lowest scores of the quadrant
  int wb_row[4];
  float wb_z[4][kDecQ];          // q.k of that row (log2 units) ...
  float wb_m[4][kDecQ];          // ... and the stabiliser its weights were taken at
  uint4 wb_v[4][16];             // value row, bf16
  uint4 wb_phi[4][16];           // feature row, bf16
  uint64_t bars[20];
  uint32_t tmem_slot;
  int abort_word;
};
static_assert(sizeof(Decode2Misc) <= 28672, "misc region too small");

__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t"
      "}\n"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}

// The tile loader as a real function: the issuing threads reach it from many places, and every inlined copy
// would add to an instruction footprint that four different roles already share.
template <int DPL>
__device__ __noinline__ void decode2_issue_tile(uint32_t dst, const CUtensorMap* tm_g, const CUtensorMap* tm_w, int tile, int nGB, int nRB,
                                                int unit, uint32_t bar) {
  decode_issue_tile<DPL>(dst, tm_g, tm_w, tile, nGB, nRB, unit, bar);
}

template <int DPL, int QR>
__global__ void __launch_bounds__(kDec2Threads, 1)
k_decode2_tc(Layer L, Call c, const __grid_constant__ CUtensorMap tm_gk, const __grid_constant__ CUtensorMap tm_gv,
             const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv, const uint4* wt_image) {
  using S = DecodeSmem<DPL>;
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
  Decode2Misc& X = *reinterpret_cast<Decode2Misc*>(sm + S::misc);

  const int unit = blockIdx.x, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int role = warp < 8 ? 0 : (warp < 16 ? 1 : warp - 14);   // 0 feature, 1 score, 2 / 3 / 4 issuing threads
  const int gtid = tid & 255;                // index inside a compute group
  const int gw = warp & 7;
  const int wq = gw & 3;                     // tensor-memory lane quadrant of this warp (= warp % 4)
  const int hf = gw >> 2;                    // which half of the row's work this thread does
  const int t = wq * 32 + lane;              // row of the tile = tensor-memory lane
  const int lam = L.lam, eta = L.eta, g = L.g;
  const int nGB = lam / 64, nRB = (eta + 63) / 64, NT = (nGB + nRB + 1) / 2;
  const int s_ev = c.n_seen % eta;           // ring slot of the pair that leaves = slot the new pair takes
  const int pos_ev = c.n_seen - eta;
  const float sl2 = L.scale * kLog2e;        // q.k in log2 units
  float* scu = L.score + (size_t)unit * (lam + L.cmax);
  volatile int* abw = &X.abort_word;

  const uint32_t bars = sbase + S::misc + (uint32_t)offsetof(Decode2Misc, bars);
  auto bar_kfull = [&](int i) { return bars + 8u * (uint32_t)i; };
  auto bar_vfull = [&](int i) { return bars + 16u + 8u * (uint32_t)i; };
  auto bar_u = [&](int i) { return bars + 32u + 8u * (uint32_t)i; };
  auto bar_phidone = [&](int i) { return bars + 48u + 8u * (uint32_t)i; };
  const uint32_t bar_p = bars + 64u, bar_pfree = bars + 72u;
  auto bar_ptready = [&](int i) { return bars + 80u + 8u * (uint32_t)i; };
  auto bar_o = [&](int i) { return bars + 96u + 8u * (uint32_t)i; };
  const uint32_t bar_w = bars + 112u, bar_phiq = bars + 120u, bar_ht = bars + 128u;
  auto bar_uread = [&](int i) { return bars + 136u + 8u * (uint32_t)i; };
  auto stage_k = [&](int i) { return sbase + S::stage0 + (uint32_t)i * S::stage_bytes + S::st_k; };
  auto stage_v = [&](int i) { return sbase + S::stage0 + (uint32_t)i * S::stage_bytes + S::st_v; };
  auto stage_pt = [&](int i) { return S::stage0 + (uint32_t)i * S::stage_bytes + S::st_pt; };   // offset from sm

  // everything the prologue needs from global memory is requested first, so that the round trips overlap
  const int pre_status = *reinterpret_cast<volatile const int*>(L.status);   // (acted on below: an earlier kernel failed: do nothing)
  float pre_s = 0.f, pre_k = 0.f, pre_v = 0.f;
  uint4 pre_q = make_uint4(0, 0, 0, 0);
  if (tid < D) pre_s = L.s[(size_t)unit * D + tid];
  if (tid < 16 * (d / 8) && tid / (d / 8) < g)
    pre_q = *reinterpret_cast<const uint4*>((const T*)c.q + ((size_t)b * L.Hq + h * g + tid / (d / 8)) * d + (tid % (d / 8)) * 8);
  uint4 pre_ring = make_uint4(0, 0, 0, 0), pre_new = pre_ring;
  if (tid >= 384 && tid < 384 + 2 * (d / 8)) {
    const int i = tid - 384, ch = i % (d / 8);
    const bool is_k = i < d / 8;
    pre_ring = *reinterpret_cast<const uint4*>((is_k ? (const T*)L.wk : (const T*)L.wv) + ((size_t)unit * eta + s_ev) * d + ch * 8);
    pre_new = *reinterpret_cast<const uint4*>((is_k ? (const T*)c.k : (const T*)c.v) + ((size_t)b * L.Hkv + h) * d + ch * 8);
  }
  if (tid >= 256 && tid < 256 + d) {
    pre_k = ldf<T>((const T*)c.k + ((size_t)b * L.Hkv + h) * d + (tid - 256));
    pre_v = ldf<T>((const T*)c.v + ((size_t)b * L.Hkv + h) * d + (tid - 256));
  }
  // H (fp32 [D][d]) straight into registers: compute thread x gathers, for DPL items (column c, 8 consecutive j),
  // the eight values H[j][c]; lanes = consecutive columns, so every load of a warp is one 128-byte line.  They
  // become the bf16 operand image H^T below; no staging buffer, so both stages stream key and value tiles from
  // the start
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

  if (tid == 0) {
    X.abort_word = 0;
    for (int i = 0; i < 19; ++i) {
      const bool group = (i == 6 || i == 7 || i == 9 || i == 10 || i == 11 || i >= 15);
      tc::mbar_init(bars + 8u * i, i == 16 ? 512u : (group ? 256u : 1u));   // (16: H^T written, by both groups)
    }
    tc::mbar_init_fence();
  }
  if (warp == 0) tc::tmem_alloc(&X.tmem_slot, 512);
  __syncthreads();
  if (pre_status != 0) {                             // the state's status word is set: leave the memories as they are
    if (warp == 0) tc::tmem_dealloc(X.tmem_slot, 512);
    return;
  }
  if (tid == 17 * 32) {
    // W^T straight into the operand rows; the first two tiles start to stream at once
    tc::mbar_expect_tx(bar_w, (uint32_t)kblk * 8192u);
    for (int kb = 0; kb < kblk; ++kb)
      tc::bulk_copy_g2s(sbase + S::b1 + (uint32_t)kb * S::b1_blk, wt_image + ((size_t)h * kblk + kb) * 512, 8192u, bar_w);
    decode2_issue_tile<DPL>(stage_k(0), &tm_gk, &tm_wk, 0, nGB, nRB, unit, bar_kfull(0));
    decode2_issue_tile<DPL>(stage_v(0), &tm_gv, &tm_wv, 0, nGB, nRB, unit, bar_vfull(0));
    if (NT > 1) {
      decode2_issue_tile<DPL>(stage_k(1), &tm_gk, &tm_wk, 1, nGB, nRB, unit, bar_kfull(1));
      decode2_issue_tile<DPL>(stage_v(1), &tm_gv, &tm_wv, 1, nGB, nRB, unit, bar_vfull(1));
    }
  }

  // ---- operands that stay for the whole unit (compute warps)
  if (role < 2) {
    // rows d, d+1: s as the sum of two bf16 parts (phi . s_hi + phi . s_lo keeps the fp32 normaliser)
    if (tid < D) {
      const float sv = pre_s;
      X.s_f[tid] = sv;
      const __nv_bfloat16 hi = __float2bfloat16_rn(sv);
      const __nv_bfloat16 lo = __float2bfloat16_rn(sv - __bfloat162float(hi));
      const int ch = (tid & 63) >> 3;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d, ch) + (tid & 7) * 2) = hi;
      *reinterpret_cast<T*>(sm + S::ht + (tid >> 6) * S::ht_blk + tc::sw128_off(d + 1, ch) + (tid & 7) * 2) = lo;
    }
    // rows d+2 .. d+15 of both j blocks: zero
    for (int i = tid; i < 2 * 14 * 8; i += 512) {
      const int jb = i / (14 * 8), r = (i / 8) % 14, ch = i % 8;
      *reinterpret_cast<uint4*>(sm + S::ht + jb * S::ht_blk + tc::sw128_off(d + 2 + r, ch)) = make_uint4(0, 0, 0, 0);
    }
    // query rows: B1 rows 64..79 (rows >= g are zero) and an fp32 copy
    constexpr int per_row = d / 8;
    if (tid < 16 * per_row) {
      const int r = tid / per_row, ch = tid % per_row;
      const uint4 val = pre_q;
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
    if (tid >= 384 && tid < 384 + 2 * (d / 8)) {
      X.ring_kv[tid - 384] = pre_ring;
      X.new_kv[tid - 384] = pre_new;
    }
    if (tid >= 256 && tid < 256 + d) {
      X.knew[tid - 256] = pre_k;
      X.vnew[tid - 256] = pre_v;
    }
    // zero phi(Q) and both Pr^T tiles
    for (int i = tid; i < 256; i += 512) {
      *reinterpret_cast<uint4*>(sm + S::phiq + i * 16) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(sm + stage_pt(0) + i * 16) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(sm + stage_pt(1) + i * 16) = make_uint4(0, 0, 0, 0);
    }
    tc::fence_async_smem();
  }
  __syncthreads();

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

  if (role < 2) {
    // H -> bf16 H^T, K-major: row c, 64 j per 128-byte row, two j blocks (lanes = consecutive columns: no conflicts)
#pragma unroll
    for (int n = 0; n < DPL; ++n) {
      const int it = tid + 512 * n, cc = it % d, jc = it / d;
      *reinterpret_cast<uint4*>(sm + S::ht + (jc >> 3) * S::ht_blk + tc::sw128_off(cc, jc & 7)) = tc::pack8_bf16(pre_h[n]);
    }
    tc::fence_async_smem();
    tc::mbar_arrive(bar_ht);
  }

  if (role == 2) {
    // =================== [P | den] products ===================
    if (lane == 0) {
      // operand descriptor: the address field (units of 16 bytes) takes the offset of a K step
      const uint64_t dht = tc::make_desc_sw128(sbase + S::ht, 16, 1024);
      for (int tile = 0; tile < NT; ++tile) {
        const int i = tile & 1;
        ok = tc::mbar_wait(bar_phidone(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;   // phi(tile) is in tensor memory
        tc::fence_after_sync();
        if (tile == 0) {
          ok = tc::mbar_wait(bar_ht, 0, abw) && ok;                              // H^T is in place
        } else {
          ok = tc::mbar_wait(bar_pfree, (uint32_t)(tile - 1) & 1u, abw) && ok;   // [P | den] of the tile before is read
        }
        tc::fence_after_sync();
        const uint32_t tph = tm_phi(i);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          tc::mma_bf16_ts(tm_p, tph + ks * 8, dht + (uint64_t)(((ks >> 2) * S::ht_blk + (ks & 3) * 32) >> 4), idesc2, ks > 0);
        tc::mma_commit(bar_p);
        if (tile == 0) {
          // O^T starts as the linear term H^T phi(Q)^T, with weight exp(0 - m), m = 0 so far; the first O^T
          // product waits for it
          ok = tc::mbar_wait(bar_phiq, 0, abw) && ok;
          tc::fence_after_sync();
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks)
            tc::mma_bf16_ss(tm_o, tc::make_desc_sw128(sbase + S::ht + (ks >> 2) * S::ht_blk + (ks & 3) * 32, 16, 1024),
                            tc::make_desc_sw128(sbase + S::phiq + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024), idesc0, ks > 0);
          tc::mma_commit(bar_o(0));
        }
      }
    }
    __syncwarp();
  } else if (role == 4) {
    // =================== [U | Z] products, key tiles ===================
    if (lane == 0) {
      const uint64_t dk0 = tc::make_desc_sw128(stage_k(0), 16, 1024), dk1 = tc::make_desc_sw128(stage_k(1), 16, 1024);
      const uint64_t db1 = tc::make_desc_sw128(sbase + S::b1, 16, 1024);
      ok = tc::mbar_wait(bar_w, 0, abw) && ok;
      for (int tile = 0; tile < NT; ++tile) {
        const int i = tile & 1;
        ok = tc::mbar_wait(bar_kfull(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;
        if (tile >= 2)                               // the feature group has read [U | Z] of tile - 2
          ok = tc::mbar_wait(bar_uread(i), (uint32_t)((tile - 2) >> 1) & 1u, abw) && ok;
        tc::fence_after_sync();
        const uint64_t dk = i ? dk1 : dk0;
        const uint32_t tmu = tm_uz(i);
#pragma unroll
        for (int ks = 0; ks < d / 16; ++ks)
          tc::mma_bf16_ss(tmu, dk + (uint64_t)(((ks >> 2) * 16384 + (ks & 3) * 32) >> 4),
                          db1 + (uint64_t)(((ks >> 2) * S::b1_blk + (ks & 3) * 32) >> 4), idesc1, ks > 0);
        tc::mma_commit(bar_u(i));
        if (tile + 2 < NT) {                         // the tile after next streams into this buffer once the product has read it
          ok = tc::mbar_wait(bar_u(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;
          decode2_issue_tile<DPL>(stage_k(i), &tm_gk, &tm_wk, tile + 2, nGB, nRB, unit, bar_kfull(i));
        }
      }
    }
    __syncwarp();
  } else if (role == 3) {
    // =================== O^T products, value tiles ===================
    if (lane == 0) {
      const uint64_t dv0 = tc::make_desc_sw128(stage_v(0), 16384, 1024), dv1 = tc::make_desc_sw128(stage_v(1), 16384, 1024);
      const uint64_t dp0 = tc::make_desc_sw128(sbase + stage_pt(0), 16, 1024), dp1 = tc::make_desc_sw128(sbase + stage_pt(1), 16, 1024);
      for (int tile = 0; tile < NT; ++tile) {
        const int i = tile & 1;
        ok = tc::mbar_wait(bar_ptready(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;
        if (tile == 0) ok = tc::mbar_wait(bar_o(0), 0, abw) && ok;   // the linear term is in O^T
        tc::fence_after_sync();
        const uint64_t dv = i ? dv1 : dv0, dp = i ? dp1 : dp0;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          tc::mma_bf16_ss(tm_o, dv + (uint64_t)((ks * 2048) >> 4), dp + (uint64_t)(((ks >> 2) * 2048 + (ks & 3) * 32) >> 4), idesc3, 1u);
        const int ev = tile + 1;                                      // completion event of this product
        tc::mma_commit(bar_o(ev & 1));
        ok = tc::mbar_wait(bar_o(ev & 1), (uint32_t)(ev >> 1) & 1u, abw) && ok;
        if (tile + 2 < NT) decode2_issue_tile<DPL>(stage_v(i), &tm_gv, &tm_wv, tile + 2, nGB, nRB, unit, bar_vfull(i));
      }
    }
    __syncwarp();
  } else if (role == 0) {
    // =================== feature group ===================
    // this thread's query rows: [hf * QH, hf * QH + QH)
    const bool exp_kind = L.phi_kind == 1;
    for (int tile = 0; tile < NT; ++tile) {
      const int i = tile & 1;
      const int R = tile * 128 + t;
      const bool valid = R < lam || R - lam < eta;
      ok = tc::mbar_wait(bar_u(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;
      tc::fence_after_sync();
      // [U | Z] of this row in one round trip to tensor memory: this thread's q.k columns (log2 units after
      // scaling; their warp maxima go to the score group, which turns them into weights) and all of U
      float z[QH], wm[QH];
      uint32_t pk2[32];
      {
        uint32_t u[64], zraw[QH];
        if (QH == 4) tc::tmem_ld64u_and4(tm_uz(i) + lane_addr, u, tm_uz(i) + lane_addr + 64 + hf * QH, reinterpret_cast<uint32_t(&)[4]>(zraw));
        else tc::tmem_ld64u_and2(tm_uz(i) + lane_addr, u, tm_uz(i) + lane_addr + 64 + hf * QH, reinterpret_cast<uint32_t(&)[2]>(zraw));
        tc::fence_before_sync();
        tc::mbar_arrive(bar_uread(i));               // [U | Z] of this tile is in registers: the buffer may take tile + 2
#pragma unroll
        for (int r = 0; r < QH; ++r) {
          z[r] = valid ? __uint_as_float(zraw[r]) * sl2 : -CUDART_INF_F;
          wm[r] = warp_max_redux(z[r]);
        }
        // this thread's half of the feature map: hf = 0: softmax(u), hf = 1: softmax(-u)
        tc::phi_half(u, hf != 0, exp_kind, pk2);
      }
      if (tile >= 2) {                               // the score group is done with the buffers of tile - 2
        ok = tc::mbar_wait(bar_ptready(i), (uint32_t)((tile - 2) >> 1) & 1u, abw) && ok;
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
      tc::mbar_arrive(bar_phidone(i));               // (release: the shared-memory writes above are visible to whoever acquires it)
    }
  } else {
    // =================== score group ===================
    // first: what the linear term needs.  u = q W on the CUDA cores (g rows only) from the W^T operand image
    ok = tc::mbar_wait(bar_w, 0, abw) && ok;
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
    tc::named_bar_sync(2, 256);
    // phi(q), its normaliser phi(q) . s and q . k_new
    if (gw < g) {
      const int r = gw;
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
        ld = fmaf(vals[q], X.s_f[j], ld);
      }
      ld = warp_sum(ld);
      float zz = 0.f;
      for (int j = lane; j < d; j += 32) zz = fmaf(X.qf[r][j], X.knew[j], zz);
      zz = warp_sum(zz);
      if (lane == 0) { X.lden[r] = ld; X.zn[r] = zz * sl2; }
    }
    tc::fence_async_smem();
    tc::mbar_arrive(bar_phiq);                       // phi(Q) is in its operand rows

    // running maxima of q.k per query row (log2 units; every valid row counts, also the one that will be
    // folded: any m >= the true maximum leaves Eq. 14 unchanged) and this thread's share of the sums
    float lpart[QH], m_run[QR];
    unsigned long long w_key = ~0ull;                // lowest (score, then youngest) pair of this warp's rows so far
    float w_a1 = CUDART_INF_F, w_a2 = CUDART_INF_F;  // the two lowest scores of this warp's rows so far
#pragma unroll
    for (int r = 0; r < QR; ++r) m_run[r] = 0.f;
#pragma unroll
    for (int r = 0; r < QH; ++r) lpart[r] = 0.f;
    // token position of this thread's row, fetched one tile ahead (its round trip to the L2 would otherwise sit
    // in front of the lowest-score reduction of every tile)
    const int* gpos_u = L.gpos + (size_t)unit * lam;
    int pos_next = t < lam ? ld_global_i32(gpos_u + t) : pos_ev;
    for (int tile = 0; tile < NT; ++tile) {
      const int i = tile & 1;
      const int R = tile * 128 + t;
      const bool is_g = R < lam;
      const int slot = R - lam;
      const bool scored = is_g || slot == s_ev;
      const int pos = pos_next;
      pos_next = (tile + 1 < NT && R + 128 < lam) ? ld_global_i32(gpos_u + R + 128) : pos_ev;
      const uint8_t* vtile = sm + S::stage0 + (size_t)i * S::stage_bytes + S::st_v;
      uint8_t* ptile = sm + stage_pt(i);

      ok = tc::mbar_wait(bar_vfull(i), (uint32_t)(tile >> 1) & 1u, abw) && ok;
      ok = tc::mbar_wait(bar_p, (uint32_t)tile & 1u, abw) && ok;   // (its commit follows the feature group's arrival: z_s, redmax are visible)
      if (tile >= 2) {                               // the Pr^T operand of tile - 2 was consumed by its O^T product
        const int ev = tile - 1;
        ok = tc::mbar_wait(bar_o(ev & 1), (uint32_t)(ev >> 1) & 1u, abw) && ok;
      }
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
          moved = moved || (m_new[r] > m_run[r] + kDec2Lazy);
        }
        // The stabiliser only follows the maximum when it has run away by more than 2^kDec2Lazy: any m within
        // that distance of the true maximum leaves Eq. 14 unchanged (weights up to 2^kDec2Lazy are exact in
        // bf16's and fp32's range), and moving it means waiting for the O^T product of the tile before.
        if (moved) {                                 // uniform over the group, rare
          float alpha[QR];
#pragma unroll
          for (int r = 0; r < QR; ++r) alpha[r] = tc::fast_exp2(m_run[r] - m_new[r]);
#pragma unroll
          for (int r = 0; r < QH; ++r) lpart[r] *= hf ? alpha[QH + r] : alpha[r];
          if (hf == 0) {
            // O^T so far (the products up to the tile before, or the linear term) moves to the new maximum
            ok = tc::mbar_wait(bar_o(tile & 1), (uint32_t)(tile >> 1) & 1u, abw) && ok;
            tc::fence_after_sync();
            float ov[8];
            tc::tmem_ld8(tm_o + lane_addr, ov);
#pragma unroll
            for (int r = 0; r < QR; ++r) ov[r] *= alpha[r];
            tc::tmem_st8(tm_o + lane_addr, ov);
          }
          // all rows move together
#pragma unroll
          for (int r = 0; r < QR; ++r) m_run[r] = m_new[r];
        }
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
      float ss;
      {
        // packed pairs: d = v - P / den, four running sums of squares (columns 4k, 4k+1 | 4k+2, 4k+3)
        uint64_t ninv2 = 0;
        uint64_t accA = tc::pack_f2(0.f, 0.f), accB = accA;
#pragma unroll
        for (int c0 = 0; c0 < HC; c0 += 32) {
          uint32_t p[32];
          if (c0 == 0) {                                 // the two parts of the denominator come with the first columns
            uint32_t dn[2];
            tc::tmem_ld32u_and2(tm_p + lane_addr + hf * HC, p, tm_p + lane_addr + d, dn);
            const float den = __uint_as_float(dn[0]) + __uint_as_float(dn[1]);
            const float inv = den > 0.f ? 1.0f / den : 0.f;
            ninv2 = tc::pack_f2(-inv, -inv);
          } else {
            tc::tmem_ld32u(tm_p + lane_addr + hf * HC + c0, p);
          }
          if (c0 + 32 >= HC) {                 // [P | den] is read: the next tile's product may overwrite it
            tc::fence_before_sync();
            tc::mbar_arrive(bar_pfree);
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
        ss = (a0 + a1) + (a2 + a3);
      }
      // every row stays in O^T and in the sums; the one pair that is folded in the end is taken out again
      // after the last tile, so nothing here needs the other quadrants
#pragma unroll
      for (int r = 0; r < QH; ++r) lpart[r] += pw[r];
      if (hf == 1) X.ssp[i][t] = ss;
      tc::named_bar_sync(4 + wq, 64);                // the two warps of this row quadrant
      if (hf == 0) {
        const float score = sqrtf(ss + X.ssp[i][t]);
        if (scored && ok) scu[is_g ? R : lam] = score;
        // lowest score of the quadrant's rows in this tile (ties: the younger pair) and the runner-up;
        // scores are norms (>= 0): their bit patterns order like unsigned integers
        const unsigned sb = scored ? __float_as_uint(score) : 0xffffffffu;
        const unsigned smin = __reduce_min_sync(0xffffffffu, sb);
        const unsigned tb_ = (sb == smin && scored) ? (unsigned)(0x7fffffff - pos) : 0xffffffffu;
        const unsigned tmin = __reduce_min_sync(0xffffffffu, tb_);
        const bool is_min = scored && sb == smin && tb_ == tmin;
        const unsigned s2 = __reduce_min_sync(0xffffffffu, is_min ? 0xffffffffu : sb);
        const float c1 = smin == 0xffffffffu ? CUDART_INF_F : __uint_as_float(smin);
        const float c2 = s2 == 0xffffffffu ? CUDART_INF_F : __uint_as_float(s2);
        w_a2 = fminf(fmaxf(w_a1, c1), fminf(w_a2, c2));
        w_a1 = fminf(w_a1, c1);
        const unsigned long long k = smin != 0xffffffffu ? (((unsigned long long)smin << 32) | tmin) : ~0ull;
        if (k < w_key) {                             // (uniform over the warp) a new lowest pair of this quadrant:
          w_key = k;                                 // keep what the fold and Eq. 14 need of it
          const int src = __ffs(__ballot_sync(0xffffffffu, is_min)) - 1;
          uint32_t pr[32];
#pragma unroll
          for (int half = 0; half < 2; ++half) {     // its feature row, read back from tensor memory
            tc::tmem_ld32u(tm_phi(i) + lane_addr + half * 32, pr);
            if (is_min) {
              uint4* dst = &X.wb_phi[wq][half * 8];
#pragma unroll
              for (int q = 0; q < 8; ++q) dst[q] = make_uint4(pr[4 * q], pr[4 * q + 1], pr[4 * q + 2], pr[4 * q + 3]);
            }
          }
          if (lane < d / 8)                          // its value row: one 16-byte piece per lane
            X.wb_v[wq][lane] = *reinterpret_cast<const uint4*>(vtile + (lane >> 3) * 16384 + tc::sw128_off(wq * 32 + src, lane & 7));
          if (is_min) {
            X.wb_row[wq] = R;
#pragma unroll
            for (int r = 0; r < QR; ++r) {
              X.wb_z[wq][r] = X.z_s[i][r][t];
              X.wb_m[wq][r] = m_run[r];
            }
          }
        }
      }
      tc::fence_async_smem();
      tc::fence_before_sync();
      tc::mbar_arrive(bar_ptready(i));
    }
    if (hf == 0 && lane == 0) { X.wb_key[wq] = w_key; X.wb_a1[wq] = w_a1; X.wb_a2[wq] = w_a2; }
#pragma unroll
    for (int r = 0; r < QH; ++r) {
      float ls = warp_sum(lpart[r]);
      if (lane == 0) X.l_s[wq][hf * QH + r] = ls;
    }
    if (gtid == 0) {
#pragma unroll
      for (int r = 0; r < QR; ++r) X.m_s[0][r] = m_run[r];
    }
  }

  // ---- after the last tile the two compute groups split the rest: the feature group folds (Eq. 13), the score
  // group writes the outputs (Eq. 14) and the memories; the issuing warps go straight to the end
  if (role < 2) {
    tc::fence_before_sync();
    tc::named_bar_sync(9, 512);                      // the score group has finished the last tile
    tc::fence_after_sync();
    // the pair to fold: lowest (score, then youngest) over the four quadrants
    int lt = 0;
    {
      unsigned long long best = X.wb_key[0];
#pragma unroll
      for (int i = 1; i < 4; ++i)
        if (X.wb_key[i] < best) { best = X.wb_key[i]; lt = i; }
    }
    const __nv_bfloat16* phiL = reinterpret_cast<const __nv_bfloat16*>(&X.wb_phi[lt][0]);
    const __nv_bfloat16* vL = reinterpret_cast<const __nv_bfloat16*>(&X.wb_v[lt][0]);
    // the stage the last tile did not use is free once the O^T product of the tile before the last is complete
    const uint32_t free_stage = S::stage0 + (uint32_t)(NT & 1) * S::stage_bytes;
    if (role == 0) {
      // ---- Eq. 13: H += phi_fold v_fold^T.  The update (fp32 [D][d], the layout of H) is staged in the free
      // stage and added to H by bulk reductions: the additions happen at the L2, nothing is read back
      if (NT >= 2) ok = tc::mbar_wait(bar_o((NT - 1) & 1), (uint32_t)((NT - 1) >> 1) & 1u, abw) && ok;
      const bool okb = X.abort_word == 0;
      if (okb) {
        constexpr int per_row = d / 4;
        float4* dH = reinterpret_cast<float4*>(sm + free_stage);
        for (int i = tid; i < D * per_row; i += 256) {
          const int j = i / per_row, c4 = (i % per_row) * 4;
          const float pj = __bfloat162float(phiL[j]);
          const uint2 vv = *reinterpret_cast<const uint2*>(vL + c4);
          dH[i] = make_float4(pj * bf16lo_f(vv.x), pj * bf16hi_f(vv.x), pj * bf16lo_f(vv.y), pj * bf16hi_f(vv.y));
        }
        tc::fence_async_smem();
      }
      tc::named_bar_sync(10, 256);
      if (okb && tid == 0) {
        float* Hgw = L.H + (size_t)unit * D * d;
        constexpr uint32_t half_bytes = (uint32_t)(D * d * 4 / 2);
        tc::bulk_reduce_add_f32(Hgw, sbase + free_stage, half_bytes);
        tc::bulk_reduce_add_f32(Hgw + D * d / 2, sbase + free_stage + half_bytes, half_bytes);
        tc::bulk_commit_group();
      }
      if (okb && tid < D) atomicAdd(L.s + (size_t)unit * D + tid, __bfloat162float(phiL[tid]));
    } else {
      if (gw < g) {                                  // phi(q) . phi_fold
        const int r = gw;
        float a = 0.f;
        for (int j = lane; j < D; j += 32) a = fmaf(X.phiq_f[r][j], __bfloat162float(phiL[j]), a);
        a = warp_sum(a);
        if (lane == 0) X.dotL[r] = a;
      }
      // O^T is complete with the product of the last tile
      ok = tc::mbar_wait(bar_o(NT & 1), (uint32_t)(NT >> 1) & 1u, abw) && ok;
      tc::fence_after_sync();
      float* opart = reinterpret_cast<float*>(sm + free_stage + S::st_pt);   // [128][QR], in the free stage's Pr^T tile
      if (gw < 4) {
        float ov[8];
        tc::tmem_ld8(tm_o + lane_addr, ov);
#pragma unroll
        for (int r = 0; r < QR; ++r) opart[t * QR + r] = ov[r];
      }
      tc::named_bar_sync(11, 256);
      const bool okb = X.abort_word == 0;
      // ---- Eq. 14: thread (query row r, value column cc)
      if (okb) {
        for (int i = gtid; i < g * d; i += 256) {
          const int r = i / d, cc = i % d;
          const float m0 = X.m_s[0][r];              // the score group left the final maxima there
          const float mf = fmaxf(m0, X.zn[r]);
          const float a0 = tc::fast_exp2(m0 - mf);
          float l0 = 0.f;
#pragma unroll
          for (int w = 0; w < 4; ++w) l0 += X.l_s[w][r];
          // the folded pair leaves the softmax part again: its weight as the tile's product used it (bf16, taken
          // at the stabiliser of that tile), brought to the final stabiliser like everything else in O^T
          const float vLc = __bfloat162float(vL[cc]);
          const float pL = round_bf16f(tc::fast_exp2(X.wb_z[lt][r] - X.wb_m[lt][r])) * tc::fast_exp2(X.wb_m[lt][r] - m0);
          float num = a0 * fmaf(-pL, vLc, opart[cc * QR + r]);
          float den = a0 * (l0 - pL);
          const float pn = tc::fast_exp2(X.zn[r] - mf);
          num = fmaf(pn, X.vnew[cc], num);
          den += pn;
          const float e = tc::fast_exp2(-mf);
          num = fmaf(e * X.dotL[r], vLc, num);
          den = fmaf(e, X.lden[r] + X.dotL[r], den);
          ((T*)c.out)[((size_t)b * L.Hq + h * g + r) * d + cc] = __float2bfloat16_rn(num / den);
        }
        // ---- the evicted pair takes the folded member's slot (nothing moves when it is folded itself) and
        // the new pair enters the window ring; both were fetched at the start
        const int rowL = X.wb_row[lt];
        constexpr int nch = d / 8;
        if (gtid < 2 * nch && rowL < lam) {
          T* dst = (gtid < nch ? (T*)L.gk : (T*)L.gv) + ((size_t)unit * lam + rowL) * d;
          *reinterpret_cast<uint4*>(dst + (gtid % nch) * 8) = X.ring_kv[gtid];
        }
        if (gtid >= 32 && gtid < 32 + 2 * nch) {
          const int i = gtid - 32;
          T* dst = (i < nch ? (T*)L.wk : (T*)L.wv) + ((size_t)unit * eta + s_ev) * d;
          *reinterpret_cast<uint4*>(dst + (i % nch) * 8) = X.new_kv[i];
        }
        if (gtid == 64 && rowL < lam) {
          L.gpos[(size_t)unit * lam + rowL] = pos_ev;
          scu[rowL] = scu[lam];
        }
        if (gtid == 96) {
          // lowest kept / highest folded score of this update
          float second = X.wb_a2[lt];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (i != lt) second = fminf(second, X.wb_a1[i]);
          L.thr[(size_t)unit * 2 + 0] = second;
          L.thr[(size_t)unit * 2 + 1] = X.wb_a1[lt];
        }
      }
    }
  }
  if (tid == 0) tc::bulk_wait_group_read();        // the bulk reductions have read shared memory (they are performed by the end of the kernel)
  tc::fence_before_sync();
  __syncthreads();
  if (tid == 0 && X.abort_word != 0) atomicOr(L.status, 8);
  if (warp == 0) tc::tmem_dealloc(tmem, 512);
}

}  // namespace lola
