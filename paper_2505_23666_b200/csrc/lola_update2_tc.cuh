// Eq. 12 and Eq. 13 of the chunkwise update in one kernel (bf16 layer, F = 64), one CTA per unit:
//   1. exact top-lambda of the eligible set by (score descending, older first): the n_fold = |E| - lambda
//      lowest keys are found with a 4-pass byte radix select over the score bits; ties on the
//      threshold score are resolved by position (the younger pair is folded first);
//   2. ordered compaction into three lists (pairs to fold, freed slots, leaving pairs that stay);
//   3. the folded pairs are gathered into operand tiles, phi(K_S) is recomputed
//      (tcgen05.mma K_S W, feature map with one thread pair per row, rounded to bf16) and
//      [dH | ds] = phi(K_S)^T [V_S | 1]   (tcgen05.mma, M = 128 features, N = d + 16, K = folded pairs)
//      is added to H, s.  Eq. 13 folds phi(k) itself into the fp32 state: phi goes in as two bf16 parts
//      (hi in operand rows 0..63, lo = phi - hi in rows 64..127, the value rows repeated), so the product
//      carries 16 significant bits of phi at no extra instruction.  The new H is also written as the bf16
//      operand image the other kernels load;
//   4. leaving pairs that stay move into the freed slots; the incoming pairs enter the window ring.
// Every wait on an mbarrier is bounded; a wait that runs out sets bit 32 of the status word.
#pragma once
#include <cuda.h>

#include "lola_decode_tc.cuh"
#include "lola_generic.cuh"
#include "lola_tc.cuh"

namespace lola {

constexpr int kUp2Threads = 512;
constexpr int kUp2MaxE = 4096;      // eligible pairs this kernel handles (scores and positions in shared memory)
constexpr int kUp2MaxFold = 64;     // folded pairs per call (half an operand tile: the other half holds the low parts)

template <int DPL>
struct Update2Smem {
  static constexpr int d = DPL * 32;
  static constexpr int kblk = d / 64;
  static constexpr uint32_t b1 = 0;                        // W^T, K-major: [kblk][64][128B]
  static constexpr uint32_t kt = 16384;                    // K_S tile, K-major [kblk][128][128B]; then phi tile [2][128][128B]
  static constexpr uint32_t vt = kt + 32768;               // [V_S | 1], MN-major: [kblk + 1 column blocks][128 pairs][128B]
  static constexpr uint32_t misc = vt + 3 * 16384;
  static constexpr uint32_t hs = misc + 2 * kUp2MaxE * 4 + 8192;   // H of the unit, fp32, rows padded by 4 floats
  static constexpr uint32_t hs_row = (d + 4) * 4;
  static constexpr uint32_t total = hs + 128 * hs_row;
  static constexpr uint32_t bytes = total + 1024;
};

struct Update2Misc {
  unsigned key[kUp2MaxE];           // score bits
  int pos[kUp2MaxE];                // position; bit 31 set once the pair is chosen for folding
  unsigned hist[4][256];
  int scan[kUp2Threads / 32][3];
  int fold_e[kUp2MaxFold];          // E indices of the folded pairs, ascending
  int free_slot[kUp2MaxFold];       // sparse-cache slots of folded members, ascending
  int mover[kUp2MaxFold];           // leaving-pair indices that stay, ascending
  unsigned min_keep;
  int n_equal;
  int equal_e[kUp2MaxFold];         // pairs whose score equals the selection threshold
  unsigned char fold_mark[kUp2MaxFold];
  uint64_t bars[2];
  uint32_t tmem_slot;
};
static_assert(sizeof(Update2Misc) <= 2 * kUp2MaxE * 4 + 8192, "misc region too small");

// PHASE 1: selection only (steps 1-2; the lists go to the state's work-list arrays, so it can run beside
// the attention kernel, which only reads the memories).  PHASE 2: steps 3-4 from those lists.
// The body works on one unit with a block of kUp2Threads threads and `sm`, 1024-byte aligned dynamic shared
// memory (PHASE 1 needs sizeof(Update2Misc) bytes of it, the others Update2Smem<DPL>::total); the scoring
// kernel runs PHASE 1 in its last block of a unit.
template <int DPL, int PHASE>
__device__ __forceinline__ void update2_body(const Layer& L, const Call& c, const uint4* wt_image, __nv_bfloat16* ht_image,
                                             uint8_t* sm, const int unit) {
  using S = Update2Smem<DPL>;
  constexpr int d = DPL * 32;
  constexpr int kblk = d / 64;
  constexpr int D = 128;
  constexpr int nch = d / 8;
  typedef __nv_bfloat16 T;
  const uint32_t sbase = tc::smem_u32(sm);
  constexpr uint32_t kMisc = PHASE == 1 ? 0u : S::misc;          // the selection needs the small arrays only
  Update2Misc& X = *reinterpret_cast<Update2Misc*>(sm + kMisc);

  const int b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int lam = L.lam, eta = L.eta;
  // PHASE 2 also serves calls that fold nothing (nothing leaves the window yet, or every leaving pair
  // still finds a free slot): then only the moves and the window roll run
  const bool fold = c.mode == UPD_SELECT;
  const int cg = c.count_g, nE = cg + c.r, nF = fold ? nE - lam : 0;   // folding: 1 <= nF <= min(r, kUp2MaxFold)
  float* scu = L.score + (size_t)unit * (lam + L.cmax);
  const uint32_t bar = sbase + kMisc + (uint32_t)offsetof(Update2Misc, bars);
  int* g_fold = L.fold_idx + (size_t)unit * L.cmax;
  int* g_src = L.move_src + (size_t)unit * L.cmax;
  int* g_dst = L.move_dst + (size_t)unit * L.cmax;
  int* g_cnt = L.counts + (size_t)unit * 4;
  uint32_t ph = 0;
  bool ok = true;

  if (tid == 0) { tc::mbar_init(bar, 1); tc::mbar_init_fence(); X.min_keep = 0xffffffffu; X.n_equal = 0; }
  if (PHASE != 1 && fold && warp == 0) tc::tmem_alloc(&X.tmem_slot, 256);
  if (PHASE == 2) {
    // launched early (programmatic dependent launch): the zeroed operand tiles need nothing from memory
    if (tid == 0) tc::grid_dep_launch_dependents();
    if (fold)
      for (int i = tid; i < (32768 + 3 * 16384) / 16; i += kUp2Threads)
        *reinterpret_cast<uint4*>(sm + S::kt + i * 16) = make_uint4(0, 0, 0, 0);
    tc::grid_dep_wait();                             // the attention kernel has read the memories this kernel changes
  }
  // everything the set-up needs from global memory is requested at once (one round trip): the work lists
  // and their counts, the W^T image
  int pre_cnt = 0, pre_fold = 0, pre_src = 0, pre_dst = 0;
  uint4 pre_w[kblk];
  if (PHASE == 2) {
    pre_cnt = g_cnt[1];
    if (tid < nF) pre_fold = g_fold[tid];
    if (tid < min(L.cmax, kUp2MaxFold)) { pre_src = g_src[tid]; pre_dst = g_dst[tid]; }
    if (fold) {
      const uint4* img = wt_image + (size_t)h * kblk * 512;
#pragma unroll
      for (int q = 0; q < kblk; ++q) pre_w[q] = img[tid + q * kUp2Threads];
    }
  }
  // H of the unit streams into shared memory (asynchronous 16-byte copies) meanwhile.  PHASE 2 never reads H:
  // it adds the fold's product to H in memory (reductions at the L2) and keeps no operand image
  if (PHASE == 0 && fold) {
    const float* Hg = L.H + (size_t)unit * D * d;
    for (int i = tid; i < D * (d / 4); i += kUp2Threads) {
      const int row = i / (d / 4), c4 = i % (d / 4);
      const uint32_t dst = sbase + S::hs + (uint32_t)row * S::hs_row + (uint32_t)c4 * 16u;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(Hg + (size_t)i * 4) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  if (PHASE != 2)
    for (int i = tid; i < 4 * 256; i += kUp2Threads) (&X.hist[0][0])[i] = 0;
  // W^T image and zeroed operand tiles
  if (PHASE != 1 && fold) {
    if (PHASE == 2) {
#pragma unroll
      for (int q = 0; q < kblk; ++q) *reinterpret_cast<uint4*>(sm + S::b1 + (tid + q * kUp2Threads) * 16) = pre_w[q];
    } else {
      const uint4* img = wt_image + (size_t)h * kblk * 512;
      for (int i = tid; i < kblk * 512; i += kUp2Threads) *reinterpret_cast<uint4*>(sm + S::b1 + i * 16) = img[i];
    }
    if (PHASE != 2)
      for (int i = tid; i < (32768 + 3 * 16384) / 16; i += kUp2Threads)
        *reinterpret_cast<uint4*>(sm + S::kt + i * 16) = make_uint4(0, 0, 0, 0);
  }
  int nGL = 0, nMove = 0;
  unsigned thr_key = 0;
  if (PHASE != 2) {
  const unsigned key0 = __float_as_uint(scu[cg > 0 ? 0 : lam]);      // any one score: a guess at the leading byte
  bool top_differs = false;
  for (int e = tid; e < nE; e += kUp2Threads) {
    unsigned k;
    if (e < cg) { k = __float_as_uint(scu[e]); X.pos[e] = L.gpos[(size_t)unit * lam + e]; }
    else { k = __float_as_uint(scu[lam + (e - cg)]); X.pos[e] = c.r_pos0 + (e - cg); }
    X.key[e] = k;
    top_differs = top_differs || ((k ^ key0) >> 24) != 0u;
  }
  // ---- 1. radix select of the nF lowest scores (scores are norms >= 0: bit patterns order like unsigned)
  unsigned prefix = 0, mask = 0, need = (unsigned)nF;
  // scores of one unit are of one magnitude: when they all share the leading byte, its pass is skipped
  const int first_pass = __syncthreads_or(top_differs ? 1 : 0) ? 0 : 1;
  if (first_pass == 1) { prefix = key0 & 0xff000000u; mask = 0xff000000u; }
  for (int pass = first_pass; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int e = tid; e < nE; e += kUp2Threads) {
      const unsigned k = X.key[e];
      if ((k & mask) == prefix) atomicAdd(&X.hist[pass][(k >> shift) & 255u], 1u);
    }
    __syncthreads();
    {
      // every warp scans the 256 bins itself (8 per lane): no broadcast through shared memory
      unsigned cnt[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { cnt[i] = X.hist[pass][lane * 8 + i]; tot += cnt[i]; }
      unsigned incl = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      unsigned run = incl - tot;                     // elements in lower bins
      const bool mine = run < need && need <= incl;  // exactly one lane holds the bin of the need-th lowest
      unsigned np = 0, nn = 0;
      if (mine) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < need && need <= run + cnt[i]) { np = prefix | ((unsigned)(lane * 8 + i) << shift); nn = need - run; }
          run += cnt[i];
        }
      }
      const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
      prefix = __shfl_sync(0xffffffffu, np, src);
      need = __shfl_sync(0xffffffffu, nn, src);
    }
    mask |= 255u << shift;
  }
  // prefix = the nF-th lowest score; `need` of the pairs with exactly that score are folded: the youngest.
  // Pairs below the threshold are marked at once; pairs on it are collected into a short list first
  // (normally one entry) and ranked among themselves by position.
  thr_key = prefix;
  for (int e = tid; e < nE; e += kUp2Threads) {
    const unsigned k = X.key[e];
    if (k < thr_key) X.pos[e] |= (int)0x80000000;
    else if (k == thr_key) {
      const int at = atomicAdd(&X.n_equal, 1);
      if (at < kUp2MaxFold) X.equal_e[at] = e;
    } else atomicMin(&X.min_keep, k);
  }
  __syncthreads();
  {
    const int neq = X.n_equal;
    if (neq <= kUp2MaxFold) {
      for (int i = tid; i < neq; i += kUp2Threads) {
        const int e = X.equal_e[i], pe = X.pos[e];
        unsigned younger = 0;
        for (int j = 0; j < neq; ++j) younger += X.pos[X.equal_e[j]] > pe ? 1u : 0u;
        if (younger < need) X.fold_mark[i] = 1; else { X.fold_mark[i] = 0; atomicMin(&X.min_keep, thr_key); }
      }
      __syncthreads();
      for (int i = tid; i < neq; i += kUp2Threads)
        if (X.fold_mark[i]) X.pos[X.equal_e[i]] |= (int)0x80000000;
    } else {
      // many equal scores (degenerate inputs): rank every one of them against all pairs
      for (int e = tid; e < nE; e += kUp2Threads) {
        if (X.key[e] != thr_key) continue;
        const int pe = X.pos[e] & 0x7fffffff;
        unsigned younger = 0;
        for (int j = 0; j < nE; ++j) younger += (X.key[j] == thr_key && (X.pos[j] & 0x7fffffff) > pe) ? 1u : 0u;
        if (younger < need) atomicOr(reinterpret_cast<unsigned*>(&X.pos[e]), 0x80000000u);
        else atomicMin(&X.min_keep, thr_key);
      }
    }
  }
  __syncthreads();
  // ---- 2. ordered compaction: each thread owns a contiguous range of E
  {
    const int per = (nE + kUp2Threads - 1) / kUp2Threads;
    const int e0 = min(nE, tid * per), e1 = min(nE, e0 + per);
    int nf = 0, ng = 0, nm = 0;                      // folded, folded members of G, leaving pairs that stay
    for (int e = e0; e < e1; ++e) {
      const bool fold = X.pos[e] < 0;
      nf += fold ? 1 : 0;
      ng += (fold && e < cg) ? 1 : 0;
      nm += (!fold && e >= cg) ? 1 : 0;
    }
    int inf = nf, ing = ng, inm = nm;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int a = __shfl_up_sync(0xffffffffu, inf, o), bq = __shfl_up_sync(0xffffffffu, ing, o), cq = __shfl_up_sync(0xffffffffu, inm, o);
      if (lane >= o) { inf += a; ing += bq; inm += cq; }
    }
    if (lane == 31) { X.scan[warp][0] = inf; X.scan[warp][1] = ing; X.scan[warp][2] = inm; }
    __syncthreads();
    int bf = 0, bg = 0, bm = 0;
    for (int w = 0; w < warp; ++w) { bf += X.scan[w][0]; bg += X.scan[w][1]; bm += X.scan[w][2]; }
    int of = bf + inf - nf, og = bg + ing - ng, om = bm + inm - nm;
    for (int e = e0; e < e1; ++e) {
      const bool fold = X.pos[e] < 0;
      if (fold) {
        if (of < kUp2MaxFold) X.fold_e[of] = e;
        ++of;
        if (e < cg) { if (og < kUp2MaxFold) X.free_slot[og] = e; ++og; }
      } else if (e >= cg) {
        if (om < kUp2MaxFold) X.mover[om] = e - cg;
        ++om;
      }
    }
  }
  __syncthreads();
  for (int w = 0; w < kUp2Threads / 32; ++w) { nGL += X.scan[w][1]; nMove += X.scan[w][2]; }

  }
  if (PHASE == 1) {
    // the lists leave through the state's work-list arrays
    for (int i = tid; i < nF; i += kUp2Threads) g_fold[i] = X.fold_e[i];
    for (int w = tid; w < nMove; w += kUp2Threads) {
      g_src[w] = X.mover[w];
      g_dst[w] = w < nGL ? X.free_slot[w] : cg + (w - nGL);
    }
    if (tid == 0) {
      g_cnt[0] = nF;
      g_cnt[1] = nMove;
      L.thr[(size_t)unit * 2 + 0] = __uint_as_float(X.min_keep);
      L.thr[(size_t)unit * 2 + 1] = __uint_as_float(thr_key);
    }
    return;
  }
  if (PHASE == 2) {
    nMove = c.mode == UPD_NONE ? 0 : min(pre_cnt, kUp2MaxFold);
    nGL = nMove;                                                     // every destination comes from the list
    if (tid < nF) X.fold_e[tid] = pre_fold;
    if (tid < nMove) { X.mover[tid] = pre_src; X.free_slot[tid] = pre_dst; }
    __syncthreads();
  }
  // ---- leaving pairs that stay: into the freed slots, then into the slots beyond count_g.  Copies go in
  // batches of kCopyBatch 16-byte pieces per thread, all loads of a batch before its stores: one round trip to
  // memory per batch instead of one per piece
  constexpr int kCopyBatch = 8;
  auto do_movers = [&](int t0, int nt) {
    const int total = nMove * nch * 2;
    for (int base = t0; base < total; base += nt * kCopyBatch) {
      uint4 tmp[kCopyBatch];
#pragma unroll
      for (int k = 0; k < kCopyBatch; ++k) {
        const int i = base + k * nt;
        if (i < total) {
          const int w = i / (2 * nch), rem = i % (2 * nch), isv = rem / nch, ch = rem % nch;
          const T *kp, *vp;
          locate_leaving<T>(L, c, unit, b, h, c.r_pos0 + X.mover[w], kp, vp);
          tmp[k] = *reinterpret_cast<const uint4*>((isv ? vp : kp) + ch * 8);
        }
      }
#pragma unroll
      for (int k = 0; k < kCopyBatch; ++k) {
        const int i = base + k * nt;
        if (i < total) {
          const int w = i / (2 * nch), rem = i % (2 * nch), isv = rem / nch, ch = rem % nch;
          const int src = X.mover[w];
          const int dst = w < nGL ? X.free_slot[w] : cg + (w - nGL);
          T* dp = (isv ? (T*)L.gv : (T*)L.gk) + ((size_t)unit * lam + dst) * d;
          *reinterpret_cast<uint4*>(dp + ch * 8) = tmp[k];
          if (rem == 0) {
            L.gpos[(size_t)unit * lam + dst] = c.r_pos0 + src;
            scu[dst] = fold ? scu[lam + src] : CUDART_NAN_F;         // never scored while the cache still has room
          }
        }
      }
    }
  };
  // ---- the window takes the chunk's last eta tokens (after every read of the rows it replaces)
  auto do_roll = [&](int t0, int nt) {
    if (eta <= 0) return;
    const int first = max(0, c.n - eta);
    const int total = (c.n - first) * nch * 2;
    for (int base = t0; base < total; base += nt * kCopyBatch) {
      uint4 tmp[kCopyBatch];
#pragma unroll
      for (int k = 0; k < kCopyBatch; ++k) {
        const int i = base + k * nt;
        if (i < total) {
          const int ci = first + i / (2 * nch), rem = i % (2 * nch), isv = rem / nch, ch = rem % nch;
          const T* sp = (isv ? (const T*)c.v : (const T*)c.k) + (((size_t)b * c.n + ci) * L.Hkv + h) * d;
          tmp[k] = *reinterpret_cast<const uint4*>(sp + ch * 8);
        }
      }
#pragma unroll
      for (int k = 0; k < kCopyBatch; ++k) {
        const int i = base + k * nt;
        if (i < total) {
          const int ci = first + i / (2 * nch), rem = i % (2 * nch), isv = rem / nch, ch = rem % nch;
          const int p = c.n_seen + ci;
          T* dp = (isv ? (T*)L.wv : (T*)L.wk) + ((size_t)unit * eta + (p % eta)) * d;
          *reinterpret_cast<uint4*>(dp + ch * 8) = tmp[k];
        }
      }
    }
  };
  if (fold) {
  // ---- 3. gather the folded pairs into the operand tiles (rows >= nF stay zero)
  for (int i = tid; i < nF * nch * 2; i += kUp2Threads) {
    const int row = i / (2 * nch), rem = i % (2 * nch), isv = rem / nch, ch = rem % nch;
    const int e = X.fold_e[row];
    const T *kp, *vp;
    locate_eligible<T>(L, c, unit, b, h, e, kp, vp);
    const uint4 val = *reinterpret_cast<const uint4*>((isv ? vp : kp) + ch * 8);
    *reinterpret_cast<uint4*>(sm + (isv ? S::vt : S::kt) + (ch >> 3) * 16384 + tc::sw128_off(row, ch & 7)) = val;
    if (isv)                                                         // the value row again, for the low parts of phi
      *reinterpret_cast<uint4*>(sm + S::vt + (ch >> 3) * 16384 + tc::sw128_off(row + 64, ch & 7)) = val;
  }
  if (tid < nF) {                                                    // the column of ones (block kblk, column 0)
    *reinterpret_cast<T*>(sm + S::vt + kblk * 16384 + tc::sw128_off(tid, 0)) = __float2bfloat16_rn(1.0f);
    *reinterpret_cast<T*>(sm + S::vt + kblk * 16384 + tc::sw128_off(tid + 64, 0)) = __float2bfloat16_rn(1.0f);
  }
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = X.tmem_slot;
  const uint32_t tm_u = tmem, tm_d = tmem + 64;
  const int wq = warp & 3, hf = (warp >> 2) & 1;
  const int t = wq * 32 + lane;
  const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
  if (tid == 0) {
#pragma unroll
    for (int ks = 0; ks < d / 16; ++ks)
      tc::mma_bf16_ss(tm_u, tc::make_desc_sw128(sbase + S::kt + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                      tc::make_desc_sw128(sbase + S::b1 + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024),
                      tc::make_idesc_bf16(128, 64, false, false), ks > 0);
    tc::mma_commit(bar);
  }
  // the upper half of the block moves the staying pairs meanwhile (the gather above has read every
  // slot and ring row the fold needs; the movers only read ring rows and write freed or new slots)
  if (tid >= 256) do_movers(tid - 256, kUp2Threads - 256);
  else { ok = tc::mbar_wait(bar, ph) && ok; ph ^= 1; }
  tc::fence_after_sync();
  if (tid < 256) {                                                   // one thread pair per row: half of the feature map each
    uint32_t u[64], hi[32], lo[32];
    tc::tmem_ld64u(tm_u + lane_addr, u);                             // (warp-wide: every lane takes part)
    if (t < 64) {
      tc::phi_half_split(u, hf != 0, L.phi_kind == 1, hi, lo);
      // phi tile over the key tile (consumed): row = folded pair (hi parts) and 64 + folded pair (lo parts),
      // 64 features per 128-byte row and block
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        *reinterpret_cast<uint4*>(sm + S::kt + hf * 16384 + tc::sw128_off(t, ch)) =
            make_uint4(hi[ch * 4], hi[ch * 4 + 1], hi[ch * 4 + 2], hi[ch * 4 + 3]);
        *reinterpret_cast<uint4*>(sm + S::kt + hf * 16384 + tc::sw128_off(t + 64, ch)) =
            make_uint4(lo[ch * 4], lo[ch * 4 + 1], lo[ch * 4 + 2], lo[ch * 4 + 3]);
      }
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  tc::fence_async_smem();
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    // [dH | ds] = phi^T [V | 1]: A = phi tile read MN-major (M = feature), B = value tile MN-major
    // K index = operand row: hi parts of the folded pairs, then (from row 64) their lo parts; rows of no
    // pair hold the feature map of a zero key against a zero value row
#pragma unroll
    for (int ks = 0; ks < 8; ++ks)
      tc::mma_bf16_ss(tm_d, tc::make_desc_sw128(sbase + S::kt + ks * 2048, 16384, 1024),
                      tc::make_desc_sw128(sbase + S::vt + ks * 2048, 16384, 1024),
                      tc::make_idesc_bf16(128, d + 16, true, true), ks > 0);
    tc::mma_commit(bar);
  }
  if (tid >= 256) do_roll(tid - 256, kUp2Threads - 256);             // the movers' reads of the ring ended at the barrier above
  else { ok = tc::mbar_wait(bar, ph) && ok; ph ^= 1; }
  tc::fence_after_sync();
  if (PHASE == 2) {
    if (tid < 256 && ok) {                                           // row j = t, columns [hf * d/2, +d/2)
      // dH from tensor memory into the (padded) rows of the staging area
      constexpr int HC = d / 2;
      float* Hrow = reinterpret_cast<float*>(sm + S::hs + (size_t)t * S::hs_row) + hf * HC;
#pragma unroll
      for (int c0 = 0; c0 < HC; c0 += 32) {
        float p[32];
        tc::tmem_ld32(tm_d + lane_addr + hf * HC + c0, p);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<float4*>(Hrow + c0 + q * 4) = make_float4(p[q * 4], p[q * 4 + 1], p[q * 4 + 2], p[q * 4 + 3]);
      }
      if (hf == 0) {
        float ds[2];
        tc::tmem_ld2(tm_d + lane_addr + d, ds);
        L.s[(size_t)unit * D + t] += ds[0];
      }
    }
    // (the lower half alone: the upper half is still rolling the window)
    if (tid < 256) tc::named_bar_sync(2, 256);
    if (tid < 256 && ok) {
      // H += dH: 16-byte reductions performed at the L2, a warp covers 512 consecutive bytes (nothing is read back)
      float4* Hg4 = reinterpret_cast<float4*>(L.H + (size_t)unit * D * d);
      for (int i = tid; i < D * (d / 4); i += 256) {
        const int row = i / (d / 4), c4 = i % (d / 4);
        atomicAdd(Hg4 + i, *reinterpret_cast<const float4*>(sm + S::hs + (size_t)row * S::hs_row + (size_t)c4 * 16));
      }
    }
  } else {
  if (tid < 256 && ok) {                                             // row j = t, columns [hf * d/2, +d/2)
    // H += dH in the shared-memory copy (this thread owns the half row) and the same values as bf16 in
    // the operand image layout [2 j blocks][d rows c][64 j] (row c, K index j, 128-byte swizzle), staged
    // over the consumed phi tile; both leave through coalesced stores below
    constexpr int HC = d / 2;
    float* Hrow = reinterpret_cast<float*>(sm + S::hs + (size_t)t * S::hs_row) + hf * HC;
    const uint32_t joff = (uint32_t)(t >> 6) * (d * 128) + (uint32_t)(t & 7) * 2;
    const int jch = (t & 63) >> 3;
#pragma unroll
    for (int c0 = 0; c0 < HC; c0 += 32) {
      float p[32];
      tc::tmem_ld32(tm_d + lane_addr + hf * HC + c0, p);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 hv = *reinterpret_cast<const float4*>(Hrow + c0 + q * 4);
        hv.x += p[q * 4]; hv.y += p[q * 4 + 1]; hv.z += p[q * 4 + 2]; hv.w += p[q * 4 + 3];
        *reinterpret_cast<float4*>(Hrow + c0 + q * 4) = hv;
        p[q * 4] = hv.x; p[q * 4 + 1] = hv.y; p[q * 4 + 2] = hv.z; p[q * 4 + 3] = hv.w;
      }
#pragma unroll
      for (int q = 0; q < 32; ++q) {
        const int cc = hf * HC + c0 + q;
        *reinterpret_cast<__nv_bfloat16*>(sm + S::kt + joff + tc::sw128_off(cc, jch)) = __float2bfloat16_rn(p[q]);
      }
    }
    if (hf == 0) {
      float ds[2];
      tc::tmem_ld2(tm_d + lane_addr + d, ds);
      L.s[(size_t)unit * D + t] += ds[0];
    }
  }
  __syncthreads();
  if (ok) {
    float4* Hg4 = reinterpret_cast<float4*>(L.H + (size_t)unit * D * d);
    for (int i = tid; i < D * (d / 4); i += kUp2Threads) {
      const int row = i / (d / 4), c4 = i % (d / 4);
      Hg4[i] = *reinterpret_cast<const float4*>(sm + S::hs + (size_t)row * S::hs_row + (size_t)c4 * 16);
    }
    uint4* img4 = reinterpret_cast<uint4*>(ht_image + (size_t)unit * (2 * d * 64));
    for (int i = tid; i < 2 * d * 128 / 16; i += kUp2Threads) img4[i] = *reinterpret_cast<const uint4*>(sm + S::kt + (size_t)i * 16);
  }
  }  // (PHASE 0: H and its image through shared memory)
  }  // fold
  if (!fold) {
    do_movers(tid, kUp2Threads);
    __syncthreads();                                                 // ring rows are read above before they are replaced
    do_roll(tid, kUp2Threads);
  }
  if (PHASE == 0 && tid == 0 && ok) {
    L.thr[(size_t)unit * 2 + 0] = __uint_as_float(X.min_keep);
    L.thr[(size_t)unit * 2 + 1] = __uint_as_float(thr_key);
  }
  if (!ok && tid == 0) atomicOr(L.status, 32);
  tc::fence_before_sync();
  __syncthreads();
  if (fold && warp == 0) tc::tmem_dealloc(X.tmem_slot, 256);
}

template <int DPL, int PHASE>
__global__ void __launch_bounds__(kUp2Threads, 1) k_update2_tc(Layer L, Call c, const uint4* wt_image, __nv_bfloat16* ht_image) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  extern __shared__ uint8_t smem_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  update2_body<DPL, PHASE>(L, c, wt_image, ht_image, sm, (int)blockIdx.x);
}

}  // namespace lola
