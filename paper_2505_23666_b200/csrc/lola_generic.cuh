// Shape-generic CUDA-core kernels of the LoLA step.  They serve the fp32 mode (whose selection
// must match an fp32/fp64 evaluation bit for bit up to near-ties) and every shape the tensor-core
// kernels are not built for.  All arithmetic is fp32; T is the storage type of q, k, v, out, W and
// of the cached keys and values.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "lola_params.h"

namespace lola {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float x);
template <> __device__ __forceinline__ void stf<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_min(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fminf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float round_bf16f(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Row pointers of a softmax key the queries of this call can see (Eq. 14): sparse-cache slot,
// window ring entry, or incoming pair.
template <typename T>
__device__ __forceinline__ void locate_att_key(const Layer& L, const Call& c, int unit, int b, int h, int idx,
                                               const T*& kp, const T*& vp) {
  const int d = L.d;
  if (idx < c.att_g) {
    size_t o = ((size_t)unit * L.lam + idx) * d;
    kp = (const T*)L.gk + o; vp = (const T*)L.gv + o;
  } else if (idx < c.att_g + c.att_wn) {
    int p = c.att_w0 + (idx - c.att_g);
    size_t o = ((size_t)unit * L.eta + (p % L.eta)) * d;
    kp = (const T*)L.wk + o; vp = (const T*)L.wv + o;
  } else {
    int ci = idx - c.att_g - c.att_wn;
    size_t o = (((size_t)b * c.n + ci) * L.Hkv + h) * d;
    kp = (const T*)c.k + o; vp = (const T*)c.v + o;
  }
}

// Row pointers of the pair at token position p that is leaving the window in this call: it sits in
// the ring if it arrived in an earlier call, otherwise it is one of the incoming pairs.
template <typename T>
__device__ __forceinline__ void locate_leaving(const Layer& L, const Call& c, int unit, int b, int h, int p,
                                               const T*& kp, const T*& vp) {
  const int d = L.d;
  if (p < c.n_seen) {
    size_t o = ((size_t)unit * L.eta + (p % L.eta)) * d;
    kp = (const T*)L.wk + o; vp = (const T*)L.wv + o;
  } else {
    size_t o = (((size_t)b * c.n + (p - c.n_seen)) * L.Hkv + h) * d;
    kp = (const T*)c.k + o; vp = (const T*)c.v + o;
  }
}

// Member e of the eligible set E = G ++ leaving pairs (Eq. 11 / 15).
template <typename T>
__device__ __forceinline__ void locate_eligible(const Layer& L, const Call& c, int unit, int b, int h, int e,
                                                const T*& kp, const T*& vp) {
  if (e < c.count_g) {
    size_t o = ((size_t)unit * L.lam + e) * L.d;
    kp = (const T*)L.gk + o; vp = (const T*)L.gv + o;
  } else {
    locate_leaving<T>(L, c, unit, b, h, c.r_pos0 + (e - c.count_g), kp, vp);
  }
}

// Feature map of one row x[d] (shared memory, fp32) computed by one warp into f[2F] (shared).
// u = x W; softmax kind: [softmax(u), softmax(-u)]; exp kind (Eq. 6): [exp(u), exp(-u)].
template <typename T>
__device__ __forceinline__ void warp_phi(const float* x, const T* W, int d, int F, int kind, bool round_out,
                                         float* f, int lane) {
  float u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int ff = lane + 32 * i;
    float a = 0.f;
    if (ff < F) {
      for (int j = 0; j < d; ++j) a = fmaf(x[j], ldf<T>(W + (size_t)j * F + ff), a);
    }
    u[i] = a;
  }
  if (kind == 1) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int ff = lane + 32 * i;
      if (ff < F) {
        float a = expf(u[i]), b = expf(-u[i]);
        f[ff] = round_out ? round_bf16f(a) : a;
        f[F + ff] = round_out ? round_bf16f(b) : b;
      }
    }
  } else {
    float mx = -CUDART_INF_F, mn = CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (lane + 32 * i < F) { mx = fmaxf(mx, u[i]); mn = fminf(mn, u[i]); }
    mx = warp_max(mx);
    mn = warp_min(mn);
    float e1[4], e2[4], s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      bool ok = lane + 32 * i < F;
      e1[i] = ok ? expf(u[i] - mx) : 0.f;
      e2[i] = ok ? expf(mn - u[i]) : 0.f;
      s1 += e1[i];
      s2 += e2[i];
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int ff = lane + 32 * i;
      if (ff < F) {
        float a = e1[i] / s1, b = e2[i] / s2;
        f[ff] = round_out ? round_bf16f(a) : a;
        f[F + ff] = round_out ? round_bf16f(b) : b;
      }
    }
  }
  __syncwarp();
}

constexpr int kHB = 64;  // rows of H staged in shared memory at a time

// CTA-wide: lin[r][t] += sum_j f[r][j] * H[unit][j][lane + 32 t] for the RPW rows of each warp.
template <int DPL, int RPW>
__device__ __forceinline__ void cta_lin_accumulate(const Layer& L, int unit, const float* fbase /*[rows][D]*/,
                                                   int warp, int lane, float* Hs, bool round_h,
                                                   float (&lin)[RPW][DPL]) {
  constexpr int d = DPL * 32;
  const int D = L.D;
  const float* Hu = L.H + (size_t)unit * D * d;
  for (int j0 = 0; j0 < D; j0 += kHB) {
    int nr = min(kHB, D - j0);
    __syncthreads();
    for (int i = threadIdx.x; i < nr * d; i += blockDim.x) {
      float hv = Hu[(size_t)j0 * d + i];
      Hs[i] = round_h ? round_bf16f(hv) : hv;
    }
    __syncthreads();
    for (int j = 0; j < nr; ++j) {
      float hrow[DPL];
#pragma unroll
      for (int t = 0; t < DPL; ++t) hrow[t] = Hs[j * d + lane + 32 * t];
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        float pj = fbase[(size_t)(warp * RPW + r) * D + j0 + j];
#pragma unroll
        for (int t = 0; t < DPL; ++t) lin[r][t] = fmaf(pj, hrow[t], lin[r][t]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Eq. 14: softmax over sparse cache + window + causal chunk, linear term in the same denominator.
// grid (ceil(g*nq/16), units), 256 threads; each warp owns two query rows.
constexpr int kAttRows = 16;
constexpr int kAttKT = 32;

template <int DPL>
__host__ __device__ constexpr size_t attend_smem_floats(int D) {
  return (size_t)kAttRows * DPL * 32 + (size_t)kAttRows * D + 8 * 2 * 32 + (size_t)kAttKT * (DPL * 32 + 1) +
         (size_t)kAttKT * DPL * 32;
}

template <typename T, int DPL>
__global__ void __launch_bounds__(256) k_attend(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  constexpr int d = DPL * 32;
  extern __shared__ float sm[];
  float* qs = sm;                                   // [16][d]
  float* phis = qs + kAttRows * d;                  // [16][D]
  float* ps = phis + kAttRows * L.D;                // [8][2][32]
  float* Ks = ps + 8 * 2 * 32;                      // [32][d+1]; later reused to stage H
  float* Vs = Ks + kAttKT * (d + 1);                // [32][d]
  const int unit = blockIdx.y, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nrows = L.g * c.nq;
  const int row0 = blockIdx.x * kAttRows;

  for (int i = tid; i < kAttRows * d; i += 256) {
    int rr = i / d, j = i % d, row = row0 + rr;
    float x = 0.f;
    if (row < nrows) {
      int hl = row / c.nq, r = row % c.nq;
      x = ldf<T>((const T*)c.q + (((size_t)b * c.nq + r) * L.Hq + h * L.g + hl) * d + j);
    }
    qs[i] = x;
  }
  __syncthreads();

  const int NK = c.att_g + c.att_wn + c.att_chunk;
  const int chunk0 = c.att_g + c.att_wn;
  int rtok[2];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) rtok[rr] = (row0 + warp * 2 + rr) % c.nq;
  float m[2] = {0.f, 0.f}, l[2] = {0.f, 0.f};       // m starts at 0: stabiliser max(0, max z)
  float acc[2][DPL];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr)
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[rr][t] = 0.f;
  const float* q0 = qs + (warp * 2) * d;
  const float* q1 = q0 + d;

  for (int kt = 0; kt < NK; kt += kAttKT) {
    __syncthreads();
    for (int kk = warp; kk < kAttKT; kk += 8) {
      int idx = kt + kk;
      if (idx < NK) {
        const T *kp, *vp;
        locate_att_key<T>(L, c, unit, b, h, idx, kp, vp);
        for (int j = lane; j < d; j += 32) {
          Ks[kk * (d + 1) + j] = ldf<T>(kp + j);
          Vs[kk * d + j] = ldf<T>(vp + j);
        }
      } else {
        for (int j = lane; j < d; j += 32) { Ks[kk * (d + 1) + j] = 0.f; Vs[kk * d + j] = 0.f; }
      }
    }
    __syncthreads();
    const int idx = kt + lane;
    const float* kr = Ks + lane * (d + 1);
    float z[2] = {0.f, 0.f};
#pragma unroll 8
    for (int j = 0; j < d; ++j) {
      float kv = kr[j];
      z[0] = fmaf(q0[j], kv, z[0]);
      z[1] = fmaf(q1[j], kv, z[1]);
    }
    const int ci = idx - chunk0;
#pragma unroll
    for (int rr = 0; rr < 2; ++rr) {
      bool valid = (idx < NK) && (ci < 0 || ci <= rtok[rr]);
      float zz = valid ? z[rr] * L.scale : -CUDART_INF_F;
      float mnew = fmaxf(m[rr], warp_max(zz));
      float p = valid ? expf(zz - mnew) : 0.f;
      float alpha = expf(m[rr] - mnew);
      l[rr] = l[rr] * alpha + warp_sum(p);
      m[rr] = mnew;
      ps[(warp * 2 + rr) * 32 + lane] = p;
#pragma unroll
      for (int t = 0; t < DPL; ++t) acc[rr][t] *= alpha;
    }
    __syncwarp();
    for (int i = 0; i < kAttKT; ++i) {
      float p0 = ps[(warp * 2) * 32 + i], p1 = ps[(warp * 2 + 1) * 32 + i];
#pragma unroll
      for (int t = 0; t < DPL; ++t) {
        float vv = Vs[i * d + lane + 32 * t];
        acc[0][t] = fmaf(p0, vv, acc[0][t]);
        acc[1][t] = fmaf(p1, vv, acc[1][t]);
      }
    }
  }

  // linear term: phi(q)^T H and phi(q)^T s with the H, s the call started with
  const T* Wh = (const T*)L.W + (size_t)h * d * L.F;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) warp_phi<T>(qs + (warp * 2 + rr) * d, Wh, d, L.F, L.phi_kind, false,
                                             phis + (warp * 2 + rr) * L.D, lane);
  float lden[2];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    float a = 0.f;
    for (int j = lane; j < L.D; j += 32) a = fmaf(phis[(warp * 2 + rr) * L.D + j], L.s[(size_t)unit * L.D + j], a);
    lden[rr] = warp_sum(a);
  }
  float lin[2][DPL];
#pragma unroll
  for (int rr = 0; rr < 2; ++rr)
#pragma unroll
    for (int t = 0; t < DPL; ++t) lin[rr][t] = 0.f;
  cta_lin_accumulate<DPL, 2>(L, unit, phis, warp, lane, Ks, false, lin);

#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    int row = row0 + warp * 2 + rr;
    if (row < nrows) {
      int hl = row / c.nq, r = row % c.nq;
      float e = (c.att_flags & 1) ? 0.f : expf(-m[rr]);      // (0: the queries do not see H, s)
      float den = fmaf(e, lden[rr], l[rr]);
      T* op = (T*)c.out + (((size_t)b * c.nq + r) * L.Hq + h * L.g + hl) * d;
#pragma unroll
      for (int t = 0; t < DPL; ++t) stf<T>(op + lane + 32 * t, fmaf(e, lin[rr][t], acc[rr][t]) / den);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Eq. 10 for every member of E = G ++ leaving pairs, against the H, s before the fold.
// grid (ceil(|E|/32), units), 256 threads; each warp owns four rows.
constexpr int kScoreRows = 32;

template <int DPL>
__host__ __device__ constexpr size_t score_smem_floats(int D) {
  return (size_t)kScoreRows * DPL * 32 + (size_t)kScoreRows * D + (size_t)kHB * DPL * 32;
}

template <typename T, int DPL>
__global__ void __launch_bounds__(256) k_score(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  constexpr int d = DPL * 32;
  constexpr int RPW = 4;
  extern __shared__ float sm[];
  float* xs = sm;                                   // [32][d]
  float* phis = xs + kScoreRows * d;                // [32][D]
  float* Hs = phis + kScoreRows * L.D;              // [64][d]
  const int unit = blockIdx.y, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nE = c.count_g + c.r;
  const int e0 = blockIdx.x * kScoreRows + warp * RPW;
  const bool rq = L.bf16 != 0;
  const T* Wh = (const T*)L.W + (size_t)h * d * L.F;
  const T* vrow[RPW];
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    int e = e0 + rr;
    const T *kp = nullptr, *vp = nullptr;
    if (e < nE) locate_eligible<T>(L, c, unit, b, h, e, kp, vp);
    vrow[rr] = vp;
    for (int j = lane; j < d; j += 32) xs[(warp * RPW + rr) * d + j] = (e < nE) ? ldf<T>(kp + j) : 0.f;
  }
  __syncwarp();
  float den[RPW];
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    float* f = phis + (size_t)(warp * RPW + rr) * L.D;
    warp_phi<T>(xs + (warp * RPW + rr) * d, Wh, d, L.F, L.phi_kind, rq, f, lane);
    float a = 0.f;
    for (int j = lane; j < L.D; j += 32) a = fmaf(f[j], L.s[(size_t)unit * L.D + j], a);
    den[rr] = warp_sum(a);
  }
  float lin[RPW][DPL];
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr)
#pragma unroll
    for (int t = 0; t < DPL; ++t) lin[rr][t] = 0.f;
  cta_lin_accumulate<DPL, RPW>(L, unit, phis, warp, lane, Hs, rq, lin);
#pragma unroll
  for (int rr = 0; rr < RPW; ++rr) {
    int e = e0 + rr;
    if (e >= nE) continue;                          // warp-uniform
    float ss = 0.f;
#pragma unroll
    for (int t = 0; t < DPL; ++t) {
      float vh = den[rr] > 0.f ? lin[rr][t] / den[rr] : 0.f;
      float df = vh - ldf<T>(vrow[rr] + lane + 32 * t);
      ss = fmaf(df, df, ss);
    }
    ss = warp_sum(ss);
    if (lane == 0) {
      size_t o = (size_t)unit * (L.lam + L.cmax) + (e < c.count_g ? e : L.lam + (e - c.count_g));
      L.score[o] = sqrtf(ss);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Eq. 12: exact top-lambda of E by (score descending, position ascending); emits the work lists
// the update kernel consumes.  One CTA per unit.
__device__ __forceinline__ bool better(float sa, int pa, float sb, int pb) {
  return sa > sb || (sa == sb && pa < pb);
}

__global__ void __launch_bounds__(256) k_select(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  extern __shared__ float sm[];
  const int unit = blockIdx.x, tid = threadIdx.x;
  const int nE = c.count_g + c.r;
  int* fold_idx = L.fold_idx + (size_t)unit * L.cmax;
  int* move_src = L.move_src + (size_t)unit * L.cmax;
  int* move_dst = L.move_dst + (size_t)unit * L.cmax;
  int* counts = L.counts + (size_t)unit * 4;
  if (c.mode == UPD_APPEND) {
    for (int i = tid; i < c.r; i += blockDim.x) { move_src[i] = i; move_dst[i] = c.count_g + i; }
    if (tid == 0) { counts[0] = 0; counts[1] = c.r; }
    return;
  }
  if (c.mode == UPD_FOLD_ALL) {
    for (int i = tid; i < c.r; i += blockDim.x) fold_idx[i] = c.count_g + i;
    if (tid == 0) { counts[0] = c.r; counts[1] = 0; }
    return;
  }
  float* sc = sm;                                   // [nE]
  int* pos = (int*)(sc + nE);                       // [nE]
  int* free_slot = pos + nE;                        // [cmax]
  unsigned char* keep = (unsigned char*)(free_slot + L.cmax);   // [nE]
  __shared__ unsigned int s_min_keep, s_max_lose;
  __shared__ int s_nglose;
  const float* scu = L.score + (size_t)unit * (L.lam + L.cmax);
  for (int e = tid; e < nE; e += blockDim.x) {
    if (e < c.count_g) { sc[e] = scu[e]; pos[e] = L.gpos[(size_t)unit * L.lam + e]; }
    else { sc[e] = scu[L.lam + (e - c.count_g)]; pos[e] = c.r_pos0 + (e - c.count_g); }
  }
  if (tid == 0) { s_min_keep = 0x7f800000u; s_max_lose = 0u; s_nglose = 0; }
  __syncthreads();
  for (int e = tid; e < nE; e += blockDim.x) {
    float se = sc[e];
    int pe = pos[e], rank = 0;
    for (int j = 0; j < nE; ++j) rank += better(sc[j], pos[j], se, pe) ? 1 : 0;
    bool kp = rank < L.lam;
    keep[e] = kp ? 1 : 0;
    // scores are norms (>= 0): their bit patterns order like unsigned integers
    if (kp) atomicMin(&s_min_keep, __float_as_uint(se)); else atomicMax(&s_max_lose, __float_as_uint(se));
    if (!kp && e < c.count_g) atomicAdd(&s_nglose, 1);
  }
  __syncthreads();
  const int nglose = s_nglose;
  for (int e = tid; e < nE; e += blockDim.x) {
    if (!keep[e]) {
      int idx = 0;
      for (int j = 0; j < e; ++j) idx += keep[j] ? 0 : 1;
      if (idx < L.cmax) fold_idx[idx] = e;
      if (e < c.count_g && idx < L.cmax) free_slot[idx] = e;
    }
  }
  __syncthreads();
  for (int e = c.count_g + tid; e < nE; e += blockDim.x) {
    if (keep[e]) {
      int w = 0;
      for (int j = c.count_g; j < e; ++j) w += keep[j] ? 1 : 0;
      if (w < L.cmax) {
        move_src[w] = e - c.count_g;
        move_dst[w] = (w < nglose) ? free_slot[w] : c.count_g + (w - nglose);
      }
    }
  }
  if (tid == 0) {
    int nfold = nE - L.lam;
    int nmove = L.lam - (c.count_g - nglose);
    counts[0] = nfold;
    counts[1] = nmove;
    L.thr[(size_t)unit * 2 + 0] = __uint_as_float(s_min_keep);
    L.thr[(size_t)unit * 2 + 1] = __uint_as_float(s_max_lose);
    if (nfold > L.cmax || nmove > L.cmax || nmove < 0) atomicOr(L.status, 1);
  }
}

// ---------------------------------------------------------------------------------------------
// Eq. 13 fold, then the moves into the sparse cache, then the window takes the incoming pairs.
// One CTA of 512 threads per unit.  Everything that is folded or moved is read before any slot or
// ring entry is overwritten.
constexpr int kUpdThreads = 512;
constexpr int kUpdFB = 16;   // pairs folded per pass (one per warp)
constexpr int kUpdEPT = 64;  // H entries per thread: D * d <= 512 * 64

template <int DPL>
__host__ __device__ constexpr size_t update_smem_floats(int D) {
  return (size_t)kUpdFB * DPL * 32 * 2 + (size_t)kUpdFB * D;
}

template <typename T>
__device__ __forceinline__ void copy_row(T* dst, const T* src, int d, int lane) {
  for (int j = lane; j < d; j += 32) dst[j] = src[j];
}

template <typename T, int DPL>
__global__ void __launch_bounds__(kUpdThreads) k_update(Layer L, Call c) {
  if (state_failed(L)) return;                        // an earlier kernel failed: do nothing
  constexpr int d = DPL * 32;
  extern __shared__ float sm[];
  float* xs = sm;                                   // [16][d]
  float* vs = xs + kUpdFB * d;                      // [16][d]
  float* phis = vs + kUpdFB * d;                    // [16][D]
  const int unit = blockIdx.x, b = unit / L.Hkv, h = unit % L.Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int D = L.D;
  const bool rq = L.bf16 != 0;
  const bool has_lists = c.mode != UPD_NONE;
  const int nf = has_lists ? min(L.counts[(size_t)unit * 4 + 0], L.cmax) : 0;
  const int nm = has_lists ? min(L.counts[(size_t)unit * 4 + 1], L.cmax) : 0;
  const T* Wh = (const T*)L.W + (size_t)h * d * L.F;

  if (nf > 0) {
    float hacc[kUpdEPT];
#pragma unroll
    for (int i = 0; i < kUpdEPT; ++i) hacc[i] = 0.f;
    float sacc = 0.f;
    for (int f0 = 0; f0 < nf; f0 += kUpdFB) {
      __syncthreads();
      int li = f0 + warp;
      if (li < nf) {
        int e = L.fold_idx[(size_t)unit * L.cmax + li];
        const T *kp, *vp;
        locate_eligible<T>(L, c, unit, b, h, e, kp, vp);
        for (int j = lane; j < d; j += 32) { xs[warp * d + j] = ldf<T>(kp + j); vs[warp * d + j] = ldf<T>(vp + j); }
        __syncwarp();
        warp_phi<T>(xs + warp * d, Wh, d, L.F, L.phi_kind, false, phis + (size_t)warp * D, lane);   // Eq. 13 folds phi(k) itself
      }
      __syncthreads();
      const int nb = min(kUpdFB, nf - f0);
#pragma unroll
      for (int i = 0; i < kUpdEPT; ++i) {
        int idx = tid + i * kUpdThreads;
        if (idx < D * d) {
          int j = idx / d, cc = idx % d;
          float a = hacc[i];
          for (int q = 0; q < nb; ++q) a = fmaf(phis[(size_t)q * D + j], vs[q * d + cc], a);
          hacc[i] = a;
        }
      }
      if (tid < D)
        for (int q = 0; q < nb; ++q) sacc += phis[(size_t)q * D + tid];
    }
    float* Hu = L.H + (size_t)unit * D * d;
#pragma unroll
    for (int i = 0; i < kUpdEPT; ++i) {
      int idx = tid + i * kUpdThreads;
      if (idx < D * d) Hu[idx] += hacc[i];
    }
    if (tid < D) L.s[(size_t)unit * D + tid] += sacc;
  }
  __syncthreads();

  // leaving pairs that stay: into the slots of the sparse-cache members that were folded, then free slots
  float* scu = L.score + (size_t)unit * (L.lam + L.cmax);
  for (int mi = warp; mi < nm; mi += kUpdThreads / 32) {
    int src = L.move_src[(size_t)unit * L.cmax + mi], dst = L.move_dst[(size_t)unit * L.cmax + mi];
    int p = c.r_pos0 + src;
    const T *kp, *vp;
    locate_leaving<T>(L, c, unit, b, h, p, kp, vp);
    size_t o = ((size_t)unit * L.lam + dst) * d;
    copy_row<T>((T*)L.gk + o, kp, d, lane);
    copy_row<T>((T*)L.gv + o, vp, d, lane);
    if (lane == 0) {
      L.gpos[(size_t)unit * L.lam + dst] = p;
      scu[dst] = (c.mode == UPD_SELECT) ? scu[L.lam + src] : CUDART_NAN_F;
    }
  }
  __syncthreads();

  // the window keeps the last eta positions: the newest min(eta, n) incoming pairs enter the ring
  if (L.eta > 0) {
    int first = max(0, c.n - L.eta);
    for (int ci = first + warp; ci < c.n; ci += kUpdThreads / 32) {
      int p = c.n_seen + ci;
      size_t src = (((size_t)b * c.n + ci) * L.Hkv + h) * d;
      size_t dst = ((size_t)unit * L.eta + (p % L.eta)) * d;
      copy_row<T>((T*)L.wk + dst, (const T*)c.k + src, d, lane);
      copy_row<T>((T*)L.wv + dst, (const T*)c.v + src, d, lane);
    }
  }
}

}  // namespace lola
