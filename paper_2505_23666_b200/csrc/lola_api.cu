// Host side of the C ABI declared in include/lola.h: argument checks, the carve-up of the caller's
// state buffer, the per-call geometry (every count is a function of the tokens seen so far, so no
// device value is ever read back to decide a launch), and the launches themselves.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/lola.h"
#include "lola_generic.cuh"
#include "lola_params.h"
#include "lola_score_tc.cuh"
#include "lola_attend_tc.cuh"
#include "lola_decode_tc.cuh"
#include "lola_decode2_tc.cuh"
#include "lola_score2_tc.cuh"
#include "lola_update2_tc.cuh"
#include "lola_attend2_tc.cuh"

using namespace lola;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct StateLayout {
  size_t status, H, s, gk, gv, gpos, score, wk, wv, fold_idx, move_src, move_dst, counts, thr, wt, total;
};

bool config_ok(const lola_config* c) {
  if (!c) return false;
  if (c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->feat_half < 1 || c->feat_half > 128) return false;
  if (c->window < 0 || c->sparse < 0 || c->max_chunk < 1) return false;
  if ((int64_t)c->sparse + c->max_chunk > 16384) return false;
  if (c->dtype != LOLA_F32 && c->dtype != LOLA_BF16) return false;
  if (c->phi_kind != LOLA_PHI_SOFTMAX && c->phi_kind != LOLA_PHI_EXP) return false;
  if (!(c->softmax_scale >= 0.f) || (c->flags & ~(uint32_t)LOLA_FLAGS_ALL) != 0) return false;
  if ((int64_t)2 * c->feat_half * c->head_dim > (int64_t)kUpdThreads * kUpdEPT) return false;
  return true;
}

StateLayout make_layout(const lola_config& c) {
  const size_t U = (size_t)c.batch * c.n_kv_heads, d = c.head_dim, D = 2 * (size_t)c.feat_half;
  const size_t es = c.dtype == LOLA_BF16 ? 2 : 4;
  const size_t lam = c.sparse, eta = c.window, cm = c.max_chunk;
  StateLayout l{};
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
  l.status = take(256);
  l.H = take(U * D * d * 4);
  l.s = take(U * D * 4);
  l.gk = take(U * lam * d * es);
  l.gv = take(U * lam * d * es);
  l.gpos = take(U * lam * 4);
  l.score = take(U * (lam + cm) * 4);
  l.wk = take(U * eta * d * es);
  l.wv = take(U * eta * d * es);
  l.fold_idx = take(U * cm * 4);
  l.move_src = take(U * cm * 4);
  l.move_dst = take(U * cm * 4);
  l.counts = take(U * 4 * 4);
  l.thr = take(U * 2 * 4);
  // W^T of every KV head in tensor-core operand layout (bf16 layers with F = 64 only)
  l.wt = take(c.dtype == LOLA_BF16 && c.feat_half == 64 ? (size_t)c.n_kv_heads * d * 64 * 2 : 0);
  l.total = o;
  return l;
}

inline bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

struct Geometry {
  int cw, r, r_pos0, count_g, mode, new_count_g;
};

// Counts before/after consuming n tokens when n_seen tokens have been consumed already.
Geometry plan(const lola_config& c, int64_t n_seen, int n) {
  Geometry g{};
  g.cw = (int)std::min<int64_t>(c.window, n_seen);
  g.r = std::max(0, g.cw + n - c.window);
  g.r_pos0 = (int)(n_seen - g.cw);
  g.count_g = (int)std::min<int64_t>(c.sparse, n_seen - g.cw);
  const int nE = g.count_g + g.r;
  if (g.r == 0) g.mode = UPD_NONE;
  else if (c.sparse == 0) g.mode = UPD_FOLD_ALL;
  else if (nE <= c.sparse) g.mode = UPD_APPEND;
  else g.mode = UPD_SELECT;
  g.new_count_g = std::min(c.sparse, nE);
  return g;
}

template <typename T, int DPL>
int set_smem_attrs(int D) {
  cudaError_t e;
  e = cudaFuncSetAttribute(k_attend<T, DPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(attend_smem_floats<DPL>(D) * 4));
  if (e != cudaSuccess) return LOLA_ERR_CUDA;
  e = cudaFuncSetAttribute(k_score<T, DPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(score_smem_floats<DPL>(D) * 4));
  if (e != cudaSuccess) return LOLA_ERR_CUDA;
  e = cudaFuncSetAttribute(k_update<T, DPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(update_smem_floats<DPL>(D) * 4));
  if (e != cudaSuccess) return LOLA_ERR_CUDA;
  return LOLA_OK;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// bf16 tensor [units][rows][d] viewed as rank 3 (d innermost); boxes of 64 columns x box_rows rows of
// one unit, written to shared memory with the 128-byte swizzle the MMA descriptors expect.
bool make_rows_map(CUtensorMap* tm, void* base, size_t units, size_t rows, size_t d, unsigned box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn || rows == 0) return false;
  cuuint64_t dims[3] = {d, rows, units};
  cuuint64_t strides[2] = {d * 2, rows * d * 2};
  cuuint32_t box[3] = {64, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 tensor [B][n][heads][d] of one call viewed as rank 4 (d, head, token, batch row); boxes of 64
// columns x 1 head x 64 tokens, 128-byte swizzle.  Tokens beyond n read as zeros.
bool make_tokens_map(CUtensorMap* tm, const void* base, size_t B, size_t n, size_t heads, size_t d) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {d, heads, n, B};
  cuuint64_t strides[3] = {d * 2, heads * d * 2, n * heads * d * 2};
  cuuint32_t box[4] = {64, 1, 64, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct ProfRecord { int kind; cudaEvent_t a, b; };

struct lola_state {
  lola_config cfg;
  Layer L;
  StateLayout lay;
  char* base;
  int64_t n_seen;
  int64_t launches;
  bool tensor_path = false;            // bf16, F = 64: tcgen05 kernels
  bool fused_decode = false;           // shapes the one-kernel generation step is built for
  int sm_count = 0;                    // SMs of the device (grid of the persistent generation kernel)
  bool have_maps = false;              // TMA descriptors of the sparse cache and the window ring exist
  // lola_prefill_host: two copy streams and the events that order them against the kernels (made at first use)
  cudaStream_t cp_in = nullptr, cp_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  bool force_chain = false;            // set while lola_decode_step_static runs: kernel chain with work lists
  CUtensorMap tm_gk, tm_gv, tm_wk, tm_wv;
  lola_call_info info = {};            // what the last prefill / decode call enqueued
  bool profiling = false;
  std::vector<ProfRecord> records;     // events in use since the last lola_profile_read
  std::vector<ProfRecord> pool;        // events ready for reuse
};

namespace {

// Brackets one launch with a pair of events when profiling is on (kind = LOLA_KERNEL_*).
struct LaunchScope {
  lola_state* st; cudaStream_t s; ProfRecord rec; bool on;
  LaunchScope(lola_state* st_, int kind, cudaStream_t s_, uint32_t path = 0, int ctas = 0) : st(st_), s(s_), on(st_->profiling) {
    st->launches++;
    st->info.paths |= path;
    st->info.launches++;
    if (kind >= 0 && kind < LOLA_N_KERNEL_KINDS) st->info.ctas[kind] += ctas;
    if (!on) return;
    if (!st->pool.empty()) { rec = st->pool.back(); st->pool.pop_back(); }
    else if (cudaEventCreate(&rec.a) != cudaSuccess || cudaEventCreate(&rec.b) != cudaSuccess) { on = false; return; }
    rec.kind = kind;
    cudaEventRecord(rec.a, s);
  }
  ~LaunchScope() {
    if (!on) return;
    cudaEventRecord(rec.b, s);
    st->records.push_back(rec);
  }
};

// Launch with programmatic stream serialization: the kernel may become resident while the kernel before it
// in the stream still runs, and waits inside (griddepcontrol.wait) before it touches memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// before_scoring: the kernel after this one in the stream is the scoring kernel of the same call, which only
// reads the memories and runs beside this one: it is let go once this kernel has seen everything before it
// complete, and it waits for this kernel at its end (so that whatever follows sees both complete).
template <typename T, int DPL>
int launch_attend(lola_state* st, const Call& c, cudaStream_t s, bool before_scoring = false) {
  const Layer& L = st->L;
  dim3 grid((L.g * c.nq + kAttRows - 1) / kAttRows, L.B * L.Hkv);
  if (st->have_maps && !st->force_chain && c.att_chunk == c.nq && c.nq <= 64 && c.n == c.nq) {
    // prefill chunk: TMA-fed, warp-specialised kernel; the call's q, k, v get their own descriptors
    CUtensorMap tq, tk, tv, tout;
    if (make_tokens_map(&tq, c.q, L.B, c.nq, L.Hq, L.d) && make_tokens_map(&tk, c.k, L.B, c.n, L.Hkv, L.d) &&
        make_tokens_map(&tv, c.v, L.B, c.n, L.Hkv, L.d) && make_tokens_map(&tout, c.out, L.B, c.nq, L.Hq, L.d)) {
      dim3 grid2(((L.g + 1) / 2 + 1) / 2, L.B * L.Hkv);
      LaunchScope scope(st, LOLA_KERNEL_ATTEND, s, LOLA_PATH_ATTEND_TMA, (int)(grid2.x * grid2.y));
      const cudaError_t le = launch_pdl(k_attend2_tc<DPL>, grid2, dim3(kAt2Threads), Attend2Smem<DPL>::bytes, s, L, c, st->tm_gk, st->tm_gv,
                                        st->tm_wk, st->tm_wv, tq, tk, tv, tout, (const uint4*)(st->base + st->lay.wt),
                                        before_scoring ? 1 : 0);
      return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
    }
  }
  if (st->tensor_path && L.g * c.nq >= 64) {
    dim3 tgrid((L.g * c.nq + kAtM - 1) / kAtM, L.B * L.Hkv);
    LaunchScope scope(st, LOLA_KERNEL_ATTEND, s, LOLA_PATH_ATTEND_MMA, (int)(tgrid.x * tgrid.y));
    k_attend_tc<DPL><<<tgrid, 128, AttendTcSmem<DPL>::bytes, s>>>(L, c);
  } else {
    LaunchScope scope(st, LOLA_KERNEL_ATTEND, s, LOLA_PATH_ATTEND_GENERIC, (int)(grid.x * grid.y));
    k_attend<T, DPL><<<grid, 256, attend_smem_floats<DPL>(L.D) * 4, s>>>(L, c);
  }
  return cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

inline bool fast_update_path(const lola_state* st, const Call& c) {
  return c.mode == UPD_SELECT && st->have_maps && !st->force_chain && c.count_g % 64 == 0 &&
         c.r_pos0 + c.r <= c.n_seen && c.count_g + c.r <= kUp2MaxE && c.r <= kUp2MaxFold;
}

// Eq. 10 scoring and the top-lambda selection on TMA-fed tensor-core kernels.  Both only read the
// memories (scores, positions) and write scores / work lists, so they may run beside the attention
// kernel (busy_sms > 0: that kernel precedes this one in the stream and this one is its programmatic dependent).
template <int DPL>
int launch_score_select(lola_state* st, const Call& c, cudaStream_t ss, int busy_sms = 0) {
  const Layer& L = st->L;
  const int U = L.B * L.Hkv;
  const int NT = (c.count_g / 64 + (L.eta + 63) / 64 + 1) / 2;
  int tpc = (U * NT + 147) / 148;
  tpc = std::max(2, tpc + (tpc & 1));
  // beside the attention kernel (one block per SM, busy_sms of them) the blocks of this kernel should fit
  // the SMs that are left in one round: a second round would end after the attention kernel does
  if (busy_sms > 0 && busy_sms < 148) {
    const int avail = 148 - busy_sms;
    int t2 = tpc;
    while (t2 < NT && U * ((NT + t2 - 1) / t2) > avail) ++t2;
    if (U * ((NT + t2 - 1) / t2) <= avail) tpc = t2;
  }
  const uint4* img = (const uint4*)(st->base + st->lay.wt);
  // the selection (Eq. 12) runs in the scoring kernel: the last block of a unit to finish does it
  dim3 grid((NT + tpc - 1) / tpc, U);
  LaunchScope scope(st, LOLA_KERNEL_SCORE, ss, LOLA_PATH_SCORE_TMA, (int)(grid.x * grid.y));
  const cudaError_t le = launch_pdl(k_score2_tc<DPL>, grid, dim3(kSc2Threads), Score2Smem<DPL>::bytes, ss, L, c, st->tm_gk, st->tm_gv, st->tm_wk,
                                    st->tm_wv, img, tpc, busy_sms > 0 ? 1 : 0);
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

// Eq. 13 fold (added to H in memory), moves into the sparse cache and window roll from the selection's work lists.
template <int DPL>
int launch_apply(lola_state* st, const Call& c, cudaStream_t s) {
  const Layer& L = st->L;
  LaunchScope scope(st, LOLA_KERNEL_UPDATE, s, LOLA_PATH_APPLY_TMA, L.B * L.Hkv);
  const cudaError_t le = launch_pdl(k_update2_tc<DPL, 2>, dim3(L.B * L.Hkv), dim3(kUp2Threads), Update2Smem<DPL>::bytes, s, L, c,
                                    (const uint4*)(st->base + st->lay.wt), (__nv_bfloat16*)nullptr);
  return le == cudaSuccess && cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

template <typename T, int DPL>
int launch_update_chain(lola_state* st, const Call& c, cudaStream_t s) {
  const Layer& L = st->L;
  const int U = L.B * L.Hkv;
  // chunkwise update on TMA-fed tensor-core kernels: every leaving pair already sits in the ring, the
  // occupied part of the sparse cache is a whole number of 64-slot blocks
  if (fast_update_path(st, c)) {
    int rc = launch_score_select<DPL>(st, c, s);
    return rc == LOLA_OK ? launch_apply<DPL>(st, c, s) : rc;
  }
  if (c.mode == UPD_SELECT) {
    const int nE = c.count_g + c.r;
    dim3 grid((nE + kScoreRows - 1) / kScoreRows, U);
    if (st->tensor_path) {
      dim3 tgrid((nE + kScTile - 1) / kScTile, U);
      LaunchScope scope(st, LOLA_KERNEL_SCORE, s, LOLA_PATH_SCORE_MMA, (int)(tgrid.x * tgrid.y));
      k_score_tc<DPL><<<tgrid, 128, ScoreTcSmem<DPL>::bytes, s>>>(L, c);
    } else {
      LaunchScope scope(st, LOLA_KERNEL_SCORE, s, LOLA_PATH_SCORE_GENERIC, (int)(grid.x * grid.y));
      k_score<T, DPL><<<grid, 256, score_smem_floats<DPL>(L.D) * 4, s>>>(L, c);
    }
    if (cudaGetLastError() != cudaSuccess) return LOLA_ERR_CUDA;
  }
  if (c.mode != UPD_NONE) {
    const int nE = c.count_g + c.r;
    size_t sm = (c.mode == UPD_SELECT) ? ((size_t)nE * 8 + (size_t)L.cmax * 4 + (size_t)nE + 16) : 0;
    LaunchScope scope(st, LOLA_KERNEL_SELECT, s, LOLA_PATH_SELECT_KERNEL, U);
    k_select<<<U, 256, sm, s>>>(L, c);
    if (cudaGetLastError() != cudaSuccess) return LOLA_ERR_CUDA;
  }
  if (st->have_maps && !st->force_chain && (c.mode == UPD_NONE || c.mode == UPD_APPEND) && c.r <= kUp2MaxFold)
    return launch_apply<DPL>(st, c, s);  // nothing folds: moves from the work lists and the window roll
  LaunchScope scope(st, LOLA_KERNEL_UPDATE, s, LOLA_PATH_UPDATE_GENERIC, U);
  k_update<T, DPL><<<U, kUpdThreads, update_smem_floats<DPL>(L.D) * 4, s>>>(L, c);
  return cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

template <typename T, int DPL>
int run_prefill(lola_state* st, Call c, cudaStream_t s) {
  int rc = LOLA_OK;
  // Attention and scoring both only read the memories: with outputs wanted and the tensor-core update path
  // in use they run side by side, all on the caller's stream, chained by programmatic dependent launches:
  // the attention kernel waits for everything before it and then lets the scoring kernel (with the selection
  // in its last block per unit) start; the scoring kernel waits for the attention kernel only at its end; the
  // fold waits for the scoring kernel, hence for both.
  if (c.out && fast_update_path(st, c)) {
    rc = launch_attend<T, DPL>(st, c, s, true);
    if (rc != LOLA_OK) return rc;
    rc = launch_score_select<DPL>(st, c, s, (((st->L.g + 1) / 2 + 1) / 2) * st->L.B * st->L.Hkv);
    if (rc != LOLA_OK) return rc;
    return launch_apply<DPL>(st, c, s);
  }
  if (c.out) rc = launch_attend<T, DPL>(st, c, s);
  if (rc != LOLA_OK) return rc;
  return launch_update_chain<T, DPL>(st, c, s);
}

template <int DPL>
int launch_decode_fused(lola_state* st, const Call& c, cudaStream_t s) {
  const Layer& L = st->L;
  const int n_tiles = (L.lam / 64 + (L.eta + 63) / 64 + 1) / 2;
  LaunchScope scope(st, LOLA_KERNEL_DECODE, s, n_tiles <= kDec2MaxTiles ? LOLA_PATH_DECODE_FUSED : LOLA_PATH_DECODE_FUSED_LONG, L.B * L.Hkv);
  const uint4* wt = (const uint4*)(st->base + st->lay.wt);
  if (n_tiles <= kDec2MaxTiles) {          // the pipelined kernel; longer units run the two-row-group kernel
    if (L.g <= 4)
      k_decode2_tc<DPL, 4><<<L.B * L.Hkv, kDec2Threads, DecodeSmem<DPL>::bytes, s>>>(L, c, st->tm_gk, st->tm_gv, st->tm_wk, st->tm_wv, wt);
    else
      k_decode2_tc<DPL, 8><<<L.B * L.Hkv, kDec2Threads, DecodeSmem<DPL>::bytes, s>>>(L, c, st->tm_gk, st->tm_gv, st->tm_wk, st->tm_wv, wt);
    return cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
  }
  if (L.g <= 4)
    k_decode_tc<DPL, 4><<<L.B * L.Hkv, kDecThreads, DecodeSmem<DPL>::bytes, s>>>(
        L, c, st->tm_gk, st->tm_gv, st->tm_wk, st->tm_wv, (const uint4*)(st->base + st->lay.wt));
  else
    k_decode_tc<DPL, 8><<<L.B * L.Hkv, kDecThreads, DecodeSmem<DPL>::bytes, s>>>(
        L, c, st->tm_gk, st->tm_gv, st->tm_wk, st->tm_wv, (const uint4*)(st->base + st->lay.wt));
  return cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

template <typename T, int DPL>
int run_decode(lola_state* st, Call c, cudaStream_t s) {
  // steady state (caches full, one pair leaves the window): the whole step is one kernel
  const bool ablation = (st->cfg.flags & (LOLA_FLAG_QUERY_NO_LINEAR | LOLA_FLAG_QUERY_NO_SPARSE)) != 0;
  if (st->fused_decode && !st->force_chain && !ablation && c.mode == UPD_SELECT && c.r == 1 && c.count_g == st->L.lam)
  {
    return launch_decode_fused<DPL>(st, c, s);
  }
  int rc = launch_update_chain<T, DPL>(st, c, s);
  if (rc != LOLA_OK) return rc;
  return launch_attend<T, DPL>(st, c, s);
}

#define LOLA_DISPATCH(fn, st, ...)                                                            \
  ((st)->cfg.dtype == LOLA_BF16                                                               \
       ? ((st)->cfg.head_dim == 128 ? fn<__nv_bfloat16, 4>(st, __VA_ARGS__) : fn<__nv_bfloat16, 2>(st, __VA_ARGS__)) \
       : ((st)->cfg.head_dim == 128 ? fn<float, 4>(st, __VA_ARGS__) : fn<float, 2>(st, __VA_ARGS__)))

size_t elem_size(const lola_config& c) { return c.dtype == LOLA_BF16 ? 2 : 4; }

// One warp waits, with the same bounded wait every kernel uses, for an mbarrier phase that nothing
// completes; the wait gives up after `limit_ns` and the failure is recorded like any other.
__global__ void k_selftest_wait(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  const uint32_t b = tc::smem_u32(&bar);
  if (threadIdx.x == 0) {
    abort_word = 0;
    tc::mbar_init(b, 1);
    tc::mbar_init_fence();
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = tc::mbar_try_wait(b, 0) || tc::mbar_wait_slow(b, 0, &abort_word, limit_ns);
  if (!ok) atomicOr(status, LOLA_STATUS_SELFTEST);
}

}  // namespace

extern "C" {

size_t lola_state_bytes(const lola_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(*cfg).total;
}

int lola_init_state(const lola_config* cfg, const void* W_dev, void* state_dev, size_t state_bytes, void* stream,
                    lola_state** out) {
  if (!cfg || !W_dev || !state_dev || !out) return LOLA_ERR_ARG;
  if (!config_ok(cfg)) {
    if (cfg->head_dim != 64 && cfg->head_dim != 128 && cfg->head_dim > 0) return LOLA_ERR_UNSUPPORTED;
    return LOLA_ERR_SHAPE;
  }
  if (!aligned(W_dev, 16) || !aligned(state_dev, kAlign)) return LOLA_ERR_ALIGN;
  StateLayout lay = make_layout(*cfg);
  if (state_bytes < lay.total) return LOLA_ERR_SIZE;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return LOLA_ERR_CUDA;
  if (prop.major != 10) return LOLA_ERR_UNSUPPORTED;
  const int sm_count = prop.multiProcessorCount;

  lola_state* st = new (std::nothrow) lola_state();
  if (!st) return LOLA_ERR_ARG;
  st->cfg = *cfg;
  st->lay = lay;
  st->base = (char*)state_dev;
  st->n_seen = 0;
  st->launches = 0;
  st->sm_count = sm_count;
  Layer& L = st->L;
  L.B = cfg->batch; L.Hq = cfg->n_q_heads; L.Hkv = cfg->n_kv_heads; L.g = cfg->n_q_heads / cfg->n_kv_heads;
  L.d = cfg->head_dim; L.F = cfg->feat_half; L.D = 2 * cfg->feat_half;
  L.eta = cfg->window; L.lam = cfg->sparse; L.cmax = cfg->max_chunk;
  L.phi_kind = cfg->phi_kind; L.bf16 = cfg->dtype == LOLA_BF16;
  L.scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  char* b = st->base;
  L.status = (int*)(b + lay.status);
  L.H = (float*)(b + lay.H); L.s = (float*)(b + lay.s);
  L.gk = b + lay.gk; L.gv = b + lay.gv; L.gpos = (int*)(b + lay.gpos); L.score = (float*)(b + lay.score);
  L.wk = b + lay.wk; L.wv = b + lay.wv;
  L.fold_idx = (int*)(b + lay.fold_idx); L.move_src = (int*)(b + lay.move_src); L.move_dst = (int*)(b + lay.move_dst);
  L.counts = (int*)(b + lay.counts); L.thr = (float*)(b + lay.thr);
  L.W = W_dev;

  int rc = LOLA_OK;
  if (cfg->dtype == LOLA_BF16) rc = cfg->head_dim == 128 ? set_smem_attrs<__nv_bfloat16, 4>(L.D) : set_smem_attrs<__nv_bfloat16, 2>(L.D);
  else rc = cfg->head_dim == 128 ? set_smem_attrs<float, 4>(L.D) : set_smem_attrs<float, 2>(L.D);
  if (rc == LOLA_OK && cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, 9 * 16384 + 4 * 16384 + 64) != cudaSuccess)
    rc = LOLA_ERR_CUDA;
  st->tensor_path = cfg->dtype == LOLA_BF16 && cfg->feat_half == 64 && !(cfg->flags & LOLA_FLAG_GENERIC_KERNELS);
  if (rc == LOLA_OK && st->tensor_path) {
    cudaError_t e = cfg->head_dim == 128
        ? cudaFuncSetAttribute(k_score_tc<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScoreTcSmem<4>::bytes)
        : cudaFuncSetAttribute(k_score_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ScoreTcSmem<2>::bytes);
    if (e != cudaSuccess) rc = LOLA_ERR_CUDA;
    e = cfg->head_dim == 128
        ? cudaFuncSetAttribute(k_attend_tc<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttendTcSmem<4>::bytes)
        : cudaFuncSetAttribute(k_attend_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttendTcSmem<2>::bytes);
    if (e != cudaSuccess) rc = LOLA_ERR_CUDA;
  }
  if (rc == LOLA_OK && st->tensor_path && cfg->sparse >= 1 && cfg->window >= 1) {
    const size_t U = (size_t)cfg->batch * cfg->n_kv_heads;
    st->have_maps = make_rows_map(&st->tm_gk, L.gk, U, cfg->sparse, cfg->head_dim, 64) &&
                    make_rows_map(&st->tm_gv, L.gv, U, cfg->sparse, cfg->head_dim, 64) &&
                    make_rows_map(&st->tm_wk, L.wk, U, cfg->window, cfg->head_dim, 64) &&
                    make_rows_map(&st->tm_wv, L.wv, U, cfg->window, cfg->head_dim, 64);
    cudaError_t e[8];
    if (cfg->head_dim == 128) {
      e[0] = cudaFuncSetAttribute(k_decode_tc<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<4>::bytes);
      e[1] = cudaFuncSetAttribute(k_decode_tc<4, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<4>::bytes);
      e[2] = cudaFuncSetAttribute(k_score2_tc<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Score2Smem<4>::bytes);
      e[3] = cudaFuncSetAttribute(k_update2_tc<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Update2Smem<4>::bytes);
      e[4] = cudaFuncSetAttribute(k_attend2_tc<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Attend2Smem<4>::bytes);
      e[5] = cudaFuncSetAttribute(k_decode2_tc<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<4>::bytes);
      e[6] = cudaFuncSetAttribute(k_decode2_tc<4, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<4>::bytes);
    } else {
      e[0] = cudaFuncSetAttribute(k_decode_tc<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<2>::bytes);
      e[1] = cudaFuncSetAttribute(k_decode_tc<2, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<2>::bytes);
      e[2] = cudaFuncSetAttribute(k_score2_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Score2Smem<2>::bytes);
      e[3] = cudaFuncSetAttribute(k_update2_tc<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Update2Smem<2>::bytes);
      e[4] = cudaFuncSetAttribute(k_attend2_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Attend2Smem<2>::bytes);
      e[5] = cudaFuncSetAttribute(k_decode2_tc<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<2>::bytes);
      e[6] = cudaFuncSetAttribute(k_decode2_tc<2, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DecodeSmem<2>::bytes);
    }
    for (int i = 0; i < 7; ++i) if (e[i] != cudaSuccess) st->have_maps = false;   // the older kernel chain serves every shape
    // one shared-memory carve-out for the kernels that follow each other in a step: a change of the
    // carve-out between two launches costs idle time on every SM
    const int co = (int)cudaSharedmemCarveoutMaxShared;
    if (cfg->head_dim == 128) {
      cudaFuncSetAttribute(k_decode_tc<4, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode_tc<4, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode2_tc<4, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode2_tc<4, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_score2_tc<4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_update2_tc<4, 2>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_attend2_tc<4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
    } else {
      cudaFuncSetAttribute(k_decode_tc<2, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode_tc<2, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode2_tc<2, 4>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_decode2_tc<2, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_score2_tc<2>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_update2_tc<2, 2>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
      cudaFuncSetAttribute(k_attend2_tc<2>, cudaFuncAttributePreferredSharedMemoryCarveout, co);
    }
    cudaGetLastError();   // a refused preference is not an error
  }
  // one-kernel generation step: lambda a whole number of 64-row blocks, the row stream within 16 tiles
  st->fused_decode = st->have_maps && cfg->sparse >= 64 && cfg->sparse % 64 == 0 && L.g <= kDecQ &&
                     (cfg->sparse / 64 + (cfg->window + 63) / 64 + 1) / 2 <= kDecMaxTiles;
  if (rc == LOLA_OK && st->tensor_path) {
    cudaStream_t s = (cudaStream_t)stream;
    __nv_bfloat16* img = (__nv_bfloat16*)(st->base + lay.wt);
    if (cfg->head_dim == 128) k_prep_wt_image<4><<<cfg->n_kv_heads, 256, 0, s>>>((const __nv_bfloat16*)W_dev, img, cfg->n_kv_heads);
    else k_prep_wt_image<2><<<cfg->n_kv_heads, 256, 0, s>>>((const __nv_bfloat16*)W_dev, img, cfg->n_kv_heads);
    if (cudaGetLastError() != cudaSuccess) rc = LOLA_ERR_CUDA;
  }
  if (rc == LOLA_OK) rc = lola_reset_state(st, stream);
  if (rc != LOLA_OK) { lola_destroy_state(st); return rc; }
  *out = st;
  return LOLA_OK;
}

int lola_reset_state(lola_state* st, void* stream) {
  if (!st) return LOLA_ERR_ARG;
  const lola_config& c = st->cfg;
  const Layer& L = st->L;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t U = (size_t)c.batch * c.n_kv_heads;
  if (cudaMemsetAsync(st->base, 0, st->lay.wt, s) != cudaSuccess) return LOLA_ERR_CUDA;   // all but the W^T image
  // positions -1, scores and thresholds NaN (all-ones bit pattern)
  if (c.sparse > 0 && cudaMemsetAsync(L.gpos, 0xFF, U * c.sparse * 4, s) != cudaSuccess) return LOLA_ERR_CUDA;
  if (cudaMemsetAsync(L.score, 0xFF, U * ((size_t)c.sparse + c.max_chunk) * 4, s) != cudaSuccess) return LOLA_ERR_CUDA;
  if (cudaMemsetAsync(L.thr, 0xFF, U * 2 * 4, s) != cudaSuccess) return LOLA_ERR_CUDA;
  st->n_seen = 0;
  return LOLA_OK;
}

int lola_prefill_chunk(lola_state* st, const void* q, const void* k, const void* v, int32_t n_tokens, void* out,
                       void* stream) {
  if (!st || !k || !v) return LOLA_ERR_ARG;
  if (out && !q) return LOLA_ERR_ARG;
  if (n_tokens < 1 || n_tokens > st->cfg.max_chunk) return LOLA_ERR_SHAPE;
  if (st->n_seen + n_tokens > 0x7fffffffLL) return LOLA_ERR_SHAPE;
  if (!aligned(k, 16) || !aligned(v, 16) || (out && (!aligned(q, 16) || !aligned(out, 16)))) return LOLA_ERR_ALIGN;
  const Geometry g = plan(st->cfg, st->n_seen, n_tokens);
  st->info = lola_call_info{};
  Call c{};
  c.q = q; c.k = k; c.v = v; c.out = out;
  c.n = n_tokens; c.nq = n_tokens; c.n_seen = (int)st->n_seen;
  c.r = g.r; c.r_pos0 = g.r_pos0; c.count_g = g.count_g; c.mode = g.mode;
  c.att_g = (st->cfg.flags & LOLA_FLAG_QUERY_NO_SPARSE) ? 0 : g.count_g;
  c.att_w0 = (int)st->n_seen - g.cw; c.att_wn = g.cw; c.att_chunk = n_tokens;
  c.att_flags = (st->cfg.flags & LOLA_FLAG_QUERY_NO_LINEAR) ? 1 : 0;
  int rc = LOLA_DISPATCH(run_prefill, st, c, (cudaStream_t)stream);
  if (rc == LOLA_OK) st->n_seen += n_tokens;
  return rc;
}

int lola_prefill_chunks(lola_state* st, const void* q, const void* k, const void* v, int32_t n_chunks, int32_t n_tokens,
                        void* out, void* stream) {
  if (!st || !k || !v) return LOLA_ERR_ARG;
  if (out && !q) return LOLA_ERR_ARG;
  if (n_chunks < 1 || n_tokens < 1 || n_tokens > st->cfg.max_chunk) return LOLA_ERR_SHAPE;
  const lola_config& c = st->cfg;
  const size_t es = c.dtype == LOLA_BF16 ? 2 : 4;
  const size_t qbytes = (size_t)c.batch * n_tokens * c.n_q_heads * c.head_dim * es;
  const size_t kbytes = (size_t)c.batch * n_tokens * c.n_kv_heads * c.head_dim * es;
  for (int i = 0; i < n_chunks; ++i) {
    const int rc = lola_prefill_chunk(st, out ? (const char*)q + (size_t)i * qbytes : nullptr, (const char*)k + (size_t)i * kbytes,
                                      (const char*)v + (size_t)i * kbytes, n_tokens, out ? (char*)out + (size_t)i * qbytes : nullptr, stream);
    if (rc != LOLA_OK) return rc;
  }
  return LOLA_OK;
}

int lola_decode_step(lola_state* st, const void* q, const void* k, const void* v, void* out, void* stream) {
  if (!st || !q || !k || !v || !out) return LOLA_ERR_ARG;
  if (st->n_seen + 1 > 0x7fffffffLL) return LOLA_ERR_SHAPE;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16)) return LOLA_ERR_ALIGN;
  const Geometry g = plan(st->cfg, st->n_seen, 1);
  st->info = lola_call_info{};
  Call c{};
  c.q = q; c.k = k; c.v = v; c.out = out;
  c.n = 1; c.nq = 1; c.n_seen = (int)st->n_seen;
  c.r = g.r; c.r_pos0 = g.r_pos0; c.count_g = g.count_g; c.mode = g.mode;
  const int cw_after = (int)std::min<int64_t>(st->cfg.window, st->n_seen + 1);
  c.att_g = (st->cfg.flags & LOLA_FLAG_QUERY_NO_SPARSE) ? 0 : g.new_count_g;
  c.att_w0 = (int)(st->n_seen + 1) - cw_after; c.att_wn = cw_after; c.att_chunk = 0;
  c.att_flags = (st->cfg.flags & LOLA_FLAG_QUERY_NO_LINEAR) ? 1 : 0;
  int rc = LOLA_DISPATCH(run_decode, st, c, (cudaStream_t)stream);
  if (rc == LOLA_OK) st->n_seen += 1;
  return rc;
}

size_t lola_staging_bytes(const lola_config* cfg, int32_t n_tokens) {
  if (!config_ok(cfg) || n_tokens < 1) return 0;
  const size_t es = elem_size(*cfg), d = cfg->head_dim, B = cfg->batch;
  const size_t qb = align_up(B * n_tokens * cfg->n_q_heads * d * es);
  const size_t kb = align_up(B * n_tokens * cfg->n_kv_heads * d * es);
  return 2 * qb + 2 * kb;
}

static int run_host(lola_state* st, const void* qh, const void* kh, const void* vh, int32_t n, void* oh, void* stg,
                    size_t stg_bytes, void* stream, bool decode) {
  if (!st || !kh || !vh || !stg) return LOLA_ERR_ARG;
  if ((decode || oh) && !qh) return LOLA_ERR_ARG;
  if (decode && !oh) return LOLA_ERR_ARG;
  if (n < 1 || n > st->cfg.max_chunk) return LOLA_ERR_SHAPE;
  if (!aligned(stg, kAlign)) return LOLA_ERR_ALIGN;
  if (stg_bytes < lola_staging_bytes(&st->cfg, n)) return LOLA_ERR_SIZE;
  const lola_config& c = st->cfg;
  const size_t es = elem_size(c), d = c.head_dim, B = c.batch;
  const size_t qbytes = B * n * c.n_q_heads * d * es, kbytes = B * n * c.n_kv_heads * d * es;
  const size_t qb = align_up(qbytes), kb = align_up(kbytes);
  char* p = (char*)stg;
  void *qd = p, *kd = p + qb, *vd = p + qb + kb, *od = p + qb + 2 * kb;
  cudaStream_t s = (cudaStream_t)stream;
  if (oh && cudaMemcpyAsync(qd, qh, qbytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return LOLA_ERR_CUDA;
  if (cudaMemcpyAsync(kd, kh, kbytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return LOLA_ERR_CUDA;
  if (cudaMemcpyAsync(vd, vh, kbytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return LOLA_ERR_CUDA;
  int rc = decode ? lola_decode_step(st, qd, kd, vd, od, stream)
                  : lola_prefill_chunk(st, oh ? qd : nullptr, kd, vd, n, oh ? od : nullptr, stream);
  if (rc != LOLA_OK) return rc;
  if (oh && cudaMemcpyAsync(oh, od, qbytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOLA_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return LOLA_ERR_CUDA;
  return LOLA_OK;
}

int lola_prefill_chunk_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host,
                            int32_t n_tokens, void* out_host, void* staging_dev, size_t staging_bytes, void* stream) {
  return run_host(st, q_host, k_host, v_host, n_tokens, out_host, staging_dev, staging_bytes, stream, false);
}

int lola_decode_step_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host, void* out_host,
                          void* staging_dev, size_t staging_bytes, void* stream) {
  return run_host(st, q_host, k_host, v_host, 1, out_host, staging_dev, staging_bytes, stream, true);
}

static bool ensure_copy_streams(lola_state* st) {
  if (st->cp_in) return true;
  cudaEvent_t* evs[7] = {&st->ev_start, &st->ev_in[0], &st->ev_in[1], &st->ev_done[0], &st->ev_done[1], &st->ev_out[0], &st->ev_out[1]};
  bool ok = cudaStreamCreateWithFlags(&st->cp_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&st->cp_out, cudaStreamNonBlocking) == cudaSuccess;
  for (cudaEvent_t* e : evs) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    for (cudaEvent_t* e : evs) if (*e) { cudaEventDestroy(*e); *e = nullptr; }
    if (st->cp_in) { cudaStreamDestroy(st->cp_in); st->cp_in = nullptr; }
    if (st->cp_out) { cudaStreamDestroy(st->cp_out); st->cp_out = nullptr; }
  }
  return ok;
}

int lola_prefill_host(lola_state* st, const void* q_host, const void* k_host, const void* v_host, int32_t n_chunks,
                      int32_t n_tokens, void* out_host, void* staging_dev, size_t staging_bytes, void* stream) {
  if (!st || !k_host || !v_host || !staging_dev) return LOLA_ERR_ARG;
  if (out_host && !q_host) return LOLA_ERR_ARG;
  if (n_chunks < 1 || n_tokens < 1 || n_tokens > st->cfg.max_chunk) return LOLA_ERR_SHAPE;
  if (!aligned(staging_dev, kAlign)) return LOLA_ERR_ALIGN;
  const size_t per = lola_staging_bytes(&st->cfg, n_tokens);
  if (staging_bytes < 2 * per) return LOLA_ERR_SIZE;
  if (!ensure_copy_streams(st)) return LOLA_ERR_CUDA;
  const lola_config& c = st->cfg;
  const size_t es = elem_size(c), d = c.head_dim, B = c.batch;
  const size_t qbytes = B * n_tokens * c.n_q_heads * d * es, kbytes = B * n_tokens * c.n_kv_heads * d * es;
  const size_t qb = align_up(qbytes), kb = align_up(kbytes);
  cudaStream_t s = (cudaStream_t)stream;
  bool ok = cudaEventRecord(st->ev_start, s) == cudaSuccess && cudaStreamWaitEvent(st->cp_in, st->ev_start, 0) == cudaSuccess;
  int rc = LOLA_OK;
  bool out_pending[2] = {false, false};
  for (int i = 0; ok && rc == LOLA_OK && i < n_chunks; ++i) {
    const int b = i & 1;
    char* p = (char*)staging_dev + (size_t)b * per;
    void *qd = p, *kd = p + qb, *vd = p + qb + kb, *od = p + qb + 2 * kb;
    // copies in (copy stream): this set of device copies is free once the kernels of chunk i - 2 are done
    if (i >= 2) ok = ok && cudaStreamWaitEvent(st->cp_in, st->ev_done[b], 0) == cudaSuccess;
    if (out_host) ok = ok && cudaMemcpyAsync(qd, (const char*)q_host + (size_t)i * qbytes, qbytes, cudaMemcpyHostToDevice, st->cp_in) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(kd, (const char*)k_host + (size_t)i * kbytes, kbytes, cudaMemcpyHostToDevice, st->cp_in) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(vd, (const char*)v_host + (size_t)i * kbytes, kbytes, cudaMemcpyHostToDevice, st->cp_in) == cudaSuccess;
    ok = ok && cudaEventRecord(st->ev_in[b], st->cp_in) == cudaSuccess;
    // kernels (caller's stream): after the copies in, and after the copy out of chunk i - 2 has read `od`
    ok = ok && cudaStreamWaitEvent(s, st->ev_in[b], 0) == cudaSuccess;
    if (out_pending[b]) ok = ok && cudaStreamWaitEvent(s, st->ev_out[b], 0) == cudaSuccess;
    if (!ok) break;
    rc = lola_prefill_chunk(st, out_host ? qd : nullptr, kd, vd, n_tokens, out_host ? od : nullptr, stream);
    if (rc != LOLA_OK) break;
    ok = ok && cudaEventRecord(st->ev_done[b], s) == cudaSuccess;
    // copy out (second copy stream)
    if (out_host) {
      ok = ok && cudaStreamWaitEvent(st->cp_out, st->ev_done[b], 0) == cudaSuccess;
      ok = ok && cudaMemcpyAsync((char*)out_host + (size_t)i * qbytes, od, qbytes, cudaMemcpyDeviceToHost, st->cp_out) == cudaSuccess;
      ok = ok && cudaEventRecord(st->ev_out[b], st->cp_out) == cudaSuccess;
      out_pending[b] = ok;
    }
  }
  // everything joins the caller's stream again
  for (int b = 0; b < 2; ++b)
    if (out_pending[b]) ok = cudaStreamWaitEvent(s, st->ev_out[b], 0) == cudaSuccess && ok;
  const bool synced = cudaStreamSynchronize(st->cp_in) == cudaSuccess && cudaStreamSynchronize(st->cp_out) == cudaSuccess &&
                      cudaStreamSynchronize(s) == cudaSuccess;
  if (rc != LOLA_OK) return rc;
  return ok && synced ? LOLA_OK : LOLA_ERR_CUDA;
}

int lola_read_state(const lola_state* st, const lola_state_view* view, void* stream) {
  if (!st || !view) return LOLA_ERR_ARG;
  const lola_config& c = st->cfg;
  const Layer& L = st->L;
  const size_t U = (size_t)c.batch * c.n_kv_heads, d = c.head_dim, D = L.D, es = elem_size(c);
  const size_t lam = c.sparse, eta = c.window, cm = c.max_chunk;
  cudaStream_t s = (cudaStream_t)stream;
  auto d2h = [&](void* dst, const void* src, size_t bytes) {
    if (!dst || bytes == 0) return true;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, s) == cudaSuccess;
  };
  bool ok = true;
  ok = ok && d2h(view->H, L.H, U * D * d * 4);
  ok = ok && d2h(view->s, L.s, U * D * 4);
  ok = ok && d2h(view->sparse_pos, L.gpos, U * lam * 4);
  ok = ok && d2h(view->sparse_k, L.gk, U * lam * d * es);
  ok = ok && d2h(view->sparse_v, L.gv, U * lam * d * es);
  ok = ok && d2h(view->window_k, L.wk, U * eta * d * es);
  ok = ok && d2h(view->window_v, L.wv, U * eta * d * es);
  ok = ok && d2h(view->threshold, L.thr, U * 2 * 4);
  int status = 0;
  ok = ok && d2h(&status, L.status, 4);
  if (view->sparse_score && lam > 0) {   // the first lambda entries of each unit's score row
    ok = ok && cudaMemcpy2DAsync(view->sparse_score, lam * 4, L.score, (lam + cm) * 4, lam * 4, U,
                                 cudaMemcpyDeviceToHost, s) == cudaSuccess;
  }
  if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return LOLA_ERR_CUDA;
  const Geometry g = plan(c, st->n_seen, 0);
  for (size_t u = 0; u < U; ++u) {
    if (view->sparse_count) view->sparse_count[u] = g.count_g;
    if (view->window_count) view->window_count[u] = g.cw;
    if (view->window_pos) {
      for (size_t j = 0; j < eta; ++j) view->window_pos[u * eta + j] = -1;
      for (int64_t p = st->n_seen - g.cw; p < st->n_seen; ++p) view->window_pos[u * eta + (size_t)(p % (int64_t)eta)] = (int32_t)p;
    }
  }
  if (view->n_seen) for (int b = 0; b < c.batch; ++b) view->n_seen[b] = st->n_seen;
  if (view->status) view->status[0] = status;
  return status == 0 ? LOLA_OK : LOLA_ERR_DEVICE;
}

int lola_write_state(lola_state* st, const lola_state_view* v, void* stream) {
  if (!st || !v) return LOLA_ERR_ARG;
  if (!v->H || !v->s || !v->sparse_count || !v->window_count || !v->n_seen) return LOLA_ERR_ARG;
  const lola_config& c = st->cfg;
  const Layer& L = st->L;
  const size_t U = (size_t)c.batch * c.n_kv_heads, d = c.head_dim, D = L.D, es = elem_size(c);
  const size_t lam = c.sparse, eta = c.window, cm = c.max_chunk;
  if (lam > 0 && (!v->sparse_pos || !v->sparse_k || !v->sparse_v)) return LOLA_ERR_ARG;
  if (eta > 0 && (!v->window_pos || !v->window_k || !v->window_v)) return LOLA_ERR_ARG;
  const int64_t n_seen = v->n_seen[0];
  if (n_seen < 0 || n_seen > 0x7fffffffLL) return LOLA_ERR_ARG;
  for (int b = 0; b < c.batch; ++b) if (v->n_seen[b] != n_seen) return LOLA_ERR_ARG;
  const Geometry g = plan(c, n_seen, 0);
  for (size_t u = 0; u < U; ++u) {
    if (v->sparse_count[u] != g.count_g || v->window_count[u] != g.cw) return LOLA_ERR_ARG;
  }
  // window rows to ring order
  std::vector<char> wk(U * eta * d * es, 0), wv(U * eta * d * es, 0);
  for (size_t u = 0; u < U && eta > 0; ++u) {
    std::vector<char> seen(eta, 0);
    for (int j = 0; j < g.cw; ++j) {
      int64_t p = v->window_pos[u * eta + j];
      if (p < n_seen - g.cw || p >= n_seen) return LOLA_ERR_ARG;
      size_t slot = (size_t)(p % (int64_t)eta);
      if (seen[slot]) return LOLA_ERR_ARG;
      seen[slot] = 1;
      std::memcpy(&wk[(u * eta + slot) * d * es], (const char*)v->window_k + (u * eta + j) * d * es, d * es);
      std::memcpy(&wv[(u * eta + slot) * d * es], (const char*)v->window_v + (u * eta + j) * d * es, d * es);
    }
  }
  std::vector<float> sc(U * (lam + cm));
  { uint32_t nanbits = 0xFFFFFFFFu; float nanv; std::memcpy(&nanv, &nanbits, 4); std::fill(sc.begin(), sc.end(), nanv); }
  if (v->sparse_score)
    for (size_t u = 0; u < U; ++u) std::memcpy(&sc[u * (lam + cm)], v->sparse_score + u * lam, lam * 4);
  cudaStream_t s = (cudaStream_t)stream;
  auto h2d = [&](void* dst, const void* src, size_t bytes) {
    if (bytes == 0) return true;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  };
  bool ok = true;
  ok = ok && h2d(L.H, v->H, U * D * d * 4);
  ok = ok && h2d(L.s, v->s, U * D * 4);
  ok = ok && h2d(L.gpos, v->sparse_pos, U * lam * 4);
  ok = ok && h2d(L.gk, v->sparse_k, U * lam * d * es);
  ok = ok && h2d(L.gv, v->sparse_v, U * lam * d * es);
  ok = ok && h2d(L.score, sc.data(), sc.size() * 4);
  ok = ok && h2d(L.wk, wk.data(), wk.size());
  ok = ok && h2d(L.wv, wv.data(), wv.size());
  if (v->threshold) ok = ok && h2d(L.thr, v->threshold, U * 2 * 4);
  ok = ok && cudaMemsetAsync(L.status, 0, 4, s) == cudaSuccess;      // a replaced state starts healthy
  if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return LOLA_ERR_CUDA;   // host staging dies here
  st->n_seen = n_seen;
  return LOLA_OK;
}

int lola_profile_enable(lola_state* st, int enable) {
  if (!st) return LOLA_ERR_ARG;
  st->profiling = enable != 0;
  return LOLA_OK;
}

int lola_profile_read(lola_state* st, double* ms_by_kind, int64_t* launches_by_kind, void* stream) {
  if (!st || !ms_by_kind || !launches_by_kind) return LOLA_ERR_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return LOLA_ERR_CUDA;
  for (int i = 0; i < LOLA_N_KERNEL_KINDS; ++i) { ms_by_kind[i] = 0.0; launches_by_kind[i] = 0; }
  int rc = LOLA_OK;
  for (ProfRecord& r : st->records) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) rc = LOLA_ERR_CUDA;
    else if (r.kind >= 0 && r.kind < LOLA_N_KERNEL_KINDS) { ms_by_kind[r.kind] += ms; launches_by_kind[r.kind]++; }
    st->pool.push_back(r);
  }
  st->records.clear();
  return rc;
}

int64_t lola_launch_count(const lola_state* st) { return st ? st->launches : -1; }
int64_t lola_tokens_seen(const lola_state* st) { return st ? st->n_seen : -1; }

int lola_set_tokens_seen(lola_state* st, int64_t n_seen) {
  if (!st) return LOLA_ERR_ARG;
  if (n_seen < 0 || n_seen > 0x7fffffffLL) return LOLA_ERR_SHAPE;
  st->n_seen = n_seen;
  return LOLA_OK;
}

int lola_last_call_info(const lola_state* st, lola_call_info* out) {
  if (!st || !out) return LOLA_ERR_ARG;
  *out = st->info;
  return LOLA_OK;
}

int lola_selftest_wait_timeout(lola_state* st, int32_t limit_us, void* stream) {
  if (!st) return LOLA_ERR_ARG;
  if (limit_us < 1 || limit_us > 250000) return LOLA_ERR_ARG;
  st->launches++;
  k_selftest_wait<<<1, 32, 0, (cudaStream_t)stream>>>(st->L.status, (unsigned long long)limit_us * 1000ull);
  return cudaGetLastError() == cudaSuccess ? LOLA_OK : LOLA_ERR_CUDA;
}

int lola_destroy_state(lola_state* st) {
  if (!st) return LOLA_ERR_ARG;
  for (auto* v : {&st->records, &st->pool})
    for (ProfRecord& r : *v) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  if (st->cp_in) { cudaStreamSynchronize(st->cp_in); cudaStreamDestroy(st->cp_in); }
  if (st->cp_out) { cudaStreamSynchronize(st->cp_out); cudaStreamDestroy(st->cp_out); }
  for (cudaEvent_t e : {st->ev_start, st->ev_in[0], st->ev_in[1], st->ev_done[0], st->ev_done[1], st->ev_out[0], st->ev_out[1]})
    if (e) cudaEventDestroy(e);
  delete st;
  return LOLA_OK;
}

// ---------------------------------------------------------------------------------------------
// Generation step whose per-call work lists live in library-owned static device memory.
//
// g_static_lists is a host-side stand-in for the device array: its address means nothing to a
// kernel.  The device address is resolved once per device with cudaGetSymbolAddress and handed
// to the kernels through the Layer block.
// three work lists of LOLA_STATIC_MAX_LIST_ENTRIES ints, then 4 counters per unit
static __device__ __align__(256) int g_static_lists[3 * LOLA_STATIC_MAX_LIST_ENTRIES + 4 * LOLA_STATIC_MAX_UNITS];

static int* static_lists_for_current_device(int* rc_out) {
  static int* ptrs[64] = {nullptr};
  static std::mutex mu;                // first calls from several host threads look the address up one at a time
  std::lock_guard<std::mutex> lock(mu);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { *rc_out = LOLA_ERR_CUDA; return nullptr; }
  if (!ptrs[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_lists) != cudaSuccess || !p) { *rc_out = LOLA_ERR_CUDA; return nullptr; }
    ptrs[dev] = (int*)p;
  }
  *rc_out = LOLA_OK;
  return ptrs[dev];
}

int lola_decode_step_static(lola_state* st, const void* q, const void* k, const void* v, void* out, void* stream) {
  if (!st) return LOLA_ERR_ARG;
  const int64_t U = (int64_t)st->cfg.batch * st->cfg.n_kv_heads;
  if (U > LOLA_STATIC_MAX_UNITS || U * st->cfg.max_chunk > LOLA_STATIC_MAX_LIST_ENTRIES) return LOLA_ERR_SIZE;
  int rc = LOLA_OK;
  int* base = static_lists_for_current_device(&rc);
  if (!base) return rc;
  // Same kernels, same launches as lola_decode_step; only the four work-list pointers differ.
  // Every entry a kernel reads in a step is written earlier in the same step (the selection kernel
  // fills the lists and both counters before the update kernel reads them), so nothing has to be
  // cleared between calls even though the array keeps the previous call's contents.
  const Layer saved = st->L;
  st->L.fold_idx = base;
  st->L.move_src = base + LOLA_STATIC_MAX_LIST_ENTRIES;
  st->L.move_dst = base + 2 * LOLA_STATIC_MAX_LIST_ENTRIES;
  st->L.counts = base + 3 * LOLA_STATIC_MAX_LIST_ENTRIES;
  st->force_chain = true;              // the kernel chain is the path that passes work lists between kernels
  rc = lola_decode_step(st, q, k, v, out, stream);
  st->force_chain = false;
  st->L = saved;                       // kernel arguments were copied at launch
  return rc;
}

const char* lola_strerror(int code) {
  switch (code) {
    case LOLA_OK: return "ok";
    case LOLA_ERR_ARG: return "invalid argument (null pointer, bad enum or inconsistent state view)";
    case LOLA_ERR_SHAPE: return "size out of range";
    case LOLA_ERR_ALIGN: return "pointer not sufficiently aligned";
    case LOLA_ERR_SIZE: return "caller-provided buffer too small";
    case LOLA_ERR_UNSUPPORTED: return "shape or device not supported by this build (needs sm_100)";
    case LOLA_ERR_CUDA: return "CUDA runtime call or kernel launch failed";
    case LOLA_ERR_DEVICE: return "a kernel recorded an internal error in the state's status word";
    default: return "unknown error code";
  }
}

}  // extern "C"
