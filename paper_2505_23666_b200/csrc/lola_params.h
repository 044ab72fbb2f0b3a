// Device-visible parameter blocks shared by the host API and the kernels.
#pragma once
#include <cstdint>

namespace lola {

// Update kinds for one call (decided on the host: every count is a function of tokens seen).
enum UpdateMode : int {
  UPD_NONE = 0,    // nothing leaves the window
  UPD_APPEND = 1,  // |E| <= lambda: leaving pairs go to free slots, nothing scored or folded
  UPD_SELECT = 2,  // score E, keep top-lambda, fold the rest
  UPD_FOLD_ALL = 3 // lambda == 0: every leaving pair is folded, nothing scored
};

struct Layer {          // fixed for the life of a state
  int B, Hq, Hkv, g, d, F, D, eta, lam, cmax;
  int phi_kind;         // 0 softmax halves, 1 exp
  int bf16;             // 1: bf16 storage and bf16-rounded operands in the scoring contraction
  float scale;
  // state arrays (device)
  float* H;             // [U, D, d]
  float* s;             // [U, D]
  void* gk;             // [U, lam, d]
  void* gv;             // [U, lam, d]
  int* gpos;            // [U, lam]
  float* score;         // [U, lam + cmax]: slot scores, then scores of the leaving pairs
  void* wk;             // [U, eta, d] ring, slot = position % eta
  void* wv;
  int* fold_idx;        // [U, cmax] E-indices of the pairs to fold
  int* move_src;        // [U, cmax] index (into the leaving pairs) of each pair entering G
  int* move_dst;        // [U, cmax] slot it goes to
  int* counts;          // [U, 4]: n_fold, n_move, scoring blocks that have finished (0 between calls), (unused)
  float* thr;           // [U, 2]
  int* status;          // [1]
  const void* W;        // [Hkv, d, F]
};

// Sticky device status word: once a kernel has recorded a failure (a bounded wait that ran out, a bounds
// violation) every later kernel of the state returns at once, so the memories stay as the failure left them
// until lola_reset_state / lola_write_state.
#ifdef __CUDACC__
__device__ __forceinline__ bool state_failed(const Layer& L) { return *reinterpret_cast<volatile const int*>(L.status) != 0; }
#endif

struct Call {           // one prefill chunk or decode step
  const void* q;        // [B, nq, Hq, d]
  const void* k;        // [B, n, Hkv, d] incoming pairs
  const void* v;
  void* out;            // [B, nq, Hq, d]
  int n;                // incoming tokens
  int nq;               // query rows per head
  int n_seen;           // tokens consumed before this call
  // eviction geometry
  int r;                // pairs leaving the window
  int r_pos0;           // position of the first leaving pair
  int count_g;          // occupied slots before the update
  int mode;             // UpdateMode
  // attention geometry
  int att_g;            // occupied slots the queries see
  int att_w0;           // first window position the queries see
  int att_wn;           // number of window positions the queries see (all in the ring)
  int att_chunk;        // incoming tokens seen causally straight from k, v (prefill) or 0 (decode)
  int att_flags;        // bit 0: the queries do not see H, s (the linear terms of Eq. 14 are left out)
};

}  // namespace lola
