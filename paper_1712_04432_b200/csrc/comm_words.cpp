// mbd_comm_words: bandwidth terms of the paper's communication-cost model, Eq. 8
// (integrated model + batch parallelism) and Eq. 9 (with domain-split layers), per
// layer, as exact 64-bit integers.  Host only.
//
// Each term is evaluated as one fraction -- multiply first (128-bit), divide last --
// and rounded up when it is not integral.  The halo terms vanish for a single strip,
// the dX all-reduce is absent for the first layer (Section 2.2), |W_i| follows Eq. 2.
#include "../../include/mbd.h"

namespace {

typedef __int128 i128;

bool ceil_div_to_i64(i128 num, i128 den, int64_t* out) {
  if (den <= 0 || num < 0) return false;
  const i128 q = (num + den - 1) / den;
  if (q > static_cast<i128>(INT64_MAX)) return false;
  *out = static_cast<int64_t>(q);
  return true;
}

}  // namespace

extern "C" mbd_status mbd_comm_words(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, mbd_words* out) {
  if (!layers || !out || L < 1 || B < 1) return MBD_E_INVALID;
  if (P_r < 1 || P_c < 1 || P_c > B) return MBD_E_GRID;
  const i128 P = static_cast<i128>(P_r) * P_c;
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    mbd_words w = {0, 0, 0, 0, 0};
    i128 nW, din, dout;
    if (l.kind == MBD_CONV3X3) {
      if (l.C_in < 1 || l.C_out < 1 || l.H < 1 || l.W < 1 || l.kh < 1 || l.kw < 1) return MBD_E_INVALID;
      nW = static_cast<i128>(l.kh) * l.kw * l.C_in * l.C_out;      // Eq. 2
      const int st = l.stride > 1 ? l.stride : 1;
      if (l.H % st || l.W % st) return MBD_E_INVALID;
      din = static_cast<i128>(l.H) * l.W * l.C_in;
      dout = static_cast<i128>(l.H / st) * (l.W / st) * l.C_out;      // a stride-s layer keeps every s-th position
    } else if (l.kind == MBD_FC) {
      if (l.d_in < 1 || l.d_out < 1) return MBD_E_INVALID;
      nW = static_cast<i128>(l.d_in) * l.d_out;
      din = l.d_in;
      dout = l.d_out;
    } else {
      return MBD_E_INVALID;
    }
    bool ok = true;
    if (l.split == MBD_SPLIT_MODEL) {
      ok = ok && ceil_div_to_i64(static_cast<i128>(B) * (P_r - 1) * dout, P, &w.allgather_y);
      if (i >= 1) ok = ok && ceil_div_to_i64(static_cast<i128>(2) * B * (P_r - 1) * din, P, &w.allreduce_dx);
      ok = ok && ceil_div_to_i64(static_cast<i128>(2) * (P_c - 1) * nW, P, &w.allreduce_dw);
    } else if (l.split == MBD_SPLIT_DOMAIN) {
      if (l.kind != MBD_CONV3X3) return MBD_E_INVALID;   // no halo notion for an FC layer
      if (P_r > 1) {
        ok = ok && ceil_div_to_i64(static_cast<i128>(B) * l.W * l.C_in * (l.kh / 2), P_c, &w.halo_fwd);
        ok = ok && ceil_div_to_i64(static_cast<i128>(B) * (l.W / (l.stride > 1 ? l.stride : 1)) * l.C_out * (l.kh / 2), P_c, &w.halo_bwd);   // Y_W
      }
      ok = ok && ceil_div_to_i64(static_cast<i128>(2) * (P - 1) * nW, P, &w.allreduce_dw);
    } else if (l.split == MBD_SPLIT_BATCH) {
      if (P > static_cast<i128>(B)) return MBD_E_GRID;      // one sample per process at least
      // Section 3's improved case: the layer is batch-parallel on 1 x P; its one term is Eq. 4's all-reduce over all P
      ok = ok && ceil_div_to_i64(static_cast<i128>(2) * (P - 1) * nW, P, &w.allreduce_dw);
    } else {
      return MBD_E_INVALID;
    }
    if (!ok) return MBD_E_INVALID;   // overflow of int64
    out[i] = w;
  }
  return MBD_OK;
}

extern "C" const char* mbd_strerror(mbd_status s) {
  switch (s) {
    case MBD_OK: return "ok";
    case MBD_E_INVALID: return "invalid argument";
    case MBD_E_GRID: return "process grid not realisable for this network and batch";
    case MBD_E_ALLOC: return "allocation failed";
    case MBD_E_CUDA: return "CUDA call failed";
    case MBD_E_STATE: return "call order violated (forward -> backward -> sgd_step)";
    case MBD_E_TIMEOUT: return "a bounded device-side wait timed out";
    case MBD_E_UNSUPPORTED: return "unsupported shape or layer kind";
    case MBD_E_TOO_LARGE: return "problem exceeds the fixed scratch capacity of the allocation-free entry point";
  }
  return "unknown status";
}
