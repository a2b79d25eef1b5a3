// Communication time model of the paper (Eq. 3-9 with their latency terms) and the choice
// of the process grid by evaluating it for every factorisation of P (Section 3).  Host only.
//
// A collective costs alpha * messages + beta * words.  Bruck all-gather over a group of p
// processes: ceil(log2 p) messages; ring all-reduce: twice that, and twice the words; a halo
// exchange: one message.  The word counts are the real-valued terms of Eq. 8 / Eq. 9 (the
// integer counts of mbd_comm_words are these, rounded up).
#include <vector>

#include "../../include/mbd.h"

namespace {

int ceil_log2(long long p) {
  int k = 0;
  while ((1ll << k) < p) ++k;
  return k;
}

struct Dims {
  double nW, din, dout;
  bool conv;
};

bool layer_dims(const mbd_layer& l, Dims* d) {
  if (l.kind == MBD_CONV3X3) {
    if (l.C_in < 1 || l.C_out < 1 || l.H < 1 || l.W < 1 || l.kh < 1 || l.kw < 1) return false;
    d->nW = static_cast<double>(l.kh) * l.kw * l.C_in * l.C_out;      // Eq. 2
    d->din = static_cast<double>(l.H) * l.W * l.C_in;
    const int st = l.stride > 1 ? l.stride : 1;                      // a stride-s layer keeps every s-th position
    d->dout = static_cast<double>(l.H / st) * (l.W / st) * l.C_out;
    d->conv = true;
    return true;
  }
  if (l.kind == MBD_FC) {
    if (l.d_in < 1 || l.d_out < 1) return false;
    d->nW = static_cast<double>(l.d_in) * static_cast<double>(l.d_out);
    d->din = static_cast<double>(l.d_in);
    d->dout = static_cast<double>(l.d_out);
    d->conv = false;
    return true;
  }
  return false;
}

// One layer's row of Eq. 9 on its own grid.  `first` = the network's first layer (no dX).
mbd_status layer_row(const mbd_layer& l, int split, bool first, double B, int P_r, int P_c, const mbd_machine& m,
                     mbd_times* t) {
  Dims d;
  if (!layer_dims(l, &d)) return MBD_E_INVALID;
  *t = mbd_times{0, 0, 0, 0, 0};
  const double pr = P_r, pc = P_c, P = pr * pc;
  if (split == MBD_SPLIT_MODEL) {
    const double share = (B / pc) * ((pr - 1.0) / pr);
    t->allgather_y = m.alpha * ceil_log2(P_r) + m.beta * share * d.dout;
    if (!first) t->allreduce_dx = 2.0 * (m.alpha * ceil_log2(P_r) + m.beta * share * d.din);
    t->allreduce_dw = 2.0 * (m.alpha * ceil_log2(P_c) + m.beta * ((pc - 1.0) / pc) * (d.nW / pr));
    return MBD_OK;
  }
  if (split == MBD_SPLIT_DOMAIN) {
    if (!d.conv) return MBD_E_INVALID;   // no halo notion for a fully connected layer
    if (P_r > 1 && l.kh / 2 > 0) {         // a 1 x 1 convolution exchanges nothing (remark after Eq. 7)
      const double rows = static_cast<double>(l.kh / 2);
      t->halo_fwd = m.alpha + m.beta * (B / pc) * l.W * l.C_in * rows;
      t->halo_bwd = m.alpha + m.beta * (B / pc) * (l.W / (l.stride > 1 ? l.stride : 1)) * l.C_out * rows;     // Y_W
    }
    t->allreduce_dw = 2.0 * (m.alpha * ceil_log2(static_cast<long long>(P_r) * P_c) + m.beta * ((P - 1.0) / P) * d.nW);
    return MBD_OK;
  }
  if (split == MBD_SPLIT_BATCH)   // forced onto 1 x P (Section 3's improved case): only dW moves, over all P processes
    return layer_row(l, MBD_SPLIT_MODEL, first, B, 1, P_r * P_c, m, t);
  return MBD_E_INVALID;
}

bool feasible(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c, bool fc_only) {
  if (P_c > B) return false;
  for (int i = 0; i < L; ++i) {
    const mbd_layer& l = layers[i];
    if (fc_only && l.kind != MBD_FC) continue;
    if (l.split == MBD_SPLIT_MODEL) {
      const int st = l.stride > 1 ? l.stride : 1;
      const double dout = l.kind == MBD_FC ? static_cast<double>(l.d_out) : static_cast<double>(l.H / st) * (l.W / st) * l.C_out;
      if (static_cast<double>(P_r) > dout) return false;
    } else if (l.split == MBD_SPLIT_BATCH) {
      if (static_cast<int64_t>(P_r) * P_c > B) return false;
    } else if (P_r > l.H) {
      return false;
    }
  }
  return true;
}

bool valid_machine(const mbd_machine* m) { return m && m->alpha >= 0.0 && m->beta >= 0.0; }

double total_time(double compute, double fwd, double bwd, int overlap) {
  if (!overlap) return compute + fwd + bwd;
  const double exposed = bwd - 2.0 * compute / 3.0;
  return compute + fwd + (exposed > 0.0 ? exposed : 0.0);
}

mbd_status table(const mbd_layer* layers, int L, int64_t B, int P, const mbd_machine* m, int policy, double compute,
                 int overlap, int charge, std::vector<mbd_grid_row>* rows) {
  if (!layers || L < 1 || B < 1 || P < 1 || !valid_machine(m) || compute < 0.0) return MBD_E_INVALID;
  if (policy != MBD_GRID_UNIFORM && policy != MBD_GRID_CONV_BATCH) return MBD_E_INVALID;
  for (int pr = 1; pr <= P; ++pr) {
    if (P % pr) continue;
    const int pc = P / pr;
    if (policy == MBD_GRID_CONV_BATCH ? (P > B || !feasible(layers, L, B, pr, pc, true)) : !feasible(layers, L, B, pr, pc, false))
      continue;
    double fwd = 0.0, bwd = 0.0;
    bool charged = false;
    for (int i = 0; i < L; ++i) {
      const mbd_layer& l = layers[i];
      mbd_times t;
      mbd_status s;
      if (policy == MBD_GRID_CONV_BATCH && l.kind == MBD_CONV3X3) {
        s = layer_row(l, MBD_SPLIT_MODEL, i == 0, static_cast<double>(B), 1, P, *m, &t);   // pure batch: only dW moves
      } else {
        s = layer_row(l, l.split, i == 0, static_cast<double>(B), pr, pc, *m, &t);
        if (policy == MBD_GRID_CONV_BATCH && charge && !charged && pr > 1 && i > 0 && l.kind == MBD_FC) {
          // first fully connected layer: its input arrives batch-distributed from the convolutions
          bool first_fc = true;
          for (int j = 0; j < i; ++j) first_fc = first_fc && layers[j].kind != MBD_FC;
          if (first_fc) {
            fwd += m->alpha * ceil_log2(pr) +
                   m->beta * (static_cast<double>(B) / pc) * ((pr - 1.0) / pr) * static_cast<double>(l.d_in);
            charged = true;
          }
        }
      }
      if (s != MBD_OK) return s;
      fwd += t.allgather_y + t.halo_fwd;
      bwd += t.allreduce_dx + t.allreduce_dw + t.halo_bwd;
    }
    mbd_grid_row r;
    r.P_r = pr; r.P_c = pc;
    r.comm_fwd = fwd; r.comm_bwd = bwd; r.comm = fwd + bwd;
    r.total = total_time(compute, fwd, bwd, overlap);
    rows->push_back(r);
  }
  return MBD_OK;
}

}  // namespace

extern "C" mbd_status mbd_comm_time(const mbd_layer* layers, int L, int64_t B, int P_r, int P_c,
                                    const mbd_machine* machine, mbd_times* out) {
  if (!layers || !out || L < 1 || B < 1 || !valid_machine(machine)) return MBD_E_INVALID;
  if (P_r < 1 || P_c < 1 || P_c > B) return MBD_E_GRID;
  for (int i = 0; i < L; ++i) {
    const mbd_status s = layer_row(layers[i], layers[i].split, i == 0, static_cast<double>(B), P_r, P_c, *machine, &out[i]);
    if (s != MBD_OK) return s;
  }
  return MBD_OK;
}

extern "C" mbd_status mbd_redistribute_time(int64_t B, int P_r, int P_c, int64_t d, const mbd_machine* machine,
                                            double* out) {
  if (!out || B < 1 || d < 1 || !valid_machine(machine)) return MBD_E_INVALID;
  if (P_r < 1 || P_c < 1 || P_c > B) return MBD_E_GRID;
  *out = machine->alpha * ceil_log2(P_r) +
         machine->beta * (static_cast<double>(B) / P_c) * ((P_r - 1.0) / P_r) * static_cast<double>(d);
  return MBD_OK;
}

extern "C" mbd_status mbd_total_time(double compute, double comm_fwd, double comm_bwd, int overlap, double* out) {
  if (!out || compute < 0.0 || comm_fwd < 0.0 || comm_bwd < 0.0) return MBD_E_INVALID;
  *out = total_time(compute, comm_fwd, comm_bwd, overlap);
  return MBD_OK;
}

extern "C" mbd_status mbd_grid_table(const mbd_layer* layers, int L, int64_t B, int P, const mbd_machine* machine,
                                     int policy, double compute, int overlap, int charge_redistribution,
                                     mbd_grid_row* rows, int cap, int* n_rows) {
  if (!n_rows || cap < 0) return MBD_E_INVALID;
  std::vector<mbd_grid_row> t;
  const mbd_status s = table(layers, L, B, P, machine, policy, compute, overlap, charge_redistribution, &t);
  if (s != MBD_OK) return s;
  *n_rows = static_cast<int>(t.size());
  if (!rows) return MBD_OK;
  if (cap < *n_rows) return MBD_E_INVALID;
  for (int i = 0; i < *n_rows; ++i) rows[i] = t[i];
  return MBD_OK;
}

extern "C" mbd_status mbd_choose_grid(const mbd_layer* layers, int L, int64_t B, int P, const mbd_machine* machine,
                                      int policy, double compute, int overlap, int charge_redistribution,
                                      mbd_grid_row* best) {
  if (!best) return MBD_E_INVALID;
  std::vector<mbd_grid_row> t;
  const mbd_status s = table(layers, L, B, P, machine, policy, compute, overlap, charge_redistribution, &t);
  if (s != MBD_OK) return s;
  if (t.empty()) return MBD_E_GRID;
  size_t b = 0;
  for (size_t i = 1; i < t.size(); ++i)
    if (t[i].total < t[b].total) b = i;       // rows ascend in P_r: a tie keeps the smaller one
  *best = t[b];
  return MBD_OK;
}
