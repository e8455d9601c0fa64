// Internal: the per-iteration plan the launch wrappers derive from (n, variant, k).
#pragma once
#include <cstdint>
#include "ceca.h"

namespace ceca {

// The permutation P^(k) as a set of disjoint cycles that a single thread can walk:
// cycle c visits rows start_stride*c, +hop, +2*hop, ... (mod n), cycle_len rows in total, and
// every visited row receives the message of the row visited just before it (the first row
// receives from the last one).
//   CECA-2P: shift by s = n_r + delta_r  -> gcd(n, s) cycles of length n / gcd(n, s).
//   CECA-1P: perfect matching             -> n / 2 cycles of length 2, even row first.
struct Walk {
  int32_t n_cycles, cycle_len, start_stride, hop;
};

struct Plan {
  ceca_round_t rd;
  Walk walk;
  float a, b, one_minus_a, one_minus_b;  // fp64 values rounded once
  bool reads_y;                          // false only when b == 0 and the message is built from x
};

// Fills `plan`; same error codes as ceca_schedule.
ceca_status_t make_plan(int32_t n, ceca_variant_t variant, int64_t k, Plan *plan);

}  // namespace ceca
