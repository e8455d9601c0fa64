// Host side of the library: the CECA schedule (integers only) and the launch plan.
//
// Sec. 3.1 "Auxiliary variables": tau = ceil(log2 n) is the bit length of n-1, delta_r is bit
// (tau-1-r) of n-1 and the recurrence n_{r+1} = 2 n_r + delta_r makes n_r the top r bits of n-1.
#include <numeric>

#include "ceca.h"
#include "plan.h"

namespace ceca {

static inline int32_t bit_length(uint32_t v) { return v == 0 ? 0 : 32 - __builtin_clz(v); }

static ceca_status_t fill_round(int32_t n, ceca_variant_t variant, int64_t k, ceca_round_t *rd) {
  if (n < 1 || k < 0) return CECA_ERR_INVALID_ARG;
  if (variant != CECA_1P && variant != CECA_2P) return CECA_ERR_INVALID_ARG;
  if (variant == CECA_1P && n > 1 && (n & 1)) return CECA_ERR_ODD_N_1P;
  const uint32_t top = (uint32_t)(n - 1);
  const int32_t tau = bit_length(top);
  rd->n = n;
  rd->tau = tau;
  if (tau == 0) {  // a single agent: nothing to mix, both models just take the SGD step
    rd->r = 0; rd->delta = 1; rd->n_r = 0; rd->payload = 0;
    rd->a_num = rd->a_den = rd->b_num = rd->b_den = 1;
    rd->a = rd->b = 1.0;
    return CECA_OK;
  }
  const int32_t r = (int32_t)(k % tau);
  const int32_t n_r = (int32_t)(top >> (tau - r));       // the r leading bits of n-1
  const int32_t delta = (int32_t)((top >> (tau - 1 - r)) & 1u);
  rd->r = r; rd->delta = delta; rd->n_r = n_r;
  rd->payload = delta ? 0 : 1;
  const int32_t den = 2 * n_r + 1;
  if (delta) { rd->a_num = 1; rd->a_den = 2; rd->b_num = n_r; rd->b_den = den; }
  else       { rd->a_num = n_r + 1; rd->a_den = den; rd->b_num = 1; rd->b_den = 2; }
  rd->a = (double)rd->a_num / (double)rd->a_den;
  rd->b = (double)rd->b_num / (double)rd->b_den;
  return CECA_OK;
}

ceca_status_t make_plan(int32_t n, ceca_variant_t variant, int64_t k, Plan *plan) {
  ceca_status_t st = fill_round(n, variant, k, &plan->rd);
  if (st != CECA_OK) return st;
  const ceca_round_t &rd = plan->rd;
  if (n == 1) {
    plan->walk = {1, 1, 1, 0};
  } else if (variant == CECA_2P) {
    const int32_t s = rd.n_r + rd.delta;
    const int32_t g = std::gcd(n, s);
    plan->walk = {g, n / g, 1, s};
  } else {
    plan->walk = {n / 2, 2, 2, 2 * rd.n_r + 1};
  }
  plan->a = (float)rd.a;
  plan->b = (float)rd.b;
  plan->one_minus_a = (float)(1.0 - rd.a);
  plan->one_minus_b = (float)(1.0 - rd.b);
  plan->reads_y = !(rd.payload == 0 && rd.b_num == 0);
  return CECA_OK;
}

}  // namespace ceca

extern "C" ceca_status_t ceca_schedule(int32_t n, ceca_variant_t variant, int64_t k,
                                       ceca_round_t *round, int32_t *recv_from, int32_t *send_to) {
  ceca_round_t rd;
  ceca_status_t st = ceca::fill_round(n, variant, k, &rd);
  if (st != CECA_OK) return st;
  if (round) *round = rd;
  if (!recv_from && !send_to) return CECA_OK;
  if (n == 1) {
    if (recv_from) recv_from[0] = 0;
    if (send_to) send_to[0] = 0;
    return CECA_OK;
  }
  if (variant == CECA_2P) {
    const int32_t s = rd.n_r + rd.delta;  // 1 <= s <= n-1
    for (int32_t i = 0; i < n; ++i) {
      if (recv_from) recv_from[i] = i >= s ? i - s : i - s + n;
      if (send_to) send_to[i] = i + s < n ? i + s : i + s - n;
    }
  } else {
    const int32_t o = 2 * rd.n_r + 1;     // odd and < n for even n
    for (int32_t i = 0; i < n; i += 2) {  // even row i is matched with the odd row j
      const int32_t j = i + o < n ? i + o : i + o - n;
      if (recv_from) { recv_from[i] = j; recv_from[j] = i; }
      if (send_to) { send_to[i] = j; send_to[j] = i; }
    }
  }
  return CECA_OK;
}

extern "C" const char *ceca_status_string(ceca_status_t status) {
  switch (status) {
    case CECA_OK: return "ok";
    case CECA_ERR_INVALID_ARG: return "invalid argument";
    case CECA_ERR_ODD_N_1P: return "CECA-1P needs an even number of agents";
    case CECA_ERR_ALIGNMENT: return "fused consensus needs 16-byte aligned rows";
    case CECA_ERR_UNSUPPORTED: return "unsupported combination of arguments";
    case CECA_ERR_WORKSPACE: return "workspace missing or too small";
    case CECA_ERR_CUDA: return "CUDA call failed";
    case CECA_ERR_STATIC_SCRATCH: return "problem too large for the built-in scratch buffer";
  }
  return "unknown status";
}
