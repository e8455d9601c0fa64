// Fused SGD step + one CECA gossip round (Eq. (x-iter-dsgd), Eq. (y-iter-dsgd)), and the
// unfused multi-round consensus built from it.
//
// The permutation P^(k) is a cyclic shift (CECA-2P) or a perfect matching (CECA-1P); either way
// it splits the n rows into disjoint cycles.  One thread owns a group of adjacent columns and
// walks one cycle row by row, carrying the message u = z - gamma e of the row it just left in
// registers.  Every element of X, Y and G is therefore read exactly once and every element of
// X+ and Y+ written exactly once (20 bytes per agent-parameter, 16 when Y carries zero weight),
// the message is never stored, and because a thread reads a row before it writes it the update
// may run in place.
#include <cuda_runtime.h>

#include <cstdint>

#include "ceca.h"
#include "plan.h"

namespace ceca {

struct StepArgs {
  const float *X, *Y, *G;
  float *Xo, *Yo;
  int64_t ld;      // elements between consecutive rows
  int64_t ncolv;   // number of column groups (of V floats) this launch covers
  int32_t n, n_cycles, cycle_len, start_stride, hop;
  int32_t payload;  // 0: message from x, 1: message from y
  float a, b, one_minus_a, one_minus_b, gamma;
};

// ---- tiny vector algebra on float4 / float so one kernel body serves both widths ------------
__device__ __forceinline__ float4 vfma(float s, float4 v, float4 w) {
  return make_float4(fmaf(s, v.x, w.x), fmaf(s, v.y, w.y), fmaf(s, v.z, w.z), fmaf(s, v.w, w.w));
}
__device__ __forceinline__ float vfma(float s, float v, float w) { return fmaf(s, v, w); }
__device__ __forceinline__ float4 vmul(float s, float4 v) {
  return make_float4(s * v.x, s * v.y, s * v.z, s * v.w);
}
__device__ __forceinline__ float vmul(float s, float v) { return s * v; }
template <typename V> __device__ __forceinline__ V vzero();
template <> __device__ __forceinline__ float4 vzero<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float vzero<float>() { return 0.f; }

template <typename V> __device__ __forceinline__ V vload(const float *p) {
  return *reinterpret_cast<const V *>(p);
}
template <typename V> __device__ __forceinline__ void vstore(float *p, V v) {
  *reinterpret_cast<V *>(p) = v;
}

constexpr int kThreads = 256;

// One row's own terms: own_x = x - gamma e, own_y = y - gamma e, and the message u (one of them).
template <typename V, bool HAS_G, bool USE_Y>
struct RowRegs {
  V x, y, g;
  __device__ __forceinline__ void load(const StepArgs &p, int64_t off) {
    x = vload<V>(p.X + off);
    if (USE_Y) y = vload<V>(p.Y + off);
    if (HAS_G) g = vload<V>(p.G + off);
  }
  __device__ __forceinline__ void own_terms(const StepArgs &p, V &own_x, V &own_y, V &u) const {
    own_x = HAS_G ? vfma(-p.gamma, g, x) : x;
    own_y = USE_Y ? (HAS_G ? vfma(-p.gamma, g, y) : y) : vzero<V>();
    u = (USE_Y && p.payload) ? own_y : own_x;
  }
};

// RIF = rows whose loads are issued before any of them is consumed (memory-level parallelism per
// thread); MINB = CTAs per SM the register allocation must allow (parallelism across threads).
// Long cycles want a deep RIF, cycles of two rows have only two rows to load and want occupancy.
// YMODE: 1 = Y is read and written; 0 = Y has zero weight this round, it is only written;
//        2 = X only (n a power of two: every round builds its message from x, so X never depends on Y);
//        3 = Y is read but y+ is not stored (last round of a cycle: the next round ignores y).
template <typename V, bool HAS_G, int YMODE, int RIF, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) step_walk_kernel(const StepArgs p) {
  constexpr bool USE_Y = (YMODE == 1 || YMODE == 3);
  constexpr bool WRITE_Y = (YMODE == 0 || YMODE == 1);
  constexpr int VW = sizeof(V) / sizeof(float);
  const int64_t colv = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (colv >= p.ncolv) return;
  const int64_t col = colv * VW;
  using Row = RowRegs<V, HAS_G, USE_Y>;

  for (int32_t c = blockIdx.y; c < p.n_cycles; c += gridDim.y) {
    const int32_t first_row = c * p.start_stride;
    const int64_t first_off = (int64_t)first_row * p.ld + col;
    Row first;
    first.load(p, first_off);

    V first_own_x, first_own_y, u_prev;
    bool first_done = false;
    int32_t row = first_row;
    for (int32_t t = 1; t < p.cycle_len; t += RIF) {
      Row batch[RIF];
      int64_t offs[RIF];
#pragma unroll
      for (int j = 0; j < RIF; ++j) {
        if (t + j < p.cycle_len) {
          row += p.hop;
          if (row >= p.n) row -= p.n;
          offs[j] = (int64_t)row * p.ld + col;
          batch[j].load(p, offs[j]);
        }
      }
      if (!first_done) {
        first.own_terms(p, first_own_x, first_own_y, u_prev);
        first_done = true;
      }
#pragma unroll
      for (int j = 0; j < RIF; ++j) {
        if (t + j < p.cycle_len) {
          V own_x, own_y, u;
          batch[j].own_terms(p, own_x, own_y, u);
          vstore<V>(p.Xo + offs[j], vfma(p.a, own_x, vmul(p.one_minus_a, u_prev)));
          if (WRITE_Y) vstore<V>(p.Yo + offs[j], vfma(p.b, own_y, vmul(p.one_minus_b, u_prev)));
          u_prev = u;
        }
      }
    }
    if (!first_done) first.own_terms(p, first_own_x, first_own_y, u_prev);  // cycle of one row
    // close the cycle: the first row receives the message of the last one
    vstore<V>(p.Xo + first_off, vfma(p.a, first_own_x, vmul(p.one_minus_a, u_prev)));
    if (WRITE_Y) vstore<V>(p.Yo + first_off, vfma(p.b, first_own_y, vmul(p.one_minus_b, u_prev)));
  }
}

template <typename V, int RIF, int MINB>
static cudaError_t launch_walk_shape(const StepArgs &args, bool has_g, int ymode, cudaStream_t stream) {
  const int64_t blocks_x = (args.ncolv + kThreads - 1) / kThreads;
  if (blocks_x > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  dim3 grid((unsigned)blocks_x, (unsigned)(args.n_cycles < 65535 ? args.n_cycles : 65535));
  if (has_g) {
    if (ymode == 1)      step_walk_kernel<V, true, 1, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else if (ymode == 0) step_walk_kernel<V, true, 0, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else if (ymode == 2) step_walk_kernel<V, true, 2, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else                 step_walk_kernel<V, true, 3, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
  } else {
    if (ymode == 1)      step_walk_kernel<V, false, 1, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else if (ymode == 0) step_walk_kernel<V, false, 0, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else if (ymode == 2) step_walk_kernel<V, false, 2, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
    else                 step_walk_kernel<V, false, 3, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);
  }
  return cudaGetLastError();
}

// Launch shapes, chosen from a sweep on a B200 at n = 100, d = 25.6M and n = 24, d = 11.7M:
// cycles of two rows (every CECA-1P round, and the 2-port shift n/2) have nothing to pipeline and
// run fastest with many resident CTAs; long walks want four rows of loads in flight per thread.
template <typename V>
static cudaError_t launch_walk(const StepArgs &args, bool has_g, int ymode, cudaStream_t stream) {
  if (args.ncolv <= 0) return cudaSuccess;
  if (args.cycle_len <= 2)
    return (ymode == 1 || ymode == 3) ? launch_walk_shape<V, 1, 4>(args, has_g, ymode, stream)
                      : launch_walk_shape<V, 1, 6>(args, has_g, ymode, stream);
  if (args.cycle_len <= 4) return launch_walk_shape<V, 2, 4>(args, has_g, ymode, stream);
  return launch_walk_shape<V, 4, 2>(args, has_g, ymode, stream);
}

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Enqueues one iteration.  Arguments are assumed validated.  Yo == nullptr: y+ is not stored (the
// caller has checked that this is legal); Y is then still read if the round needs it.
cudaError_t enqueue_step(const Plan &plan, const float *X, const float *Y, const float *G, float *Xo,
                         float *Yo, int32_t n, int64_t d, int64_t ld, float gamma,
                         cudaStream_t stream) {
  StepArgs a;
  a.X = X; a.Y = Y; a.G = G; a.Xo = Xo; a.Yo = Yo;
  a.ld = ld; a.n = n;
  a.n_cycles = plan.walk.n_cycles; a.cycle_len = plan.walk.cycle_len;
  a.start_stride = plan.walk.start_stride; a.hop = plan.walk.hop;
  a.payload = plan.rd.payload;
  a.a = plan.a; a.b = plan.b; a.one_minus_a = plan.one_minus_a; a.one_minus_b = plan.one_minus_b;
  a.gamma = gamma;
  const bool has_g = (G != nullptr);
  const int ymode = Yo ? (plan.reads_y ? 1 : 0) : ((Y && plan.reads_y) ? 3 : 2);
  const bool use_y = (ymode == 1 || ymode == 3);
  const bool vec_ok = (ld % 4 == 0) && aligned16(X) && aligned16(Xo) && (!Yo || aligned16(Yo)) &&
                      (!use_y || aligned16(Y)) && (!has_g || aligned16(G));
  const int64_t d_vec = vec_ok ? (d / 4) * 4 : 0;  // columns covered by 128-bit accesses
  if (d_vec > 0) {
    a.ncolv = d_vec / 4;
    cudaError_t e = launch_walk<float4>(a, has_g, ymode, stream);
    if (e != cudaSuccess) return e;
  }
  if (d_vec < d) {  // ragged tail (or everything, when rows are not 16-byte aligned)
    StepArgs t = a;
    t.X = X + d_vec; t.Xo = Xo + d_vec; t.Yo = Yo ? Yo + d_vec : nullptr;
    t.Y = Y ? Y + d_vec : nullptr;
    t.G = G ? G + d_vec : nullptr;
    t.ncolv = d - d_vec;
    cudaError_t e = launch_walk<float>(t, has_g, ymode, stream);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

ceca_status_t check_matrix_args(const void *X, const void *X_out, int32_t n, int64_t d, int64_t ld) {
  if (!X || !X_out || n < 1 || d < 1 || ld < d) return CECA_ERR_INVALID_ARG;
  if ((uint64_t)n * (uint64_t)ld > (uint64_t)1 << 60) return CECA_ERR_INVALID_ARG;
  return CECA_OK;
}

}  // namespace ceca

extern "C" ceca_status_t ceca_gossip_sgd_step(const float *X, const float *Y, const float *G,
                                              float *X_out, float *Y_out, int32_t n, int64_t d,
                                              int64_t ld, float gamma, ceca_variant_t variant,
                                              int64_t k, void *stream) {
  ceca_status_t st = ceca::check_matrix_args(X, X_out, n, d, ld);
  if (st != CECA_OK) return st;
  ceca::Plan plan;
  st = ceca::make_plan(n, variant, k, &plan);
  if (st != CECA_OK) return st;
  if (!Y_out) {
    // y+ may be dropped in two situations: n-1 is all ones (no round ever builds its message from y,
    // so Y is not needed at all), or this is the last round of a cycle (round 0 ignores y and
    // overwrites it)
    const bool power_of_two = (n & (n - 1)) == 0;
    const bool last_round = plan.rd.tau > 0 && plan.rd.r == plan.rd.tau - 1;
    if (!(Y ? last_round : power_of_two)) return CECA_ERR_INVALID_ARG;
  } else if (!Y && plan.reads_y) {
    return CECA_ERR_INVALID_ARG;
  }
  // X_out == X and Y_out == Y are fine (read-then-write by one thread); crossed aliases are not
  if (X_out == Y_out || (const float *)X_out == Y || (Y_out && (const float *)Y_out == X) ||
      (G && ((const float *)X_out == G || (const float *)Y_out == G)))
    return CECA_ERR_UNSUPPORTED;
  cudaError_t e = ceca::enqueue_step(plan, X, Y, G, X_out, Y_out, n, d, ld, gamma,
                                     static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}
