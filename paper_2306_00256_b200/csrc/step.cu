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
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "ceca.h"
#include "plan.h"

namespace ceca {

// X, Y, X+ and Y+ are stored as TXY, G as TG (float or __nv_bfloat16); the arithmetic is fp32 either way.
struct StepArgs {
  const void *X, *Y, *G;
  void *Xo, *Yo;
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

// Eight adjacent columns: the vector width that keeps bf16 rows on 128-bit accesses.
struct F8 { float4 lo, hi; };
__device__ __forceinline__ F8 vfma(float s, F8 v, F8 w) { return {vfma(s, v.lo, w.lo), vfma(s, v.hi, w.hi)}; }
__device__ __forceinline__ F8 vmul(float s, F8 v) { return {vmul(s, v.lo), vmul(s, v.hi)}; }
template <> __device__ __forceinline__ F8 vzero<F8>() { return {vzero<float4>(), vzero<float4>()}; }
template <> __device__ __forceinline__ F8 vload<F8>(const float *p) { return {vload<float4>(p), vload<float4>(p + 4)}; }
template <> __device__ __forceinline__ void vstore<F8>(float *p, F8 v) { vstore<float4>(p, v.lo); vstore<float4>(p + 4, v.hi); }

// bf16 storage: a bf16 is the upper half of the fp32 with the same value, so widening is a shift;
// narrowing rounds to nearest even.
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t bf_pack(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a in the low half
  return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ void vstore(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void vstore(__nv_bfloat16 *p, float4 v) {
  *reinterpret_cast<uint2 *>(p) = make_uint2(bf_pack(v.x, v.y), bf_pack(v.z, v.w));
}
__device__ __forceinline__ void vstore(__nv_bfloat16 *p, F8 v) {
  *reinterpret_cast<uint4 *>(p) = make_uint4(bf_pack(v.lo.x, v.lo.y), bf_pack(v.lo.z, v.lo.w), bf_pack(v.hi.x, v.hi.y), bf_pack(v.hi.z, v.hi.w));
}
__device__ __forceinline__ void vstore(float *p, float v) { *p = v; }
__device__ __forceinline__ void vstore(float *p, float4 v) { vstore<float4>(p, v); }
__device__ __forceinline__ void vstore(float *p, F8 v) { vstore<F8>(p, v); }
template <typename V> struct VecWidth { static constexpr int value = sizeof(V) / sizeof(float); };

// What a row's slice looks like in registers between the load and its use: fp32 storage is kept
// as it is, bf16 storage stays packed (half the registers while the loads are in flight) and is
// widened when consumed.
template <typename V, typename T> struct Raw { using type = V; };
template <> struct Raw<float, __nv_bfloat16> { using type = __nv_bfloat16; };
template <> struct Raw<float4, __nv_bfloat16> { using type = uint2; };
template <> struct Raw<F8, __nv_bfloat16> { using type = uint4; };
template <typename V> __device__ __forceinline__ V widen(V v) { return v; }
template <typename V> __device__ __forceinline__ V widen(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename V> __device__ __forceinline__ V widen(uint2 w) {
  return make_float4(bf_lo(w.x), bf_hi(w.x), bf_lo(w.y), bf_hi(w.y));
}
template <typename V> __device__ __forceinline__ V widen(uint4 w) {
  return {make_float4(bf_lo(w.x), bf_hi(w.x), bf_lo(w.y), bf_hi(w.y)), make_float4(bf_lo(w.z), bf_hi(w.z), bf_lo(w.w), bf_hi(w.w))};
}
template <typename R, typename T> __device__ __forceinline__ R rload(const T *p) { return *reinterpret_cast<const R *>(p); }
template <> __device__ __forceinline__ F8 rload<F8, float>(const float *p) { return vload<F8>(p); }

constexpr int kThreads = 256;

// One row's own terms: own_x = x - gamma e, own_y = y - gamma e, and the message u (one of them).
template <typename V, typename TXY, typename TG, bool HAS_G, bool USE_Y>
struct RowRegs {
  using RXY = typename Raw<V, TXY>::type;
  using RG = typename Raw<V, TG>::type;
  RXY x, y;
  RG g;
  __device__ __forceinline__ void load(const StepArgs &p, int64_t off) {
    x = rload<RXY>(static_cast<const TXY *>(p.X) + off);
    if (USE_Y) y = rload<RXY>(static_cast<const TXY *>(p.Y) + off);
    if (HAS_G) g = rload<RG>(static_cast<const TG *>(p.G) + off);
  }
  __device__ __forceinline__ void own_terms(const StepArgs &p, V &own_x, V &own_y, V &u) const {
    const V xv = widen<V>(x);
    if (HAS_G) {
      const V gv = widen<V>(g);
      own_x = vfma(-p.gamma, gv, xv);
      own_y = USE_Y ? vfma(-p.gamma, gv, widen<V>(y)) : vzero<V>();
    } else {
      own_x = xv;
      own_y = USE_Y ? widen<V>(y) : vzero<V>();
    }
    u = (USE_Y && p.payload) ? own_y : own_x;
  }
};

// RIF = rows whose loads are issued before any of them is consumed (memory-level parallelism per
// thread); MINB = CTAs per SM the register allocation must allow (parallelism across threads).
// Long cycles want a deep RIF, cycles of two rows have only two rows to load and want occupancy.
// YMODE: 1 = Y is read and written; 0 = Y has zero weight this round, it is only written;
//        2 = X only (n a power of two: every round builds its message from x, so X never depends on Y);
//        3 = Y is read but y+ is not stored (last round of a cycle: the next round ignores y).
template <typename V, typename TXY, typename TG, bool HAS_G, int YMODE, int RIF, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) step_walk_kernel(const StepArgs p) {
  constexpr bool USE_Y = (YMODE == 1 || YMODE == 3);
  constexpr bool WRITE_Y = (YMODE == 0 || YMODE == 1);
  constexpr int VW = VecWidth<V>::value;
  TXY *const Xo = static_cast<TXY *>(p.Xo);
  TXY *const Yo = static_cast<TXY *>(p.Yo);
  const int64_t colv = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (colv >= p.ncolv) return;
  const int64_t col = colv * VW;
  using Row = RowRegs<V, TXY, TG, HAS_G, USE_Y>;

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
          vstore(Xo + offs[j], vfma(p.a, own_x, vmul(p.one_minus_a, u_prev)));
          if (WRITE_Y) vstore(Yo + offs[j], vfma(p.b, own_y, vmul(p.one_minus_b, u_prev)));
          u_prev = u;
        }
      }
    }
    if (!first_done) first.own_terms(p, first_own_x, first_own_y, u_prev);  // cycle of one row
    // close the cycle: the first row receives the message of the last one
    vstore(Xo + first_off, vfma(p.a, first_own_x, vmul(p.one_minus_a, u_prev)));
    if (WRITE_Y) vstore(Yo + first_off, vfma(p.b, first_own_y, vmul(p.one_minus_b, u_prev)));
  }
}

// Y_FORMS: bit y = YMODE y may be requested for this shape (the others are not instantiated).
template <typename V, typename TXY, typename TG, int RIF, int MINB, int Y_FORMS, bool ALLOW_NO_G>
static cudaError_t launch_walk_shape(const StepArgs &args, bool has_g, int ymode, cudaStream_t stream) {
  const int64_t blocks_x = (args.ncolv + kThreads - 1) / kThreads;
  if (blocks_x > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  dim3 grid((unsigned)blocks_x, (unsigned)(args.n_cycles < 65535 ? args.n_cycles : 65535));
  bool launched = false;
#define CECA_STEP_LAUNCH(G_, Y_)                                                                       \
  if constexpr (((Y_FORMS >> Y_) & 1) && (G_ || ALLOW_NO_G)) {                                            \
    if (has_g == G_ && ymode == Y_) {                                                                   \
      step_walk_kernel<V, TXY, TG, G_, Y_, RIF, MINB><<<grid, kThreads, 0, stream>>>(args);            \
      launched = true;                                                                                  \
    }                                                                                                   \
  }
  CECA_STEP_LAUNCH(true, 0) CECA_STEP_LAUNCH(true, 1) CECA_STEP_LAUNCH(true, 2) CECA_STEP_LAUNCH(true, 3)
  CECA_STEP_LAUNCH(false, 0) CECA_STEP_LAUNCH(false, 1) CECA_STEP_LAUNCH(false, 2) CECA_STEP_LAUNCH(false, 3)
#undef CECA_STEP_LAUNCH
  return launched ? cudaGetLastError() : cudaErrorInvalidValue;
}

// Launch shapes, chosen from a sweep on a B200 at n = 100, d = 25.6M and n = 24, d = 11.7M:
// cycles of two rows (every CECA-1P round, and the 2-port shift n/2) have nothing to pipeline and
// run fastest with many resident CTAs; long walks want four rows of loads in flight per thread.
// Y_FORMS: which YMODEs the caller may ask for (all four for fp32 storage).
template <typename V, typename TXY, typename TG, int Y_FORMS, bool ALLOW_NO_G>
static cudaError_t launch_walk(const StepArgs &args, bool has_g, int ymode, cudaStream_t stream) {
  if (args.ncolv <= 0) return cudaSuccess;
  constexpr int kReadsY = Y_FORMS & 0b1010, kNoReadY = Y_FORMS & 0b0101;
  if constexpr (VecWidth<V>::value == 8) {
    // eight columns per thread (narrow storage): the same launch shapes, one step less occupancy for short cycles
    // packed bf16 rows need half the registers: one more CTA per SM for the short cycles (measured: +13 % there,
    // while fp32 X and Y lose 15 % with it)
    constexpr int kShortMinb = sizeof(TXY) == 2 ? 4 : 3, kFourMinb = sizeof(TXY) == 2 ? 3 : 2;
    if (args.cycle_len <= 2) return launch_walk_shape<V, TXY, TG, 1, kShortMinb, Y_FORMS, ALLOW_NO_G>(args, has_g, ymode, stream);
    if (args.cycle_len <= 4) return launch_walk_shape<V, TXY, TG, 2, kFourMinb, Y_FORMS, ALLOW_NO_G>(args, has_g, ymode, stream);
    // long walks: four rows in flight when the rows are packed bf16, two when X and Y are fp32 (registers)
    constexpr int kLongRif = sizeof(TXY) == 2 ? 4 : 2;
    return launch_walk_shape<V, TXY, TG, kLongRif, 2, Y_FORMS, ALLOW_NO_G>(args, has_g, ymode, stream);
  } else {
    if (args.cycle_len <= 2)
      return (ymode == 1 || ymode == 3) ? launch_walk_shape<V, TXY, TG, 1, 4, kReadsY, ALLOW_NO_G>(args, has_g, ymode, stream)
                                        : launch_walk_shape<V, TXY, TG, 1, 6, kNoReadY, ALLOW_NO_G>(args, has_g, ymode, stream);
    if (args.cycle_len <= 4) return launch_walk_shape<V, TXY, TG, 2, 3, Y_FORMS, ALLOW_NO_G>(args, has_g, ymode, stream);
    return launch_walk_shape<V, TXY, TG, 4, 2, Y_FORMS, ALLOW_NO_G>(args, has_g, ymode, stream);
  }
}

static inline bool aligned_to(const void *p, size_t bytes) { return (reinterpret_cast<uintptr_t>(p) & (bytes - 1)) == 0; }

// Enqueues one iteration with X, Y stored as TXY and G as TG.  VW columns per thread in the vector
// body (VW elements of either type must make a 64- or 128-bit access), the scalar form for the rest.
// Arguments are assumed validated.  Yo == nullptr: y+ is not stored (the caller has checked that this
// is legal); Y is then still read if the round needs it.
template <typename V, typename TXY, typename TG, int Y_FORMS, bool ALLOW_NO_G>
static cudaError_t enqueue_step_as(const Plan &plan, const TXY *X, const TXY *Y, const TG *G, TXY *Xo, TXY *Yo,
                                   int32_t n, int64_t d, int64_t ld, float gamma, cudaStream_t stream) {
  constexpr int VW = VecWidth<V>::value;
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
  // Vector accesses need every row of every array to start on a VW-element boundary once the first
  // `head` columns are set aside: ld a multiple of VW, and all base pointers off such a boundary by
  // the same number of elements (zero for buffers that come straight from an allocator; the same
  // non-zero amount for, say, views that skip the first k elements of aligned buffers).  The head
  // and the ragged tail (fewer than VW columns each) run the scalar form.
  auto misalign = [](const void *ptr, size_t elem) { return (int64_t)((reinterpret_cast<uintptr_t>(ptr) / elem) % VW); };
  const int64_t mis = misalign(X, sizeof(TXY));
  const bool vec_ok = (ld % VW == 0) && aligned_to(X, sizeof(TXY)) && misalign(Xo, sizeof(TXY)) == mis &&
                      aligned_to(Xo, sizeof(TXY)) && (!Yo || (misalign(Yo, sizeof(TXY)) == mis && aligned_to(Yo, sizeof(TXY)))) &&
                      (!use_y || (misalign(Y, sizeof(TXY)) == mis && aligned_to(Y, sizeof(TXY)))) &&
                      (!has_g || (misalign(G, sizeof(TG)) == mis && aligned_to(G, sizeof(TG))));
  int64_t head = vec_ok ? (VW - mis) % VW : 0;   // scalar columns in front of the vector body
  if (head > d) head = d;
  const int64_t d_vec = vec_ok ? ((d - head) / VW) * VW : 0;  // columns covered by vector accesses
  auto shifted = [&](const StepArgs &from, int64_t c0, int64_t count) {
    StepArgs t = from;
    t.X = X + c0; t.Xo = Xo + c0; t.Yo = Yo ? Yo + c0 : nullptr;
    t.Y = Y ? Y + c0 : nullptr;
    t.G = G ? G + c0 : nullptr;
    t.ncolv = count;
    return t;
  };
  if (d_vec > 0) {
    const StepArgs body = shifted(a, head, d_vec / VW);
    cudaError_t e = launch_walk<V, TXY, TG, Y_FORMS, ALLOW_NO_G>(body, has_g, ymode, stream);
    if (e != cudaSuccess) return e;
  }
  if (d_vec == 0) head = 0;   // no vector body: one scalar launch covers everything
  if (head > 0) {
    const StepArgs t = shifted(a, 0, head);
    cudaError_t e = launch_walk<float, TXY, TG, Y_FORMS, ALLOW_NO_G>(t, has_g, ymode, stream);
    if (e != cudaSuccess) return e;
  }
  if (head + d_vec < d) {  // ragged tail (or everything, when rows cannot be aligned for vector accesses)
    const StepArgs t = shifted(a, head + d_vec, d - head - d_vec);
    cudaError_t e = launch_walk<float, TXY, TG, Y_FORMS, ALLOW_NO_G>(t, has_g, ymode, stream);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t enqueue_step(const Plan &plan, const float *X, const float *Y, const float *G, float *Xo,
                         float *Yo, int32_t n, int64_t d, int64_t ld, float gamma,
                         cudaStream_t stream) {
  return enqueue_step_as<float4, float, float, 0b1111, true>(plan, X, Y, G, Xo, Yo, n, d, ld, gamma, stream);
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

extern "C" ceca_status_t ceca_gossip_sgd_step_bf16(const void *X, const void *Y, const void *G, void *X_out,
                                                   void *Y_out, int32_t n, int64_t d, int64_t ld,
                                                   int32_t xy_bf16, float gamma, ceca_variant_t variant, int64_t k,
                                                   void *stream) {
  ceca_status_t st = ceca::check_matrix_args(X, X_out, n, d, ld);
  if (st != CECA_OK) return st;
  if (!G || !Y_out) return CECA_ERR_INVALID_ARG;   // the gradient is what is stored narrow; no X-only / dead-y forms here
  ceca::Plan plan;
  st = ceca::make_plan(n, variant, k, &plan);
  if (st != CECA_OK) return st;
  if (!Y && plan.reads_y) return CECA_ERR_INVALID_ARG;
  if (X_out == Y_out || X_out == Y || Y_out == X || X_out == G || Y_out == G) return CECA_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __nv_bfloat16 *g = static_cast<const __nv_bfloat16 *>(G);
  cudaError_t e;
  if (xy_bf16)
    e = ceca::enqueue_step_as<ceca::F8, __nv_bfloat16, __nv_bfloat16, 0b0011, false>(
        plan, static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(Y), g,
        static_cast<__nv_bfloat16 *>(X_out), static_cast<__nv_bfloat16 *>(Y_out), n, d, ld, gamma, s);
  else
    e = ceca::enqueue_step_as<ceca::F8, float, __nv_bfloat16, 0b0011, false>(
        plan, static_cast<const float *>(X), static_cast<const float *>(Y), g, static_cast<float *>(X_out),
        static_cast<float *>(Y_out), n, d, ld, gamma, s);
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}
