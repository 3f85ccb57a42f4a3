// Register-tile contraction core for models whose modalities all depend on the
// same three factors (one dependency group of rank 3).
//
// A "unit" is one agent at one time step.  LPU = NAP * SB lanes of a warp work
// on one unit (NAP = NA rounded up to a power of two).  The group's summed
// slice L[a][b][c] (packed order: a slowest, c fastest and padded to NCP) lives
// in registers: lane (a, bh) holds the NBL = NB / SB values b of its half and
// all c.  One Jacobi sweep of the three likelihood messages (Section IV,
// marginalisation) then needs
//   V[b]    = sum_c L[a][b][c] e_c[c]                       in-lane
//   ell_a   = sum_b V[b] e_b[b]                             in-lane (+ SB lanes)
//   ell_b   = sum_a e_a V[b]                                reduce-scatter over the a lanes
//   ell_c   = sum_a e_a sum_b e_b[b] L[a][b][c]             reduce-scatter over all lanes
// about 2 P multiply-adds for P = NA*NB*NC.  Beliefs are carried unnormalised
// (e = exp(x - max), z = sum e) and the three messages are rescaled by
// 1/(z z) afterwards, so one reciprocal per sweep replaces the divisions.
#pragma once
#include "bi_device.cuh"

template <int X> struct Pow2Ceil { static constexpr int v = X <= 1 ? 1 : 2 * Pow2Ceil<(X + 1) / 2>::v; };
template <> struct Pow2Ceil<1> { static constexpr int v = 1; };
template <int X> struct Log2 { static constexpr int v = 1 + Log2<X / 2>::v; };
template <> struct Log2<1> { static constexpr int v = 0; };

// an empty statement the optimiser cannot see through: x stays a value in a register
__device__ __forceinline__ void bi_opaque(float &x) { asm("" : "+f"(x)); }
__device__ __forceinline__ void bi_opaque(double &x) { asm("" : "+d"(x)); }

// Sum v[i] over the NL lanes {lane ^ (k * STR)}; afterwards v[0] holds the
// total of element (sub >> (log2 NL - log2 PV)), where sub is the lane's index
// within the NL lanes.  PV and NL are powers of two, PV <= NL.
template <typename R, int PV, int NL, int STR>
__device__ __forceinline__ R reduce_scatter(R (&v)[PV], int sub) {
  static_assert(PV <= NL, "more values than lanes");
  if (NL == 1) return v[0];
#pragma unroll
  for (int d = NL / 2, cur = PV; d >= 1; d >>= 1) {
    const bool up = (sub & d) != 0;
    if (cur > 1) {
      const int half = cur / 2;
#pragma unroll
      for (int i = 0; i < half; ++i) {
        // (both values are read first and made opaque: a conditional between two array elements can
        // compile to a load through a selected address, which puts the whole array in local memory)
        R lo = v[i], hi = v[i + half];
        bi_opaque(lo);
        bi_opaque(hi);
        const R send = up ? lo : hi;
        const R keep = up ? hi : lo;
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, d * STR);
      }
      cur = half;
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], d * STR);
    }
  }
  return v[0];
}

template <typename R, int NL, int STR>
__device__ __forceinline__ R group_sum(R v) {
#pragma unroll
  for (int d = NL / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d * STR);
  return v;
}
// max over the group, taken in float: any common shift close to the maximum
// makes the softmax exact, so float precision is enough for it
template <int NL, int STR>
__device__ __forceinline__ float group_max_f(float v) {
#pragma unroll
  for (int d = NL / 2; d >= 1; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d * STR));
  return v;
}
// exact argmax over the group: largest x, lowest index among equals
template <typename R, int NL, int STR>
__device__ __forceinline__ int group_argmax(R x, int idx) {
#pragma unroll
  for (int d = NL / 2; d >= 1; d >>= 1) {
    R xo = __shfl_xor_sync(0xffffffffu, x, d * STR);
    int io = __shfl_xor_sync(0xffffffffu, idx, d * STR);
    if (xo > x || (xo == x && io < idx)) { x = xo; idx = io; }
  }
  return idx;
}

__device__ __forceinline__ void ldg_vec(const float *p, float (&x)[4]) {
  float4 v = __ldg(reinterpret_cast<const float4 *>(p));
  x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
}
__device__ __forceinline__ void ldg_vec(const double *p, double (&x)[2]) {
  double2 v = __ldg(reinterpret_cast<const double2 *>(p));
  x[0] = v.x; x[1] = v.y;
}

__device__ __forceinline__ void lds_vec(const float *p, float (&x)[4]) {
  float4 v = *reinterpret_cast<const float4 *>(p);
  x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
}
__device__ __forceinline__ void lds_vec(const double *p, double (&x)[2]) {
  double2 v = *reinterpret_cast<const double2 *>(p);
  x[0] = v.x; x[1] = v.y;
}

// pairwise sum of a register array (short dependency chain)
template <typename R, int N>
__device__ __forceinline__ R tree_sum(const R (&v)[N]) {
  R t[N];
#pragma unroll
  for (int i = 0; i < N; ++i) t[i] = v[i];
#pragma unroll
  for (int w = 1; w < N; w *= 2)
#pragma unroll
    for (int i = 0; i + w < N; i += 2 * w) t[i] += t[i + w];
  return t[0];
}

// reciprocal: hardware seed refined to working precision
__device__ __forceinline__ float bi_rcp(float x) { return 1.0f / x; }
__device__ __forceinline__ double bi_rcp(double x) {
  // x is a product of sums of exponentials, each in [1, 32]: a normal number.
  // Hardware seed (about 20 bits) and two Newton steps reach full precision.
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
  double e = fma(-x, y, 1.0);
  y = fma(y, e, y);
  e = fma(-x, y, 1.0);
  return fma(y, e, y);
}

template <typename R, int NA_, int NB_, int NC_, int SB_>
struct Tile3 {
  static constexpr int NA = NA_, NB = NB_, NC = NC_, SB = SB_;
  static constexpr int NAP = Pow2Ceil<NA>::v;
  static constexpr int LPU = NAP * SB;          // lanes per unit
  static constexpr int UPW = 32 / LPU;          // units per warp
  static constexpr int NBL = NB / SB;           // b values per lane
  static constexpr int NCP = (NC + 3) & ~3;     // padded c
  static constexpr int PB = Pow2Ceil<NBL>::v;   // reduce-scatter widths
  static constexpr int PC = Pow2Ceil<NCP>::v;
  static constexpr int SHB = Log2<NAP>::v - Log2<PB>::v;  // duplicate bits of the b owner index
  static constexpr int SHC = Log2<LPU>::v - Log2<PC>::v;
  static_assert(NB % SB == 0, "SB must divide NB");
  static_assert(LPU <= 32 && PB <= NAP && PC <= LPU, "tile does not fit a warp");

  // With one lane per a (SB == 1) the cross-lane sums of the b and c messages
  // go through a small shared-memory transpose instead of shuffles: lane u
  // stores its partials as row u, then reads column u.  Fewer instructions
  // than the butterfly (no selects), and lane u simply owns b = u and c = u.
  static constexpr bool TP = SB == 1 && NB <= LPU && NC <= LPU;
  static constexpr int TP_T = NBL + NCP;
  // row stride: even, = 2 mod 4 elements, so 16-byte row stores of 8 consecutive lanes hit distinct banks
  static constexpr int TPR = (TP_T % 4 <= 2) ? TP_T - TP_T % 4 + 2 : TP_T + 3;
  static constexpr int TP_UNIT = LPU * TPR + 8;  // elements per unit (8 extra: units of a half-warp on different banks)

  // lane coordinates
  int u, a, bh;       // lane within unit, a index, b half
  int bi, ci;         // owned b (global index) and c
  bool a_ok, b_ok, c_ok;        // the owned a / b / c index is a real state
  bool own_a, own_b, own_c;     // designated writer of x_a / x_b / x_c (duplicates exist when SB > 1)
  R *tp;              // this unit's transpose area (TP only)

  R L[NBL][NCP];      // this lane's part of the summed slice
  R ea, eb[NBL], ec[NCP];  // unnormalised beliefs this lane contracts with
  R sa, sb, sc;       // message scales 1/(z_b z_c), 1/(z_a z_c), 1/(z_a z_b)

  __device__ __forceinline__ void init_lane(int lane) {
    u = lane % LPU;
    a = u / SB;
    bh = u % SB;
    a_ok = a < NA;
    own_a = a_ok && bh == 0;
    tp = nullptr;
    if (TP) {
      bi = u; ci = u;
      own_b = b_ok = u < NB;
      own_c = c_ok = u < NC;
    } else {
      const int ib = a >> SHB;
      bi = bh * NBL + ib;
      ci = u >> SHC;
      b_ok = ib < NBL;
      c_ok = ci < NC;
      own_b = b_ok && (a & ((1 << SHB) - 1)) == 0;
      own_c = c_ok && (u & ((1 << SHC) - 1)) == 0;
    }
  }

  // L[b][c] = sum over the group's modalities of their observed slices.  The
  // slices are stored lane-interleaved (16-byte vector v of lane u at
  // (v * LPU + u) * VE), so each load instruction of a unit reads LPU * 16
  // contiguous bytes.
  static constexpr int VE = 16 / (int)sizeof(R);
  static constexpr int NV = NBL * NCP / VE;
  static constexpr int P_TILE = NAP * NB * NCP;
  __device__ __forceinline__ void load_slices(const R *const *slice, int nmem) {
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl)
#pragma unroll
      for (int c = 0; c < NCP; ++c) L[bl][c] = (R)0;
    for (int mi = 0; mi < nmem; ++mi) {
      const R *p = slice[mi] + u * VE;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        R x[VE];
        ldg_vec(p + v * LPU * VE, x);
#pragma unroll
        for (int i = 0; i < VE; ++i) L[(v * VE + i) / NCP][(v * VE + i) % NCP] += x[i];
      }
    }
  }

  // the same gather, summed into shared memory (same lane-interleaved layout)
  __device__ __forceinline__ void load_slices_smem(const R *const *slice, int nmem, R *Lt) {
    R acc[NV][VE];
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
      for (int i = 0; i < VE; ++i) acc[v][i] = (R)0;
    for (int mi = 0; mi < nmem; ++mi) {
      const R *p = slice[mi] + u * VE;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        R x[VE];
        ldg_vec(p + v * LPU * VE, x);
#pragma unroll
        for (int i = 0; i < VE; ++i) acc[v][i] += x[i];
      }
    }
    __syncwarp();
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
      for (int i = 0; i < VE; ++i) Lt[(v * LPU + u) * VE + i] = acc[v][i];
    __syncwarp();
  }

  __device__ __forceinline__ void set_uniform() {
    ea = a_ok ? (R)1 : (R)0;
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl) eb[bl] = (R)1;
#pragma unroll
    for (int c = 0; c < NCP; ++c) ec[c] = c < NC ? (R)1 : (R)0;
    sa = (R)1 / (R)(NB * NC);
    sb = (R)1 / (R)(NA * NC);
    sc = (R)1 / (R)(NA * NB);
  }

  // the three likelihood messages for the logits this lane owns
  __device__ __forceinline__ void messages(R &xa, R &xb, R &xc, const R *eav = nullptr) {
    // V[b] = sum_c L[b][c] e_c[c] and W[c] = sum_b e_b[b] L[b][c]: independent
    // accumulators advance together so no multiply-add waits on the previous one
    R V[NBL], W[NCP];
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl) V[bl] = (R)0;
#pragma unroll
    for (int c = 0; c < NCP; ++c) W[c] = (R)0;
#pragma unroll
    for (int c = 0; c < NCP; ++c)
#pragma unroll
      for (int bl = 0; bl < NBL; ++bl) V[bl] = fma(L[bl][c], ec[c], V[bl]);
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl)
#pragma unroll
      for (int c = 0; c < NCP; ++c) W[c] = fma(eb[bl], L[bl][c], W[c]);
    finish(V, W, xa, xb, xc, eav);
  }

  // the same with the slice read from shared memory (lane-interleaved layout)
  // instead of registers: for kernels that keep many steps' slices on chip
  __device__ __forceinline__ void messages_smem(const R *__restrict__ Ls, R &xa, R &xb, R &xc, const R *eav = nullptr) {
    // V[b] is accumulated in VE interleaved partial sums: consecutive elements
    // of a row would otherwise form one chain of dependent multiply-adds
    R V[NBL], W[NCP], Vp[NBL][VE];
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl)
#pragma unroll
      for (int i = 0; i < VE; ++i) Vp[bl][i] = (R)0;
#pragma unroll
    for (int c = 0; c < NCP; ++c) W[c] = (R)0;
    const R *p = Ls + u * VE;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      R x[VE];
      lds_vec(p + v * LPU * VE, x);
#pragma unroll
      for (int i = 0; i < VE; ++i) {
        const int bl = (v * VE + i) / NCP, c = (v * VE + i) % NCP;
        Vp[bl][i] = fma(x[i], ec[c], Vp[bl][i]);
        W[c] = fma(eb[bl], x[i], W[c]);
      }
    }
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl) V[bl] = tree_sum<R, VE>(Vp[bl]);
    finish(V, W, xa, xb, xc, eav);
  }

  // eav: with the transpose area in use, every lane's copy of all e_a of its
  // unit (the cross-lane sums are then dot products with it); unused otherwise
  __device__ __forceinline__ void finish(R (&V)[NBL], R (&W)[NCP], R &xa, R &xb, R &xc, const R *eav = nullptr) {
    R la0 = (R)0, la1 = (R)0;
#pragma unroll
    for (int bl = 0; bl < NBL; ++bl) {
      if (bl & 1) la1 = fma(V[bl], eb[bl], la1);
      else la0 = fma(V[bl], eb[bl], la0);
    }
    R la = group_sum<R, SB, 1>(la0 + la1);
    R lb, lc;
    if (TP) {
      R *row = tp + u * TPR;
      const bool dot = eav != nullptr;   // known at compile time once inlined
      const R wa = dot ? (R)1 : ea;      // without the copies the rows are scaled by this lane's e_a
#pragma unroll
      for (int bl = 0; bl < NBL; ++bl) row[bl] = dot ? V[bl] : wa * V[bl];
#pragma unroll
      for (int c = 0; c < NCP; ++c) row[NBL + c] = dot ? W[c] : wa * W[c];
      __syncwarp();
      R b0 = (R)0, b1 = (R)0, c0 = (R)0, c1 = (R)0;
#pragma unroll
      for (int r = 0; r < NAP; ++r) {
        const R vb = tp[r * TPR + (b_ok ? u : 0)], vc = tp[r * TPR + NBL + (c_ok ? u : 0)];
        const R w = dot ? eav[r] : (R)1;
        if (r & 1) { b1 = fma(w, vb, b1); c1 = fma(w, vc, c1); }
        else { b0 = fma(w, vb, b0); c0 = fma(w, vc, c0); }
      }
      lb = b0 + b1;
      lc = c0 + c1;
      __syncwarp();
    } else {
      R pb[PB], pc[PC];
#pragma unroll
      for (int i = 0; i < PB; ++i) pb[i] = i < NBL ? ea * V[i < NBL ? i : 0] : (R)0;
#pragma unroll
      for (int c = 0; c < PC; ++c) pc[c] = c < NCP ? ea * W[c < NCP ? c : 0] : (R)0;
      lb = reduce_scatter<R, PB, NAP, SB>(pb, a);
      lc = reduce_scatter<R, PC, LPU, 1>(pc, u);
    }
    xa = la * sa;
    xb = lb * sb;
    xc = lc * sc;
  }
};
