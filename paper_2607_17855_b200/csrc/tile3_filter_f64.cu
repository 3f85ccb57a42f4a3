// Instantiations of the float64 register-tile filtering kernel (tile3_filter_f64.cuh) for the compiled
// tile shapes that give every lane of a unit one state of the first axis.
#include "tile3_filter_f64.cuh"

namespace {

template <int NA, int NB, int NC>
int launch(const Tile3Params &p, cudaStream_t stream) {
  using G = tile3_f64::Geo<NA, NB, NC>;
  const int grid = (p.N + G::UPW - 1) / G::UPW;
  // (an agent whose logits lie far below another's of the same warp carries small numerators under a
  // common shift, and the product of its three normalisers must stay a normal number: with probabilities
  // in A a logit is at least (modalities + 1) ln 1e-16, i.e. 53.2 (modalities + 1) binary orders below
  // zero, and three times that must stay under 1022: the kernel shifts per agent beyond five modalities)
  if (p.lambda != 1.0) tile3_f64::bi_tile3_filter_f64_kernel<NA, NB, NC, true><<<grid, 32, 0, stream>>>(p);
  else tile3_f64::bi_tile3_filter_f64_kernel<NA, NB, NC, false><<<grid, 32, 0, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? BI_OK : BI_ERR_CUDA;
}

}  // namespace

// BI_ERR_UNSUPPORTED when the shape has no instantiation here (the caller falls back to the general
// register-tile kernel)
int bi_tile3_filter_f64(const Tile3Params &p, int na, int nb, int nc, cudaStream_t stream) {
#define X(A, B, C, S, LS)                                                                     \
  if constexpr (S == 1 && B <= Pow2Ceil<A>::v && C <= Pow2Ceil<A>::v) {                       \
    if (na == A && nb == B && nc == C) return launch<A, B, C>(p, stream);                     \
  }
  BI_TILE3_SHAPES(X)
#undef X
  return BI_ERR_UNSUPPORTED;
}
