// Instantiations of the register-tile filtering kernel for the damped update
// (a translation unit of their own: see tile3_filter.cuh).
#include "tile3_filter.cuh"

int bi_tile3_filter_damped(const Tile3Params &p, int arith, int na, int nb, int nc, cudaStream_t stream) {
  return arith == BI_ARITH_F64 ? tile3_filter::dispatch_filter<double, true>(p, na, nb, nc, stream)
                               : tile3_filter::dispatch_filter<float, true>(p, na, nb, nc, stream);
}
