// Register-tile kernels for single-group rank-3 models (every modality depends
// on the same three factors and the model has exactly those factors).
// Filtering: a few lanes per agent, the step recursion and the iteration loop
// inside one launch, the summed slice of the current step held in registers.
#include <cstdlib>
#include "bi_internal.h"
#include "tile3.cuh"
#include "tile3_common.cuh"
#include "tile3_filter.cuh"

// (the damped update's instantiations live in tile3_damped.cu)
int bi_tile3_filter_damped(const Tile3Params &p, int arith, int na, int nb, int nc, cudaStream_t stream);
// (the float64 kernel of the plain update, for the tile shapes it covers, in tile3_filter_f64.cu)
int bi_tile3_filter_f64(const Tile3Params &p, int na, int nb, int nc, cudaStream_t stream);


int bi_tile3_shape(int na, int nb, int nc) {
#define X(A, B, C, S, LS) \
  if (na == A && nb == B && nc == C) return S;
  BI_TILE3_SHAPES(X)
#undef X
  return 0;
}

// Applicable when the model is one dependency group over exactly its three
// factors and a compiled tile shape matches; BI_ERR_UNSUPPORTED otherwise.
int bi_launch_tile3(const BiCall &c, bi_model *mut) {
  const bi_model *md = c.model;
  const BiDev &h = md->h;
  if (c.algo != BI_ALGO_FILTER) return BI_ERR_UNSUPPORTED;
  if (md->tile_sb <= 0) return BI_ERR_UNSUPPORTED;
  const BiGroup &g = h.grp[0];
  Tile3Params p;
  bi_tile3_fill_params(c, p);
  int rc;
  if (p.lambda != 1.0) {
    rc = md->arith == BI_ARITH_F64 ? bi_tile3_filter_f64(p, g.dim[0], g.dim[1], g.dim[2], c.stream) : BI_ERR_UNSUPPORTED;
    if (rc == BI_ERR_UNSUPPORTED) rc = bi_tile3_filter_damped(p, md->arith, g.dim[0], g.dim[1], g.dim[2], c.stream);
  } else if (md->arith == BI_ARITH_F64) {
    rc = bi_tile3_filter_f64(p, g.dim[0], g.dim[1], g.dim[2], c.stream);
    if (rc == BI_ERR_UNSUPPORTED) rc = tile3_filter::dispatch_filter<double, false>(p, g.dim[0], g.dim[1], g.dim[2], c.stream);
  } else
    rc = tile3_filter::dispatch_filter<float, false>(p, g.dim[0], g.dim[1], g.dim[2], c.stream);
  if (rc == BI_OK) {
    mut->launches += 1;
    mut->last_kernel = md->arith == BI_ARITH_F64 ? "tile3_filter_f64" : "tile3_filter_f32";
  }
  return rc;
}
