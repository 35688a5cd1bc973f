// The weight-streaming schedule of the tensor-core GEMM: which (tile, k-block) pieces a CTA works on, in which
// order.  It depends on the problem shape and the grid only, never on the number of tokens, which is what makes a
// token's result independent of the block it is verified in.
#pragma once

#include <cuda.h>

namespace ws {

constexpr int TILE_N = 128;       // weight rows per tile (MMA M)
constexpr int BLOCK_K = 64;       // bf16 elements per k-block: one 128-byte swizzle row

struct Span {  // one piece of a CTA's work: k-blocks [kb0, kb1) of `tile`
  int tile, kb0, kb1, n_contrib, slot, first_owner;
};

// Work of one CTA.  The last R = tiles mod grid tiles are cut stream-K fashion into equal contiguous spans of
// the (tile, k-block) space and come first, so that their partial sums are added up while the whole tiles
// (tile c, c + grid, ...) that follow are still streaming.  Depends on (tiles, kb, grid) only.
struct SpanWalker {
  int kb, per, t0, it, end, whole, grid, cta;
  __device__ SpanWalker(int tiles, int kb_, int grid_, int cta_) {
    kb = kb_;
    grid = grid_;
    cta = cta_;
    t0 = (tiles / grid) * grid;                              // tiles [0, t0) are handled whole
    int total = (tiles - t0) * kb;
    per = (total + grid - 1) / grid;
    it = min(total, cta * per);
    end = min(total, it + per);
    whole = cta;
  }
  __device__ int owner_slot(int tile, int owner) const { return ((tile - t0) * kb <= owner * per) ? 0 : 1; }
  __device__ bool next(Span &s) {
    if (it < end) {
      int rel = it / kb;
      s.tile = t0 + rel;
      s.kb0 = it - rel * kb;
      s.kb1 = min(kb, s.kb0 + (end - it));
      s.first_owner = (rel * kb) / per;
      s.n_contrib = (rel * kb + kb - 1) / per - s.first_owner + 1;
      s.slot = owner_slot(s.tile, cta);                      // first or last piece of this CTA
      it += s.kb1 - s.kb0;
      return true;
    }
    if (whole < t0) {
      s.tile = whole;
      s.kb0 = 0;
      s.kb1 = kb;
      s.n_contrib = 1;
      s.slot = 0;
      s.first_owner = cta;
      whole += grid;
      return true;
    }
    return false;
  }
};

}  // namespace ws
