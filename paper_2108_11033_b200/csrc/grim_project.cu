// Projection of a dense matrix onto the BCR-sparse set (Section 5.2, Eq. (4): the Z-step of the ADMM pruning needs
// the member of S_i - matrices whose zeros form whole rows and whole columns of blocks, with at least a given share of
// zeros - that is nearest to W + U in the Frobenius norm).  The exact projection is a combinatorial problem and the
// paper gives no algorithm; this is a deterministic greedy one that is exact for 1 x 1 blocks (magnitude pruning):
//
//   all rows and columns of all blocks start kept; a "line" is one row or one column of one block; its cost is the
//   mean square of its entries that are still kept.  Repeatedly the line of smallest cost (ties: smallest line id =
//   block * (bh + bw) + (row, or bh + column)) is removed, until at most (1 - sparsity) * M * K entries are kept.
//
// Costs are recomputed from scratch in double precision, in index order, whenever a crossing line goes, so that any
// implementation of these steps takes the same decisions bit for bit.  Host only.
#include <cmath>
#include <queue>
#include <vector>

#include "grim_internal.h"

namespace {

struct Line {
  double cost;
  int64_t id;
  uint32_t version;
};
struct Worse {
  bool operator()(const Line& a, const Line& b) const { return a.cost != b.cost ? a.cost > b.cost : a.id > b.id; }
};

}  // namespace

extern "C" grim_status_t grim_bcr_project(const float* V, int64_t ldv, int64_t M, int64_t K, int bh, int bw, double sparsity,
                                          uint8_t* mask, int64_t ldm, int64_t* kept_out) {
  if (!V || !mask || M <= 0 || K <= 0 || ldv < K || ldm < K || bh < 1 || bw < 1) return GRIM_ERR_INVALID_ARG;
  if (!(sparsity >= 0.0 && sparsity <= 1.0)) return GRIM_ERR_INVALID_ARG;
  if (bh > 16 || bw > 64) return GRIM_ERR_UNSUPPORTED;
  try {
    const int64_t nbr = (M + bh - 1) / bh, nbc = (K + bw - 1) / bw, L = bh + bw;
    const int64_t budget = (int64_t)std::floor((1.0 - sparsity) * (double)M * (double)K + 1e-9);
    std::vector<uint16_t> rowkeep((size_t)(nbr * nbc)), krs((size_t)(nbr * nbc));
    std::vector<uint64_t> colkeep((size_t)(nbr * nbc));
    std::vector<uint32_t> version((size_t)(nbr * nbc * L), 0);
    int64_t kept = M * K;
    // cost of line l of block (i, j) over the entries still kept; false when the line has none
    auto line_cost = [&](int64_t i, int64_t j, int l, double* cost) {
      const int64_t b = i * nbc + j;
      const int rows = (int)std::min<int64_t>(bh, M - i * bh), cols = (int)std::min<int64_t>(bw, K - j * bw);
      double sum = 0.0;
      int n = 0;
      if (l < bh) {
        if (l >= rows || !((rowkeep[(size_t)b] >> l) & 1u)) return false;
        for (int c = 0; c < cols; ++c)
          if ((colkeep[(size_t)b] >> c) & 1ull) { const double v = V[(i * bh + l) * ldv + j * bw + c]; sum += v * v; ++n; }
      } else {
        const int c = l - bh;
        if (c >= cols || !((colkeep[(size_t)b] >> c) & 1ull)) return false;
        for (int r = 0; r < rows; ++r)
          if ((rowkeep[(size_t)b] >> r) & 1u) { const double v = V[(i * bh + r) * ldv + j * bw + c]; sum += v * v; ++n; }
      }
      if (n == 0) return false;
      *cost = sum / n;
      return true;
    };
    std::priority_queue<Line, std::vector<Line>, Worse> heap;
    for (int64_t i = 0; i < nbr; ++i)
      for (int64_t j = 0; j < nbc; ++j) {
        const int rows = (int)std::min<int64_t>(bh, M - i * bh), cols = (int)std::min<int64_t>(bw, K - j * bw);
        rowkeep[(size_t)(i * nbc + j)] = (uint16_t)((1u << rows) - 1u);
        colkeep[(size_t)(i * nbc + j)] = cols == 64 ? ~0ull : ((1ull << cols) - 1ull);
        for (int l = 0; l < L; ++l) {
          double c;
          if (line_cost(i, j, l, &c)) heap.push(Line{c, (i * nbc + j) * L + l, 0u});
        }
      }
    while (kept > budget && !heap.empty()) {
      const Line t = heap.top();
      heap.pop();
      if (t.version != version[(size_t)t.id]) continue;  // superseded by a later cost of the same line
      const int64_t b = t.id / L, i = b / nbc, j = b % nbc;
      const int l = (int)(t.id % L);
      const int kr = __builtin_popcount(rowkeep[(size_t)b]), kc = __builtin_popcountll(colkeep[(size_t)b]);
      if (l < bh) { rowkeep[(size_t)b] &= (uint16_t)~(1u << l); kept -= kc; }
      else { colkeep[(size_t)b] &= ~(1ull << (l - bh)); kept -= kr; }
      ++version[(size_t)t.id];
      // the crossing lines of the block lost an entry: new costs
      const int lo = l < bh ? bh : 0, hi = l < bh ? (int)L : bh;
      for (int x = lo; x < hi; ++x) {
        const int64_t id = b * L + x;
        double c;
        ++version[(size_t)id];
        if (line_cost(i, j, x, &c)) heap.push(Line{c, id, version[(size_t)id]});
      }
    }
    for (int64_t r = 0; r < M; ++r)
      for (int64_t c = 0; c < K; ++c) {
        const int64_t b = (r / bh) * nbc + c / bw;
        mask[r * ldm + c] = (uint8_t)(((rowkeep[(size_t)b] >> (r % bh)) & 1u) && ((colkeep[(size_t)b] >> (c % bw)) & 1ull));
      }
    if (kept_out) *kept_out = kept;
    return GRIM_OK;
  } catch (const std::bad_alloc&) {
    return GRIM_ERR_ALLOC;
  }
}
