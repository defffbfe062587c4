// BCRC export (Section 4.3, "Compact Model Storage"): the paper's own storage format, produced from a packed handle
// on the host.  Rows are reordered so that rows with the same column list sit together; a column list shared by
// several rows is stored once.  Six arrays:
//   reorder[p]        original row placed at position p of the reordered matrix
//   row_offset[p]     first weight of reordered row p in `weights` (M + 1 entries)
//   occurrence[g]     first reordered row of group g, a run of rows that share one column list (G + 1 entries)
//   column_stride[g]  first entry of group g's column list in `compact_column` (G + 1 entries)
//   compact_column    the distinct column lists, ascending column ids, one after the other
//   weights           the kept weights row by row of the reordered matrix, ascending column order
// The paper leaves the reorder's tie-breaks open; here rows are sorted by kept-weight count (largest first), then by
// column list (lexicographically), then by row id, which puts equal lists next to each other and is reproducible.
#include <algorithm>
#include <cstring>
#include <numeric>
#include <vector>

#include "grim_internal.h"

using namespace grim;

extern "C" grim_status_t grim_bcr_export_bcrc(grim_bcr_t h, int32_t* reorder, int64_t* row_offset, int32_t* occurrence,
                                              int64_t* column_stride, int32_t* compact_column, float* weights,
                                              grim_bcrc_sizes_t* sizes) {
  if (!h || !sizes) return GRIM_ERR_INVALID_ARG;
  try {
    const int64_t M = h->M;
    // column list and weights of every original row
    std::vector<std::vector<int32_t>> cols((size_t)M);
    std::vector<std::vector<float>> vals((size_t)M);
    for (int64_t i = 0; i < h->nbr; ++i)
      for (int64_t j = 0; j < h->nbc; ++j) {
        const HostBlock& b = h->blocks[(size_t)(i * h->nbc + j)];
        if (!(b.kr && b.kc)) continue;
        const float* src = &h->vals[(size_t)b.val_off];
        for (int r = 0; r < 16; ++r) {
          if (!((b.rowmask >> r) & 1u)) continue;
          const size_t row = (size_t)(i * h->bh + r);
          for (int c = 0; c < 64; ++c)
            if ((b.colmask >> c) & 1ull) {
              cols[row].push_back((int32_t)(j * h->bw + c));
              vals[row].push_back(*src++);
            }
        }
      }
    std::vector<int32_t> order((size_t)M);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int32_t x, int32_t y) {
      if (cols[(size_t)x].size() != cols[(size_t)y].size()) return cols[(size_t)x].size() > cols[(size_t)y].size();
      if (cols[(size_t)x] != cols[(size_t)y]) return cols[(size_t)x] < cols[(size_t)y];
      return x < y;
    });
    int64_t groups = 0, ncompact = 0;
    for (int64_t p = 0; p < M; ++p)
      if (p == 0 || cols[(size_t)order[(size_t)p]] != cols[(size_t)order[(size_t)p - 1]]) {
        ++groups;
        ncompact += (int64_t)cols[(size_t)order[(size_t)p]].size();
      }
    sizes->M = M; sizes->K = h->K; sizes->nnz = h->nnz; sizes->groups = groups; sizes->compact_columns = ncompact;
    if (!reorder && !row_offset && !occurrence && !column_stride && !compact_column && !weights) return GRIM_OK;  // size query
    if (!reorder || !row_offset || !occurrence || !column_stride || !compact_column || !weights) return GRIM_ERR_INVALID_ARG;
    int64_t w = 0, g = 0, cc = 0;
    for (int64_t p = 0; p < M; ++p) {
      const size_t row = (size_t)order[(size_t)p];
      reorder[p] = (int32_t)row;
      row_offset[p] = w;
      if (p == 0 || cols[row] != cols[(size_t)order[(size_t)p - 1]]) {
        occurrence[g] = (int32_t)p;
        column_stride[g] = cc;
        if (!cols[row].empty()) std::memcpy(compact_column + cc, cols[row].data(), cols[row].size() * 4);
        cc += (int64_t)cols[row].size();
        ++g;
      }
      if (!vals[row].empty()) std::memcpy(weights + w, vals[row].data(), vals[row].size() * 4);
      w += (int64_t)vals[row].size();
    }
    row_offset[M] = w;
    occurrence[g] = (int32_t)M;
    column_stride[g] = cc;
    return GRIM_OK;
  } catch (const std::bad_alloc&) {
    return GRIM_ERR_ALLOC;
  }
}
