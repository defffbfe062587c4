// Host-side BCR packer: validates the mask, derives per-block keep lists, builds the canonical
// form and the two private device layouts, uploads them.  No device computation happens here.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <numeric>

#include "grim_internal.h"

using namespace grim;

namespace {

inline float round_bf16(float f) {
  // nearest-even rounding of the low 16 bits (finite inputs)
  uint32_t u;
  std::memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u = (u + 0x7FFFu + lsb) & 0xFFFF0000u;
  float r;
  std::memcpy(&r, &u, 4);
  return r;
}

inline uint16_t bf16_bits(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}

template <typename T>
cudaError_t upload(T** dst, const void* src, size_t bytes) {
  *dst = nullptr;
  size_t alloc = bytes ? bytes : 16;
  cudaError_t e = cudaMalloc((void**)dst, alloc);
  if (e != cudaSuccess) return e;
  if (bytes) e = cudaMemcpy(*dst, src, bytes, cudaMemcpyHostToDevice);
  return e;
}

void free_device(grim_bcr* h) {
  cudaFree(h->d_stage);
  cudaFree(h->d_blob);
  cudaFree(h->d_band_order);
  cudaFree(h->d_gemv_band_ptr);
  cudaFree(h->d_chunks);
  cudaFree(h->d_colwords);
  cudaFree(h->d_gemv_vals);
  cudaFree(h->d_tc_acc);
  cudaFree(h->d_run_ptr);
  cudaFree(h->d_runs);
  cudaFree(h->d_rc_stage);
  cudaFree(h->d_rc_blob);
  cudaFree(h->d_sl_colwords);
  cudaFree(h->d_sl_vals);
  cudaFree(h->d_sl_run_ptr);
  cudaFree(h->d_sl_runs);
  cudaFree(h->d_sl_band_of);
  cudaFree(h->d_sl_slice_of);
  cudaFree(h->d_td_stage);
  cudaFree(h->d_td_blob);
  cudaFree(h->d_status);
}

int bands_per_group(int bh) { return bh <= 4 ? 32 : (bh <= 8 ? 16 : 8); }

}  // namespace

extern "C" grim_status_t grim_bcr_pack(const float* W, int64_t ldw, const uint8_t* mask, int64_t ldm, int64_t M,
                                       int64_t K, int bh, int bw, grim_dtype_t vdt, uint32_t flags,
                                       grim_bcr_t* out) {
  if (!W || !mask || !out) return GRIM_ERR_INVALID_ARG;
  if (M <= 0 || K <= 0 || bh <= 0 || bw <= 0 || ldw < K || ldm < K) return GRIM_ERR_INVALID_ARG;
  if (vdt != GRIM_F32 && vdt != GRIM_BF16) return GRIM_ERR_DTYPE;
  if (flags & ~(GRIM_PACK_REORDER | GRIM_PACK_HOST_ONLY | GRIM_PACK_NARROW_ONLY | GRIM_PACK_WIDE_ONLY)) return GRIM_ERR_INVALID_ARG;
  if ((flags & GRIM_PACK_NARROW_ONLY) && (flags & GRIM_PACK_WIDE_ONLY)) return GRIM_ERR_INVALID_ARG;
  if (bh > 16 || bw > 64 || M >= (int64_t(1) << 31) || K >= (int64_t(1) << 31)) return GRIM_ERR_UNSUPPORTED;

  grim_bcr* h = new (std::nothrow) grim_bcr();
  if (!h) return GRIM_ERR_ALLOC;
  grim_status_t st = GRIM_OK;
  try {
    h->M = M; h->K = K; h->bh = bh; h->bw = bw; h->dtype = (int)vdt; h->flags = flags;
    h->nbr = (M + bh - 1) / bh;
    h->nbc = (K + bw - 1) / bw;
    const int64_t nbr = h->nbr, nbc = h->nbc;
    h->blocks.resize((size_t)(nbr * nbc));

    // ---- a1: per block keep vectors + rank-1 check; a3: compaction in canonical order
    std::vector<uint8_t> col_used((size_t)K, 0);
    std::vector<int64_t> row_nnz((size_t)M, 0);
    uint64_t nnz = 0;
    for (int64_t i = 0; i < nbr; ++i) {
      const int hb = (int)std::min<int64_t>(bh, M - i * bh);
      for (int64_t j = 0; j < nbc; ++j) {
        const int wb = (int)std::min<int64_t>(bw, K - j * bw);
        uint32_t rm = 0;
        uint64_t cm = 0;
        for (int r = 0; r < hb; ++r) {
          const uint8_t* mr = mask + (i * bh + r) * ldm + j * bw;
          for (int c = 0; c < wb; ++c)
            if (mr[c]) { rm |= 1u << r; cm |= 1ull << c; }
        }
        for (int r = 0; r < hb && st == GRIM_OK; ++r) {
          const uint8_t* mr = mask + (i * bh + r) * ldm + j * bw;
          for (int c = 0; c < wb; ++c) {
            const bool want = ((rm >> r) & 1u) && ((cm >> c) & 1ull);
            if ((mr[c] != 0) != want) { st = GRIM_ERR_NOT_BCR; break; }
          }
        }
        if (st != GRIM_OK) break;
        HostBlock& b = h->blocks[(size_t)(i * nbc + j)];
        b.rowmask = rm; b.colmask = cm;
        b.kr = (uint16_t)__builtin_popcount(rm);
        b.kc = (uint16_t)__builtin_popcountll(cm);
        b.val_off = nnz;
        if (b.kr && b.kc) {
          h->nonempty++;
          for (int r = 0; r < hb; ++r) {
            if (!((rm >> r) & 1u)) continue;
            row_nnz[(size_t)(i * bh + r)] += b.kc;
            const float* wr = W + (i * bh + r) * ldw + j * bw;
            for (int c = 0; c < wb; ++c)
              if ((cm >> c) & 1ull) {
                h->vals.push_back(vdt == GRIM_BF16 ? round_bf16(wr[c]) : wr[c]);
                col_used[(size_t)(j * bw + c)] = 1;
              }
          }
          nnz += (uint64_t)b.kr * b.kc;
        }
      }
      if (st != GRIM_OK) break;
    }
    if (st == GRIM_OK && nnz >= (uint64_t(1) << 32)) st = GRIM_ERR_UNSUPPORTED;
    if (st != GRIM_OK) { delete h; return st; }
    h->nnz = (int64_t)nnz;
    h->k_used = std::accumulate(col_used.begin(), col_used.end(), int64_t(0));

    // ---- a2: canonical row permutation (rows by kept-weight count, largest first, stable)
    h->row_perm.resize((size_t)M);
    std::iota(h->row_perm.begin(), h->row_perm.end(), 0);
    if (flags & GRIM_PACK_REORDER)
      std::stable_sort(h->row_perm.begin(), h->row_perm.end(),
                       [&](int32_t a, int32_t b) { return row_nnz[(size_t)a] > row_nnz[(size_t)b]; });

    // ---- a2: band schedule: heavy bands first, so bands of similar work share a thread block
    std::vector<int64_t> band_nnz((size_t)nbr, 0);
    for (int64_t i = 0; i < nbr; ++i)
      for (int64_t j = 0; j < nbc; ++j) {
        const HostBlock& b = h->blocks[(size_t)(i * nbc + j)];
        band_nnz[(size_t)i] += (int64_t)b.kr * b.kc;
      }
    h->band_order.resize((size_t)nbr);
    std::iota(h->band_order.begin(), h->band_order.end(), 0u);
    if (flags & GRIM_PACK_REORDER)
      std::stable_sort(h->band_order.begin(), h->band_order.end(),
                       [&](uint32_t a, uint32_t b) { return band_nnz[a] > band_nnz[b]; });

    // ---- stage layout for the N > 1 kernels
    const int G = bands_per_group(bh);
    h->G = G;
    h->ngroups = (nbr + G - 1) / G;
    const size_t vsz = vdt == GRIM_BF16 ? 2 : 4;
    std::vector<StageEntry> stage((size_t)(h->ngroups * nbc));
    std::vector<uint8_t> blob;
    blob.reserve((size_t)nnz * vsz + (size_t)h->nonempty * 16 + 1024);
    uint32_t max_blob = 0;
    for (int64_t g = 0; g < h->ngroups; ++g) {
      for (int64_t j = 0; j < nbc; ++j) {
        StageEntry& se = stage[(size_t)(g * nbc + j)];
        se.blob_off16 = (uint32_t)(blob.size() / 16);
        se.blob_bytes = 0;
        se.union_colmask = 0;
        BlockDesc descs[32];
        uint32_t voff = 0;
        for (int b = 0; b < G; ++b) {
          const int64_t pos = g * G + b;
          BlockDesc d{0ull, 0u, 0, 0};
          if (pos < nbr) {
            const HostBlock& hb = h->blocks[(size_t)(h->band_order[(size_t)pos] * nbc + j)];
            if (hb.kr && hb.kc) {
              d.colmask = hb.colmask; d.rowmask = (uint16_t)hb.rowmask; d.kc = hb.kc; d.val_off = voff;
              voff += (uint32_t)hb.kr * hb.kc;
              se.union_colmask |= hb.colmask;
            }
          }
          descs[b] = d;
        }
        if (voff == 0) continue;
        if (blob.size() / 16 >= (uint64_t(1) << 32)) { st = GRIM_ERR_UNSUPPORTED; break; }
        const size_t start = blob.size();
        blob.resize(start + (size_t)G * sizeof(BlockDesc));
        std::memcpy(&blob[start], descs, (size_t)G * sizeof(BlockDesc));
        for (int b = 0; b < G; ++b) {
          const int64_t pos = g * G + b;
          if (pos >= nbr) continue;
          const HostBlock& hb = h->blocks[(size_t)(h->band_order[(size_t)pos] * nbc + j)];
          const size_t n = (size_t)hb.kr * hb.kc;
          if (!n) continue;
          const float* src = &h->vals[(size_t)hb.val_off];
          const size_t at = blob.size();
          blob.resize(at + n * vsz);
          if (vdt == GRIM_BF16) {
            for (size_t t = 0; t < n; ++t) { uint16_t v = bf16_bits(src[t]); std::memcpy(&blob[at + 2 * t], &v, 2); }
          } else {
            std::memcpy(&blob[at], src, n * 4);
          }
        }
        blob.resize((blob.size() + 15) / 16 * 16, 0);
        se.blob_bytes = (uint32_t)(blob.size() - start);
        max_blob = std::max(max_blob, se.blob_bytes);
      }
      if (st != GRIM_OK) break;
    }
    if (st != GRIM_OK) { delete h; return st; }
    h->max_blob_bytes = max_blob;
    h->index_bytes_spmm = (int64_t)stage.size() * (int64_t)sizeof(StageEntry) + (int64_t)(blob.size() - (size_t)nnz * vsz) +
                          nbr * 4;

    // ---- chunk layout for the N <= 16 kernels
    // A "virtual band" is a band restricted to block columns [jlo, jhi): the whole band for the matrix-vector product,
    // one K slice of it for 2 <= N <= 16 (see below).  build_narrow lays the chunks and runs of a list of virtual
    // bands out, in list order.
    struct VBand { int64_t pos, jlo, jhi; };
    struct Narrow {
      std::vector<uint32_t> band_ptr;  // per virtual band: first chunk
      std::vector<ChunkDesc> chunks;
      std::vector<uint32_t> colwords;
      std::vector<uint8_t> gvals;
      std::vector<uint32_t> run_ptr;   // per virtual band: first run
      std::vector<RunDesc> runs;
    };
    auto build_narrow = [&](const std::vector<VBand>& vb, Narrow& o) {
      const int64_t nv = (int64_t)vb.size();
      o.band_ptr.assign((size_t)nv + 1, 0);
      o.gvals.reserve((size_t)nnz * vsz);
      std::vector<int64_t> order;
      uint64_t gv_elems = 0;
      for (int64_t v = 0; v < nv; ++v) {
        const int64_t i = h->band_order[(size_t)vb[(size_t)v].pos];
        o.band_ptr[(size_t)v] = (uint32_t)o.chunks.size();
        order.clear();
        for (int64_t j = vb[(size_t)v].jlo; j < vb[(size_t)v].jhi; ++j)
          if (h->blocks[(size_t)(i * nbc + j)].kr && h->blocks[(size_t)(i * nbc + j)].kc) order.push_back(j);
        std::stable_sort(order.begin(), order.end(), [&](int64_t a, int64_t b) {
          return h->blocks[(size_t)(i * nbc + a)].kr > h->blocks[(size_t)(i * nbc + b)].kr;
        });
        size_t t = 0;
        while (t < order.size()) {
          const int kr = h->blocks[(size_t)(i * nbc + order[t])].kr;
          // (block, local column slot) pairs of this run of equal-kr blocks
          std::vector<std::pair<int64_t, int>> cols;
          while (t < order.size() && h->blocks[(size_t)(i * nbc + order[t])].kr == kr) {
            const HostBlock& hb = h->blocks[(size_t)(i * nbc + order[t])];
            for (int b = 0; b < hb.kc; ++b) cols.emplace_back(order[t], b);
            ++t;
          }
          for (size_t c0 = 0; c0 < cols.size(); c0 += 32) {
            const int nc = (int)std::min<size_t>(32, cols.size() - c0);
            ChunkDesc cd;
            cd.val_off = (uint32_t)gv_elems;
            cd.cw_off = (uint32_t)o.colwords.size();
            cd.ncols_kr = (uint32_t)nc | ((uint32_t)kr << 16);
            o.chunks.push_back(cd);
            for (int l = 0; l < nc; ++l) {
              const int64_t j = cols[c0 + l].first;
              const HostBlock& hb = h->blocks[(size_t)(i * nbc + j)];
              // local index of the b-th kept column
              int b = cols[c0 + l].second, c = 0;
              for (uint64_t m = hb.colmask;; ++c)
                if ((m >> c) & 1ull) { if (b-- == 0) break; }
              o.colwords.push_back((uint32_t)(j * bw + c) | (hb.rowmask << 16));
            }
            o.colwords.resize(o.chunks.size() * 32, 0u);  // every chunk owns 32 words; unused slots: no row kept
            for (int sr = 0; sr < kr; ++sr)
              for (int l = 0; l < nc; ++l) {
                const HostBlock& hb = h->blocks[(size_t)(i * nbc + cols[c0 + l].first)];
                const float v = h->vals[(size_t)(hb.val_off + (uint64_t)sr * hb.kc + (uint64_t)cols[c0 + l].second)];
                if (vdt == GRIM_BF16) {
                  uint16_t u = bf16_bits(v);
                  o.gvals.insert(o.gvals.end(), (uint8_t*)&u, (uint8_t*)&u + 2);
                } else {
                  o.gvals.insert(o.gvals.end(), (const uint8_t*)&v, (const uint8_t*)&v + 4);
                }
                ++gv_elems;
              }
          }
        }
      }
      o.gvals.resize(o.gvals.size() + 64 * vsz, 0);  // the kernels may read (and discard) up to a warp's width past a chunk
      o.band_ptr[(size_t)nv] = (uint32_t)o.chunks.size();
      // runs: the transfer units of the streaming kernel
      o.run_ptr.assign((size_t)nv + 1, 0);
      for (int64_t v = 0; v < nv; ++v) {
        o.run_ptr[(size_t)v] = (uint32_t)o.runs.size();
        uint32_t c = o.band_ptr[(size_t)v];
        const uint32_t ce = o.band_ptr[(size_t)v + 1];
        while (c < ce) {
          o.runs.push_back(RunDesc{c, o.chunks[c].val_off});
          size_t bytes = 0;
          int n = 0;
          while (c < ce && n < kRunChunks) {
            const uint32_t nk = o.chunks[c].ncols_kr;
            const size_t cb = (size_t)(nk & 0xFFFFu) * (nk >> 16) * vsz;
            if (n > 0 && bytes + cb > (size_t)kRunValueBytes) break;
            bytes += cb;
            ++n;
            ++c;
          }
        }
      }
      o.run_ptr[(size_t)nv] = (uint32_t)o.runs.size();
      o.runs.push_back(RunDesc{(uint32_t)o.chunks.size(), (uint32_t)gv_elems});
    };
    Narrow nar, sl;  // whole bands; K slices
    std::vector<uint32_t> sl_band_of, sl_slice_of;  // sliced copy: band and slice of every virtual band
    h->gemv_ok = K <= 65536;
    if (h->gemv_ok) {
      std::vector<VBand> vb;
      for (int64_t pos = 0; pos < nbr; ++pos) vb.push_back(VBand{pos, 0, nbc});
      build_narrow(vb, nar);
      h->nruns = (int64_t)nar.runs.size() - 1;
      h->nchunks = (int64_t)nar.chunks.size();
      h->h_gemv_band_ptr = nar.band_ptr;
      h->h_chunks = nar.chunks;
      h->n_colwords = (int64_t)nar.colwords.size();
      // what the streaming kernel reads besides the values: column words, the run table, the band tables
      h->index_bytes_gemv = (int64_t)nar.colwords.size() * 4 + (int64_t)nar.runs.size() * (int64_t)sizeof(RunDesc) +
                            (nbr + 1) * 4 + nbr * 4;
      // K slices for 2 <= N <= 16: a thread block stages the slice's rows of X in shared memory once and multiplies the
      // slice's part of many bands from there (Section 4.4: a needed input row is loaded once), instead of gathering
      // them from L2 for every band.  A second copy of the values in slice-major order; only built when K has more
      // than one slice (otherwise the whole-band layout is its own single slice).
      const int64_t spb = std::max<int64_t>(1, kSliceRows / bw);  // block columns per slice
      h->sl_rows = (int)(spb * bw);
      h->sl_nslices = (nbc + spb - 1) / spb;
      if (h->sl_nslices > 1 && !(flags & GRIM_PACK_WIDE_ONLY)) {
        std::vector<VBand> vs;
        for (int64_t sidx = 0; sidx < h->sl_nslices; ++sidx)
          for (int64_t pos = 0; pos < nbr; ++pos) {
            vs.push_back(VBand{pos, sidx * spb, std::min<int64_t>((sidx + 1) * spb, nbc)});
            sl_band_of.push_back(h->band_order[(size_t)pos]);
            sl_slice_of.push_back((uint32_t)sidx);
          }
        build_narrow(vs, sl);
        h->sl_nruns = (int64_t)sl.runs.size() - 1;
        h->index_bytes_sliced = (int64_t)sl.colwords.size() * 4 + (int64_t)sl.runs.size() * (int64_t)sizeof(RunDesc) +
                                ((int64_t)vs.size() + 1) * 4 + (int64_t)vs.size() * 8;
      }
    }

    // ---- row-chunk layout for the register-tiled and tensor-core kernels
    std::vector<RcStage> rc_stage;
    std::vector<uint8_t> rc_blob;
    {
      h->rc_groups = (nbr + kRcBands - 1) / kRcBands;
      rc_stage.resize((size_t)(h->rc_groups * nbc));
      rc_blob.reserve((size_t)nnz * 5 + (size_t)h->nonempty * 32 + 1024);
      uint32_t rc_max = 0;
      for (int64_t g = 0; g < h->rc_groups && st == GRIM_OK; ++g) {
        for (int64_t j = 0; j < nbc; ++j) {
          RcStage& se = rc_stage[(size_t)(g * nbc + j)];
          se.off16 = (uint32_t)(rc_blob.size() / 16);
          se.bytes = 0;
          bool any = false;
          for (int b = 0; b < kRcBands && !any; ++b) {
            const int64_t pos = g * kRcBands + b;
            if (pos >= nbr) break;
            const HostBlock& hb = h->blocks[(size_t)(h->band_order[(size_t)pos] * nbc + j)];
            any = hb.kr && hb.kc;
          }
          if (!any) continue;
          if (rc_blob.size() / 16 >= (uint64_t(1) << 32)) { st = GRIM_ERR_UNSUPPORTED; break; }
          const size_t start = rc_blob.size();
          rc_blob.resize(start + kRcBands * 4, 0);
          for (int b = 0; b < kRcBands; ++b) {
            const int64_t pos = g * kRcBands + b;
            if (pos >= nbr) break;
            const HostBlock& hb = h->blocks[(size_t)(h->band_order[(size_t)pos] * nbc + j)];
            if (!(hb.kr && hb.kc)) continue;
            const int kr = hb.kr, kc = hb.kc, nch = (kc + kRcChunk - 1) / kRcChunk;
            const size_t rec = rc_blob.size();
            const uint32_t hdr = (uint32_t)((rec - start) / 16) | ((uint32_t)kr << 16) | ((uint32_t)nch << 24);
            std::memcpy(&rc_blob[start + (size_t)b * 4], &hdr, 4);
            const size_t idx_bytes = ((size_t)8 + (size_t)nch * kRcChunk + 15) / 16 * 16;
            rc_blob.resize(rec + idx_bytes + (size_t)nch * kr * kRcChunk * 4, 0);
            const uint64_t rows = (uint64_t)hb.rowmask | ((uint64_t)kc << 32);  // low word: bit r = row r kept; high word: kc
            std::memcpy(&rc_blob[rec], &rows, 8);
            uint8_t cols[64];
            int n = 0;
            for (int c = 0; c < 64; ++c)
              if ((hb.colmask >> c) & 1ull) cols[n++] = (uint8_t)c;
            for (int c = 0; c < nch * kRcChunk; ++c) rc_blob[rec + 8 + (size_t)c] = cols[c < kc ? c : 0];
            float* w = reinterpret_cast<float*>(&rc_blob[rec + idx_bytes]);
            const float* src = &h->vals[(size_t)hb.val_off];
            for (int c = 0; c < kc; ++c)
              for (int aa = 0; aa < kr; ++aa)
                w[((size_t)(c / kRcChunk) * kr + aa) * kRcChunk + (c % kRcChunk)] = src[(size_t)aa * kc + c];
          }
          se.bytes = (uint32_t)(rc_blob.size() - start);
          rc_max = std::max(rc_max, se.bytes);
        }
      }
      if (st != GRIM_OK) { delete h; return st; }
      h->rc_max_blob = rc_max;
      h->index_bytes_rc = (int64_t)rc_stage.size() * (int64_t)sizeof(RcStage) + (int64_t)rc_blob.size() - (int64_t)nnz * 4 +
                          nbr * 4;
    }

    // ---- tensor-core tiling (bf16 handles whose block shape tiles 128 x 64 evenly)
    const bool tc_shape = vdt == GRIM_BF16 && (bh == 4 || bh == 8 || bh == 16) && (bw == 16 || bw == 32 || bw == 64);
    if (tc_shape) {
      h->tc_mtiles = (nbr + kTcRows / bh - 1) / (kTcRows / bh);
      h->tc_ktiles = (nbc + kTcK / bw - 1) / (kTcK / bw);
    }

    // ---- scatter layout of the tensor-core kernels (same shapes and tiles as above): per tile the kept values, each
    // with the byte offset of its place in the expanded, swizzled 128 x 64 tile
    std::vector<RcStage> td_stage;
    std::vector<uint8_t> td_blob;
    if (tc_shape) {
      const int S = kTcRows / bh, J = kTcK / bw;
      td_stage.resize((size_t)(h->tc_mtiles * h->tc_ktiles));
      uint32_t td_max = 0;
      std::vector<uint32_t> ent;
      for (int64_t t = 0; t < h->tc_mtiles && st == GRIM_OK; ++t)
        for (int64_t kt = 0; kt < h->tc_ktiles; ++kt) {
          ent.clear();
          for (int ts = 0; ts < S; ++ts) {
            const int64_t pos = t * S + ts;
            if (pos >= nbr) break;
            for (int jj = 0; jj < J; ++jj) {
              const int64_t j = kt * J + jj;
              if (j >= nbc) break;
              const HostBlock& hb = h->blocks[(size_t)(h->band_order[(size_t)pos] * nbc + j)];
              if (!(hb.kr && hb.kc)) continue;
              size_t v = (size_t)hb.val_off;
              for (int r = 0; r < bh; ++r) {
                if (!((hb.rowmask >> r) & 1u)) continue;
                const uint32_t row = (uint32_t)(ts * bh + r);
                for (int c = 0; c < bw; ++c) {
                  if (!((hb.colmask >> c) & 1ull)) continue;
                  const uint32_t col = (uint32_t)(jj * bw + c);
                  ent.push_back((uint32_t)bf16_bits(h->vals[v++]) | (td_offset(row, col) << 16));
                }
              }
            }
          }
          RcStage& se = td_stage[(size_t)(t * h->tc_ktiles + kt)];
          se.off16 = (uint32_t)(td_blob.size() / 16);
          se.bytes = 0;
          if (ent.empty()) continue;
          if (td_blob.size() / 16 >= (uint64_t(1) << 32)) { st = GRIM_ERR_UNSUPPORTED; break; }
          while (ent.size() % 4) ent.push_back(ent.back());  // whole 16-byte vectors; a repeated entry writes the same value again
          // Order for conflict-free stores: a thread reads four consecutive entries and the 32 lanes of a warp store
          // their k-th entry together, so entries 4 * lane + k of a run of 128 should fall into 32 different
          // shared-memory banks.  Entries are dealt from per-bank piles in turn (32 consecutive picks hit 32 banks
          // while all piles last) and pick i of a run goes to lane i % 32, store i / 32.
          {
            std::vector<uint32_t> pile[32];
            for (uint32_t e : ent) pile[((e >> 16) >> 2) & 31u].push_back(e);
            std::vector<uint32_t> dealt;
            dealt.reserve(ent.size());
            for (size_t r = 0; dealt.size() < ent.size(); ++r)
              for (int b = 0; b < 32; ++b)
                if (pile[b].size() > r) dealt.push_back(pile[b][r]);
            for (size_t base = 0; base < ent.size(); base += 128) {
              const size_t n = std::min<size_t>(128, ent.size() - base);  // a multiple of 4
              const size_t lanes = n / 4;                                   // lanes that read a whole vector of this run
              for (size_t i = 0; i < n; ++i) ent[base + 4 * (i % lanes) + i / lanes] = dealt[base + i];
            }
          }
          const size_t start = td_blob.size();
          td_blob.resize(start + ent.size() * 4);
          std::memcpy(&td_blob[start], ent.data(), ent.size() * 4);
          se.bytes = (uint32_t)(ent.size() * 4);
          td_max = std::max(td_max, se.bytes);
        }
      if (st != GRIM_OK) { delete h; return st; }
      h->td_max_rec = td_max;
      h->index_bytes_tc = (int64_t)td_stage.size() * (int64_t)sizeof(RcStage) + (int64_t)td_blob.size() - (int64_t)nnz * 2 + nbr * 4;
    }

    // ---- upload
    if (!(flags & GRIM_PACK_HOST_ONLY)) {
      cudaError_t e = cudaGetDevice(&h->device);
      // a handle packed for one regime keeps only that regime's layouts in device memory
      const bool wide = !(flags & GRIM_PACK_NARROW_ONLY), narrow = !(flags & GRIM_PACK_WIDE_ONLY);
      if (e == cudaSuccess && wide) e = upload(&h->d_stage, stage.data(), stage.size() * sizeof(StageEntry));
      if (e == cudaSuccess && wide) e = upload(&h->d_blob, blob.data(), blob.size());
      if (e == cudaSuccess) e = upload(&h->d_band_order, h->band_order.data(), h->band_order.size() * 4);
      if (e == cudaSuccess && wide) e = upload(&h->d_rc_stage, rc_stage.data(), rc_stage.size() * sizeof(RcStage));
      if (e == cudaSuccess && wide) e = upload(&h->d_rc_blob, rc_blob.data(), rc_blob.size());
      if (e == cudaSuccess && tc_shape && wide) {
        e = upload(&h->d_td_stage, td_stage.data(), td_stage.size() * sizeof(RcStage));
        if (e == cudaSuccess) e = upload(&h->d_td_blob, td_blob.data(), td_blob.size());
      }
      const unsigned zero = 0;
      if (e == cudaSuccess) e = upload(&h->d_status, &zero, 4);
      if (e == cudaSuccess && h->gemv_ok && narrow) {
        e = upload(&h->d_gemv_band_ptr, nar.band_ptr.data(), nar.band_ptr.size() * 4);
        if (e == cudaSuccess) e = upload(&h->d_chunks, nar.chunks.data(), nar.chunks.size() * sizeof(ChunkDesc));
        if (e == cudaSuccess) e = upload(&h->d_colwords, nar.colwords.data(), nar.colwords.size() * 4);
        if (e == cudaSuccess) e = upload((uint8_t**)&h->d_gemv_vals, nar.gvals.data(), nar.gvals.size());
        if (e == cudaSuccess) e = upload(&h->d_run_ptr, nar.run_ptr.data(), nar.run_ptr.size() * 4);
        if (e == cudaSuccess) e = upload(&h->d_runs, nar.runs.data(), nar.runs.size() * sizeof(RunDesc));
        if (e == cudaSuccess && !sl.runs.empty()) {
          e = upload(&h->d_sl_colwords, sl.colwords.data(), sl.colwords.size() * 4);
          if (e == cudaSuccess) e = upload((uint8_t**)&h->d_sl_vals, sl.gvals.data(), sl.gvals.size());
          if (e == cudaSuccess) e = upload(&h->d_sl_run_ptr, sl.run_ptr.data(), sl.run_ptr.size() * 4);
          if (e == cudaSuccess) e = upload(&h->d_sl_runs, sl.runs.data(), sl.runs.size() * sizeof(RunDesc));
          if (e == cudaSuccess) e = upload(&h->d_sl_band_of, sl_band_of.data(), sl_band_of.size() * 4);
          if (e == cudaSuccess) e = upload(&h->d_sl_slice_of, sl_slice_of.data(), sl_slice_of.size() * 4);
        }
      }
      if (e != cudaSuccess) {
        st = (e == cudaErrorMemoryAllocation) ? GRIM_ERR_ALLOC : GRIM_ERR_CUDA;
        cudaGetLastError();
        free_device(h);
        delete h;
        return st;
      }
    }
  } catch (const std::bad_alloc&) {
    free_device(h);
    delete h;
    return GRIM_ERR_ALLOC;
  }
  *out = h;
  return GRIM_OK;
}

extern "C" grim_status_t grim_bcr_destroy(grim_bcr_t h) {
  if (!h) return GRIM_OK;
  if (h->device >= 0) {
    int cur = -1;
    cudaGetDevice(&cur);
    if (cur != h->device) cudaSetDevice(h->device);
    free_device(h);
    if (cur != h->device && cur >= 0) cudaSetDevice(cur);
  }
  delete h;
  return GRIM_OK;
}

static int64_t export_size(const grim_bcr* h) {
  int64_t lists = 0;
  for (const HostBlock& b : h->blocks) lists += 4 + 2 * (int64_t)(b.kr && b.kc ? b.kr + b.kc : 0);
  return 64 + lists + h->nnz * (h->dtype == GRIM_BF16 ? 2 : 4) + 4 * h->M;
}

extern "C" grim_status_t grim_bcr_info(grim_bcr_t h, grim_bcr_info_t* info) {
  if (!h || !info) return GRIM_ERR_INVALID_ARG;
  std::memset(info, 0, sizeof(*info));
  info->M = h->M; info->K = h->K; info->bh = h->bh; info->bw = h->bw; info->nbr = h->nbr; info->nbc = h->nbc;
  info->nnz = h->nnz; info->nonempty_blocks = h->nonempty; info->k_used = h->k_used; info->dtype = h->dtype;
  info->flags = h->flags; info->on_device = h->device >= 0;
  info->value_bytes = h->nnz * (h->dtype == GRIM_BF16 ? 2 : 4);
  info->index_bytes_spmm = h->index_bytes_rc;
  info->index_bytes_gemv = h->index_bytes_gemv;
  info->export_bytes = export_size(h);
  info->index_bytes_tc = h->index_bytes_tc;
  return GRIM_OK;
}

extern "C" grim_status_t grim_bcr_export(grim_bcr_t h, void* buf, int64_t capacity, int64_t* written) {
  if (!h || !buf) return GRIM_ERR_INVALID_ARG;
  const int64_t need = export_size(h);
  if (capacity < need) return GRIM_ERR_INVALID_ARG;
  uint8_t* p = (uint8_t*)buf;
  int64_t magic = 0;  // the eight characters as a little-endian integer
  const char* tag = "GRIMBCR1";
  for (int i = 7; i >= 0; --i) magic = (magic << 8) | (uint8_t)tag[i];
  const int64_t hdr[8] = {magic, h->M, h->K, h->bh, h->bw, h->nbr, h->nbc, h->dtype};
  std::memcpy(p, hdr, 64);
  p += 64;
  for (const HostBlock& b : h->blocks) {
    const bool live = b.kr && b.kc;
    const uint16_t krkc[2] = {(uint16_t)(live ? b.kr : 0), (uint16_t)(live ? b.kc : 0)};
    std::memcpy(p, krkc, 4);
    p += 4;
    if (!live) continue;
    for (int r = 0; r < 16; ++r)
      if ((b.rowmask >> r) & 1u) { uint16_t v = (uint16_t)r; std::memcpy(p, &v, 2); p += 2; }
    for (int c = 0; c < 64; ++c)
      if ((b.colmask >> c) & 1ull) { uint16_t v = (uint16_t)c; std::memcpy(p, &v, 2); p += 2; }
    const size_t n = (size_t)b.kr * b.kc;
    const float* src = &h->vals[(size_t)b.val_off];
    if (h->dtype == GRIM_BF16) {
      for (size_t t = 0; t < n; ++t) { uint16_t v = bf16_bits(src[t]); std::memcpy(p, &v, 2); p += 2; }
    } else {
      std::memcpy(p, src, n * 4);
      p += n * 4;
    }
  }
  std::memcpy(p, h->row_perm.data(), (size_t)h->M * 4);
  p += h->M * 4;
  if (written) *written = (int64_t)(p - (uint8_t*)buf);
  return (p - (uint8_t*)buf) == need ? GRIM_OK : GRIM_ERR_INVALID_ARG;
}

extern "C" grim_status_t grim_bcr_unpack_dense(grim_bcr_t h, float* W, int64_t ldw) {
  if (!h || !W || ldw < h->K) return GRIM_ERR_INVALID_ARG;
  for (int64_t r = 0; r < h->M; ++r) std::memset(W + r * ldw, 0, (size_t)h->K * 4);
  for (int64_t i = 0; i < h->nbr; ++i)
    for (int64_t j = 0; j < h->nbc; ++j) {
      const HostBlock& b = h->blocks[(size_t)(i * h->nbc + j)];
      if (!(b.kr && b.kc)) continue;
      const float* src = &h->vals[(size_t)b.val_off];
      for (int r = 0; r < 16; ++r) {
        if (!((b.rowmask >> r) & 1u)) continue;
        for (int c = 0; c < 64; ++c)
          if ((b.colmask >> c) & 1ull) W[(i * h->bh + r) * ldw + j * h->bw + c] = *src++;
      }
    }
  return GRIM_OK;
}

extern "C" grim_status_t grim_bcr_status(grim_bcr_t h) {
  if (!h || h->device < 0 || !h->d_status) return GRIM_ERR_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return GRIM_ERR_CUDA;
  unsigned v = 0;
  if (cudaMemcpy(&v, h->d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return GRIM_ERR_CUDA;
  if (v != 0) cudaMemset(h->d_status, 0, 4);
  return (grim_status_t)(v & 0xFFu);  // the upper bits say which wait gave up (a debugging aid of the kernels)
}
