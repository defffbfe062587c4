// Internal definitions shared by the host packer and the CUDA translation units of libgrim.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "grim.h"

namespace grim {

// ---------------------------------------------------------------------------------------------
// Device layout for the N > 1 kernels ("stage" layout).
//
// Row bands (block rows) are taken in schedule order and cut into groups of G bands; one thread
// block owns one group.  For group g and block column j the G block descriptors and the kept
// values of those blocks are stored back to back ("blob"), so that a thread block streams one
// contiguous piece of memory per block column (the compact, reordered storage idea of
// Sections 4.2 - 4.3 laid out for a CTA instead of a CPU thread).
// ---------------------------------------------------------------------------------------------
struct __align__(16) BlockDesc {
  unsigned long long colmask;  // bit c set: block-local column c kept (bw <= 64)
  uint32_t val_off;            // first value of this block, in elements from the blob's value area
  uint16_t rowmask;            // bit r set: block-local row r kept (bh <= 16)
  uint16_t kc;                 // popcount(colmask)
};

struct __align__(16) StageEntry {
  uint32_t blob_off16;               // blob start, in 16-byte units from the blob base
  uint32_t blob_bytes;               // multiple of 16; 0 when no block of the group keeps anything here
  unsigned long long union_colmask;  // columns kept by at least one of the G blocks
};

// ---------------------------------------------------------------------------------------------
// Device layout for the N = 1 kernel ("chunk" layout).
//
// Per band the kept columns of all its blocks are concatenated after sorting the blocks by
// kept-row count, and cut into chunks of at most 32 columns that all have the same kept-row count kr.
// Lane l of a warp owns column l of a chunk.  A column word is (global column | rowmask << 16).
// Every chunk owns 32 column words (chunk c starts at word 32 * c; unused slots are 0, i.e. "no
// row kept"), so that a warp can fetch the words without reading the descriptor first.
// The chunk's values are stored step-major: value s of lane l is at val_off + s * ncols + l.
// ---------------------------------------------------------------------------------------------
struct ChunkDesc {
  uint32_t val_off;
  uint32_t cw_off;
  uint32_t ncols_kr;  // ncols | kr << 16
};
// The streaming kernel moves the chunk layout in "runs": up to kRunChunks consecutive chunks of one band whose
// values take at most kRunValueBytes (no single chunk is larger: 16 rows x 32 columns x 4 bytes is half of it).  Run r covers chunks [runs[r].c0, runs[r + 1].c0) and values [runs[r].v0, runs[r + 1].v0); the
// table ends with a sentinel.  run_ptr[pos] .. run_ptr[pos + 1] are the runs of the band at schedule position pos.
constexpr int kSliceRows = 1024;  // rows of X per K slice of the sliced copy (see grim_bcr::sl_*)
constexpr int kRunChunks = 4;
constexpr int kRunValueBytes = 4096;
struct RunDesc {
  uint32_t c0;  // first chunk
  uint32_t v0;  // first value, in elements
};

// ---------------------------------------------------------------------------------------------
// Device layout for the register-tiled N > 16 kernel and the tensor-core kernel ("row-chunk"
// layout).  Bands in schedule order are cut into groups of kRcBands; for group g and block column
// j one contiguous blob:
//   u32 hdr[kRcBands]     per band slot: record offset in 16-byte units | kr << 16 | nch << 24
//   per band with kr > 0, 16-byte aligned:
//     u32 rowmask, u32 kc bit r of rowmask set: block-local row r kept (kept rows are numbered a = 0.. ascending)
//     u8  cols[nch * 8]   block-local kept columns, padded to a multiple of 8 by repeating the
//                         first kept column (its padded weights are 0); then padding to 16 bytes
//     f32 w[nch][kr][8]   w[c][a][e] = weight of kept row a and column cols[c * 8 + e]
// Values are always fp32 here (bf16 handles store the rounded values widened to fp32).
// ---------------------------------------------------------------------------------------------
constexpr int kRcBands = 16;
constexpr int kRcChunk = 8;
struct RcStage {
  uint32_t off16;  // blob start in 16-byte units from the blob base
  uint32_t bytes;  // multiple of 16; 0 when no band of the group keeps anything in this block column
};

// ---------------------------------------------------------------------------------------------
// Tiling of the tensor-core kernels (bf16 handles with bh in {4, 8, 16}, bw in {16, 32, 64}): the matrix is cut into
// tiles of kTcRows rows (consecutive bands in schedule order) x kTcK columns, one record per tile.
// ---------------------------------------------------------------------------------------------
constexpr int kTcRows = 128;
constexpr int kTcK = 64;

// ---------------------------------------------------------------------------------------------
// Scatter layout of the tensor-core kernels: a record is the list of the tile's kept values as
// 32-bit entries: bf16 value (low half) | byte offset of the element in the expanded tile (high half), the tile being
// K-major with rows of 128 bytes whose 16-byte pieces are XOR-ed with the row's low three bits (the tensor core's
// 128-byte swizzle).  Entries are in canonical order (band, block column, kept row, kept column) and padded to a
// multiple of four by repeating the last one.  Expanding a tile is then: clear it, and per entry one 2-byte store
// - no index arithmetic on the device.  The price is 2 index bytes per value.
// ---------------------------------------------------------------------------------------------
inline uint32_t td_offset(uint32_t row, uint32_t col) {
  return row * 128u + ((((col >> 3) ^ (row & 7u))) << 4) + (col & 7u) * 2u;
}

struct HostBlock {
  uint64_t colmask = 0;
  uint32_t rowmask = 0;
  uint16_t kr = 0, kc = 0;
  uint64_t val_off = 0;  // into grim_bcr::vals (canonical order)
};

}  // namespace grim

struct grim_bcr {
  int64_t M = 0, K = 0;
  int bh = 0, bw = 0;
  int64_t nbr = 0, nbc = 0;
  int dtype = 0;
  uint32_t flags = 0;
  int64_t nnz = 0, nonempty = 0, k_used = 0;
  // host-side canonical data
  std::vector<grim::HostBlock> blocks;  // nbr * nbc, row-major
  std::vector<float> vals;              // kept values, canonical order (bf16 handles: already rounded)
  std::vector<int32_t> row_perm;        // canonical row permutation
  std::vector<uint32_t> band_order;     // schedule position -> band
  // stage layout
  int G = 0;  // bands per group
  int64_t ngroups = 0;
  uint32_t max_blob_bytes = 0;
  int64_t index_bytes_spmm = 0, index_bytes_gemv = 0;
  bool gemv_ok = false;
  int64_t nchunks = 0;
  std::vector<uint32_t> h_gemv_band_ptr;   // host copies of the chunk tables (sizing of on-chip weight residency)
  std::vector<grim::ChunkDesc> h_chunks;
  int64_t n_colwords = 0;
  // row-chunk layout
  int64_t rc_groups = 0;
  uint32_t rc_max_blob = 0;
  int64_t index_bytes_rc = 0;
  // device
  int device = -1;
  grim::RcStage* d_rc_stage = nullptr;
  uint8_t* d_rc_blob = nullptr;
  // tensor-core layout
  int64_t tc_mtiles = 0, tc_ktiles = 0;
  int64_t index_bytes_tc = 0;
  uint32_t td_max_rec = 0;
  grim::RcStage* d_td_stage = nullptr;
  uint8_t* d_td_blob = nullptr;
  float* d_tc_acc = nullptr;  // fp32 scratch of the split tensor-core multiply (M x N); grim_bcr_reserve allocates it
  size_t tc_acc_bytes = 0;
  // answers of grim_bcr_tune, one per (log2 bucket of N, X dtype, Y dtype); path 0 = not tuned
  grim_tune_t tuned[32][2][2] = {};
  unsigned* d_status = nullptr;  // error word written by kernels whose bounded waits ran out
  grim::StageEntry* d_stage = nullptr;
  uint8_t* d_blob = nullptr;
  uint32_t* d_band_order = nullptr;
  uint32_t* d_gemv_band_ptr = nullptr;
  grim::ChunkDesc* d_chunks = nullptr;
  uint32_t* d_colwords = nullptr;
  void* d_gemv_vals = nullptr;
  uint32_t* d_run_ptr = nullptr;
  grim::RunDesc* d_runs = nullptr;
  int64_t nruns = 0;
  // K-sliced copy of the chunk layout for 2 <= N <= 16 (absent when K has a single slice): virtual band v = slice *
  // nbr + schedule position; per virtual band its runs, its band and its slice
  int sl_rows = 0;          // rows of X per slice (a multiple of bw)
  int64_t sl_nslices = 0, sl_nruns = 0, index_bytes_sliced = 0;
  uint32_t* d_sl_colwords = nullptr;
  void* d_sl_vals = nullptr;
  uint32_t* d_sl_run_ptr = nullptr;
  grim::RunDesc* d_sl_runs = nullptr;
  uint32_t* d_sl_band_of = nullptr;
  uint32_t* d_sl_slice_of = nullptr;
  // dense bf16 copy for the tensor-core path is decompressed on the fly; nothing stored here
};

namespace grim {

// epilogue / addressing description handed to the N > 1 kernel
struct SpmmArgs {
  const void* X = nullptr;  // activations
  void* Y = nullptr;
  int64_t ncols = 0;        // GEMM N
  int64_t x_sk = 0, x_sq = 1;  // X(k, q) at k * x_sk + q * x_sq (elements)
  int64_t y_sr = 0, y_sq = 1;  // Y(r, q) at r * y_sr + q * y_sq
  int x_dtype = 0, y_dtype = 0;
  const float* bias = nullptr;  // per output row, or null
  int relu = 0;
  // implicit im2col (conv != 0): q = (img, oh, ow); k = (c, kh, kw)
  int conv = 0;
  int C = 0, H = 0, W = 0, KH = 0, KW = 0, stride = 1, pad = 0, OH = 0, OW = 0;
  int tile_n = 0;  // 0 = default
  int y_prefilled = 0;  // Y already holds the bias in every column: a split multiply adds onto it (no clearing, no
                        // bias pass; not with relu); an unsplit multiply ignores the flag
};

grim_status_t launch_spmm(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s);
constexpr int kSkinnyMaxN = 16;  // widest right-hand side taken by the lane-per-column kernel
grim_status_t launch_skinny(const grim_bcr* h, const void* X, int x_dtype, int64_t ldx, int64_t N, void* Y, int y_dtype,
                            int64_t ldy, cudaStream_t s);
// same product through per-warp rings filled by bulk asynchronous copies (persistent thread blocks)
grim_status_t launch_stream(const grim_bcr* h, const void* X, int x_dtype, int64_t ldx, int64_t N, void* Y, int y_dtype,
                            int64_t ldy, cudaStream_t s);
bool stream_path_supported(const grim_bcr* h, int64_t N);
grim_status_t launch_ffma(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s);
bool ffma_path_supported(const grim_bcr* h, const SpmmArgs& a);
grim_status_t launch_spmm_tc(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s);
bool tc_path_supported(const grim_bcr* h, const SpmmArgs& a);
// the paired (two thread blocks per tile pair) tensor-core kernel: matrices, bf16 handles
grim_status_t launch_spmm_tc2(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s);
bool tc2_path_supported(const grim_bcr* h, const SpmmArgs& a);
void count_launch(int n = 1);
// streaming multiprocessors of a device (read once per device through the runtime)
int sm_count(int device);
// raises a kernel's dynamic shared-memory limit to `bytes` unless an earlier call already did (the attribute is
// kept by the kernel, so it is set once per kernel and size, not per launch)
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);

// Launch with programmatic stream serialization: the kernel may begin while the launch before it in the stream still
// runs; it calls griddepcontrol.wait before it touches anything but the packed matrix and its own shared memory.
template <typename K, typename... A>
cudaError_t launch_pdl(K kern, dim3 grid, dim3 block, size_t smem, cudaStream_t s, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

}  // namespace grim
