/*
 * grim.h - C ABI of libgrim: multiply a Block-based Column-Row (BCR) pruned weight matrix by
 * dense activations on one NVIDIA B200 (sm_100a).
 *
 * Background (paper sections are cited per entry point):
 *   - Section 3.2 defines BCR pruning: the weight matrix W (M x K) is tiled into equal blocks of
 *     bh rows x bw columns; inside every block whole rows and whole columns are removed
 *     independently, and what remains of a block is a full kr x kc sub-matrix.
 *   - Section 3.1 treats every CNN / RNN layer as W times an input matrix (GEMM) or vector (GEMV).
 *   - Sections 4.2 - 4.5 describe the execution-side ideas this library re-derives for sm_100a:
 *     row reorder / grouping, a compact storage that shares index lists inside a block, loading
 *     every needed input row once and reusing it for all kept rows of a block, tiling with
 *     tuned tile shapes, and convolution as an (implicit) im2col GEMM that skips pruned columns.
 *
 * Conventions
 *   - Every function returns a grim_status_t; nothing aborts or throws across this boundary.
 *     On failure output handles / buffers are left untouched unless stated otherwise.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global memory of the
 *     current device.  Handles own the device and host buffers they create; activations, outputs,
 *     biases passed at call time stay owned by the caller.
 *   - Compute calls are asynchronous on the given CUDA stream and do not synchronise.  A handle
 *     must not be used by two streams at the same time (the GRU handle owns scratch buffers).
 *   - There is no CPU fallback: compute calls need a CUDA device and fail with GRIM_ERR_CUDA
 *     otherwise.
 *   - Matrices are row-major.  Block shapes are rows x columns.
 */
#ifndef GRIM_H_
#define GRIM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GRIM_OK = 0,
  GRIM_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad flag */
  GRIM_ERR_SHAPE = 2,       /* operand shapes do not match the handle */
  GRIM_ERR_DTYPE = 3,       /* operand dtype does not match the handle */
  GRIM_ERR_NOT_BCR = 4,     /* some block's mask is not (kept rows) x (kept columns) */
  GRIM_ERR_ALLOC = 5,       /* host or device allocation failed */
  GRIM_ERR_CUDA = 6,        /* a CUDA runtime call failed (no device, launch error, ...) */
  GRIM_ERR_UNSUPPORTED = 7, /* valid request outside the implemented range */
  GRIM_ERR_TIMEOUT = 8      /* a bounded device-side wait gave up; results are invalid */
} grim_status_t;

typedef enum { GRIM_F32 = 0, GRIM_BF16 = 1 } grim_dtype_t;

/* Same object as cudaStream_t (NULL = the legacy default stream). */
typedef struct CUstream_st* grim_stream_t;

typedef struct grim_bcr* grim_bcr_t; /* a packed BCR weight matrix */
typedef struct grim_gru* grim_gru_t; /* a multi-layer GRU built from packed matrices */

/* A dense row-major matrix in DEVICE memory: element (r, c) is at ptr[r * ld + c]. */
typedef struct {
  void* ptr;
  int64_t rows, cols, ld;
  grim_dtype_t dtype;
} grim_mat_t;

/* grim_bcr_pack flags */
#define GRIM_PACK_REORDER 1u   /* schedule row bands by decreasing work; export the row permutation */
#define GRIM_PACK_HOST_ONLY 2u /* build host-side data only (no CUDA call); compute calls then fail */
/* A handle normally uploads one private device layout per kernel regime (3 - 4 x the compact size in device memory).
 * A handle that will only see narrow right-hand sides (N <= 16, GRU matrices) or only wide ones can say so and keep
 * just that regime's layouts; a multiply outside the regime then returns GRIM_ERR_UNSUPPORTED. */
#define GRIM_PACK_NARROW_ONLY 4u
#define GRIM_PACK_WIDE_ONLY 8u

typedef struct {
  int64_t M, K;
  int32_t bh, bw;
  int64_t nbr, nbc;         /* block grid: ceil(M/bh) x ceil(K/bw) */
  int64_t nnz;              /* kept weights = sum over blocks of kr*kc (mask count) */
  int64_t nonempty_blocks;
  int64_t k_used;           /* columns of W kept by at least one block (input rows actually read) */
  int32_t dtype;            /* grim_dtype_t of the stored values */
  uint32_t flags;
  int32_t on_device;        /* 0 for GRIM_PACK_HOST_ONLY handles */
  int32_t reserved;
  int64_t value_bytes;      /* nnz * sizeof(value) */
  int64_t index_bytes_spmm; /* bytes of headers / column lists / padding read by the register-tiled N > 16 kernel */
  int64_t index_bytes_gemv; /* bytes of column words / chunk tables read by the N <= 16 kernel */
  int64_t export_bytes;     /* size of the canonical byte string written by grim_bcr_export */
  int64_t index_bytes_tc;   /* bytes of column words / tables read by the tensor-core kernel (0: layout not built) */
} grim_bcr_info_t;

/* Tile-shape choice for the N > 1 kernel (Section 4.5: tile sizes are tuned per kernel).
 * Zero in a field means "library default for this problem". */
typedef struct {
  int32_t tile_n;  /* path 4: output columns per thread block (16, 32, 64 or 128);
                      path 1: groups of 16 row bands per thread block (1, 2 or 4) with 128 output columns per
                      thread block, or 8 / 9 = 256 output columns per thread block (a lane owns two 4-column
                      pieces) with 1 / 2 groups (block height <= 8 / <= 4), or 17 / 18 / 20 = the 16-column tile
                      for N <= 16 (a lane owns one column) with 1 / 2 / 4 groups; plus 256 x the number of
                      thread blocks that share a tile's block columns (split multiply, 1 - 8);
                      path 3: 1 = values staged in registers, 2 = values streamed through shared memory by bulk
                      asynchronous copies (persistent thread blocks), 0 = the streaming variant when it fits */
  int32_t path;    /* 0 auto; 1 register-tiled CUDA-core kernel (N > 16); 2 tcgen05 tensor-core tiles (bf16
                      handles only); 3 lane-per-column kernel (N <= 16, N = 1 is the matrix-vector product);
                      4 shared-memory slab kernel (any N; the fall-back for operands the others do not take);
                      5 paired tcgen05 kernel: two thread blocks multiply 256 rows x 512 columns together
                      (bf16 handles; the default for wide right-hand sides on matrices of 256 rows or more).
                      A path that cannot take the request returns GRIM_ERR_UNSUPPORTED. */
  int32_t reserved[6];
} grim_tune_t;

/* ---------------------------------------------------------------------------------------------
 * Packing (host).  Section 3.2 (pattern), Sections 4.2 - 4.3 (reorder + compact storage).
 *
 * grim_bcr_pack reads a dense fp32 weight W_host[M x K] (row stride ldw) and a keep-mask
 * mask_host[M x K] (row stride ldm; non-zero = kept) from HOST memory and builds a handle.
 *   - A row / column of a block counts as kept when any of its entries is kept.  Every block's
 *     mask must equal (kept rows) x (kept columns), otherwise GRIM_ERR_NOT_BCR.
 *   - The mask is authoritative: a kept weight whose value is 0.0 stays stored and counted.
 *   - M or K need not be multiples of bh / bw: edge blocks are smaller (equivalent to zero padding).
 *   - Blocks that keep nothing are legal and cost nothing.
 *   - value_dtype GRIM_BF16 rounds the kept weights to bf16 (nearest, ties to even) once, here.
 *   - Limits: 1 <= bh <= 16, 1 <= bw <= 64, M, K < 2^31, nnz < 2^32; else GRIM_ERR_UNSUPPORTED.
 *   - Synchronous.  Unless GRIM_PACK_HOST_ONLY is set it allocates device memory on the current
 *     device and uploads the packed arrays (one blocking copy per array).
 * W_host and mask_host are only read during the call.
 */
grim_status_t grim_bcr_pack(const float* W_host, int64_t ldw, const uint8_t* mask_host, int64_t ldm,
                            int64_t M, int64_t K, int bh, int bw, grim_dtype_t value_dtype,
                            uint32_t flags, grim_bcr_t* out);

/* Frees the handle's host and device buffers.  NULL is accepted. */
grim_status_t grim_bcr_destroy(grim_bcr_t h);

grim_status_t grim_bcr_info(grim_bcr_t h, grim_bcr_info_t* info);

/* Canonical packed form (the compact storage idea of Section 4.3 in a fully specified layout),
 * written to HOST memory as a little-endian byte string of info.export_bytes bytes:
 *   8 x int64: magic "GRIMBCR1", M, K, bh, bw, nbr, nbc, dtype
 *   per block, row-major over the block grid: u16 kr, u16 kc, u16 rows[kr], u16 cols[kc]
 *     (block-local, ascending), values[kr*kc] row-major over (rows, cols) as fp32 or bf16 bits
 *   int32 row_perm[M]: with GRIM_PACK_REORDER the rows sorted by kept-weight count, largest
 *     first, ties by row index (the reorder array of Section 4.3); identity otherwise.
 * capacity < export_bytes gives GRIM_ERR_INVALID_ARG; *written receives the size.
 */
grim_status_t grim_bcr_export(grim_bcr_t h, void* buf_host, int64_t capacity, int64_t* written);

/* BCRC, the storage format of Section 4.3, written to HOST arrays.  Rows are reordered by kept-weight count (largest
 * first), then by column list, then by row id, so that rows with the same column list are neighbours; such a run of
 * rows is a group and its column list is stored once:
 *   reorder[M]                 original row at each position of the reordered matrix
 *   row_offset[M + 1]          first weight of each reordered row in `weights`
 *   occurrence[groups + 1]     first reordered row of each group
 *   column_stride[groups + 1]  first entry of each group's column list in compact_column
 *   compact_column[compact_columns]   the groups' column lists (ascending column ids)
 *   weights[nnz]               kept weights row by row of the reordered matrix, fp32 (bf16 handles: the rounded values)
 * Call once with all six array pointers NULL to learn the sizes, then with arrays of those sizes.  (The figure that
 * carries the paper's worked example is not part of the available text; the fragments quoted in the text are
 * reproduced by a test.) */
typedef struct {
  int64_t M, K, nnz;
  int64_t groups;           /* runs of reordered rows that share one column list */
  int64_t compact_columns;  /* entries of compact_column */
} grim_bcrc_sizes_t;
grim_status_t grim_bcr_export_bcrc(grim_bcr_t h, int32_t* reorder, int64_t* row_offset, int32_t* occurrence,
                                   int64_t* column_stride, int32_t* compact_column, float* weights,
                                   grim_bcrc_sizes_t* sizes);

/* Projection onto the BCR-sparse set (Section 5.2, Eq. (4): the step of the ADMM pruning that produces the masks this
 * library packs).  V_host [M x K] (row stride ldv) is read, mask_host [M x K] (row stride ldm) receives 1 for kept and
 * 0 for pruned entries; the projected matrix is V with the pruned entries set to zero.  The mask is BCR on the bh x bw
 * grid and keeps at most (1 - sparsity) * M * K entries.  The exact nearest member of the set is a combinatorial
 * problem and the paper gives no algorithm; this is a deterministic greedy one: a line (one row or one column of one
 * block) costs the mean square of its entries that are still kept, and the cheapest line (ties: smallest
 * block * (bh + bw) + row, or + bh + column) goes until the budget is met.  With 1 x 1 blocks it is magnitude pruning,
 * i.e. the exact projection.  HOST only; *kept (may be NULL) receives the number of kept entries. */
grim_status_t grim_bcr_project(const float* V_host, int64_t ldv, int64_t M, int64_t K, int bh, int bw, double sparsity,
                               uint8_t* mask_host, int64_t ldm, int64_t* kept);

/* Writes the masked weight (zeros at pruned positions; bf16 handles: the rounded values) as
 * fp32 into HOST memory W_host[M x K], row stride ldw. */
grim_status_t grim_bcr_unpack_dense(grim_bcr_t h, float* W_host, int64_t ldw);

/* ---------------------------------------------------------------------------------------------
 * Y = W * X.  Section 3.1 (unified GEMM / GEMV view), Sections 4.2, 4.4, 4.5 (execution).
 *
 * X: K x N, Y: M x N, both DEVICE, row-major with their own ld (>= cols).  X->dtype must equal
 * the handle's value dtype; Y->dtype is GRIM_F32, or GRIM_BF16 for bf16 handles (rounded once,
 * after fp32 accumulation).  Y is fully overwritten (all M rows, beta = 0): rows kept by no
 * block are written as +0.  N = 1 selects the matrix-vector kernel.  X and Y must not overlap.
 * Shape mismatch -> GRIM_ERR_SHAPE, dtype mismatch -> GRIM_ERR_DTYPE, both before any launch.
 * Asynchronous on `stream`; never allocates.  A handle is used on one stream at a time.  The kernels are launched
 * with programmatic stream serialization: their set-up may overlap the end of the launch before them on the stream,
 * and they wait for that launch to complete before they read X or write Y - stream order is what the caller sees.
 * Without an explicit choice (grim_bcr_spmm_ex) the kernel and tile shape are the ones grim_bcr_tune found for
 * this handle and this kind of request (same power-of-two bucket of N, same dtypes), else a static default.
 */
grim_status_t grim_bcr_spmm(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, grim_stream_t stream);

/* Workspace of the split tensor-core multiply (Section 4.5: the tile plan depends on the problem; bf16 handles with
 * few output tiles and a long K - small batches of the deeper convolution layers - are split over K through an fp32
 * scratch of M x N floats).  Compute calls never allocate: grim_bcr_reserve allocates that scratch for right-hand
 * sides of up to max_ncols columns (for a convolution: images x OH x OW), once, at set-up time; it synchronises the
 * device.  Without it (or beyond max_ncols) such multiplies simply run unsplit, slower.  max_ncols = 0 frees it.
 * More than 2^30 bytes -> GRIM_ERR_UNSUPPORTED. */
grim_status_t grim_bcr_reserve(grim_bcr_t h, int64_t max_ncols);

/* The multiply kernels bound every device-side wait (on a shared-memory barrier that an asynchronous copy
 * completes).  If one ever gives up, the kernel leaves, Y is invalid and an error word in the handle is set.
 * grim_bcr_status synchronises the device, returns GRIM_ERR_TIMEOUT in that case (GRIM_OK otherwise) and
 * clears the word.  (Robustness aid; no counterpart in the paper.) */
grim_status_t grim_bcr_status(grim_bcr_t h);

/* Same with an explicit tile choice (Section 4.5, tuning).  tune may be NULL. */
grim_status_t grim_bcr_spmm_ex(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, const grim_tune_t* tune,
                               grim_stream_t stream);

/* Times the candidate tile shapes for (handle, X/Y shapes and dtypes) on `stream` (synchronises)
 * and returns the fastest in *best (Section 4.5: per-kernel tuning of tile shape; the paper's
 * genetic search is replaced by a small fixed candidate set).  Y is overwritten.  The answer is also
 * stored in the handle: later grim_bcr_spmm calls with N in the same power-of-two bucket and the same
 * dtypes use it.  reps > 0: every candidate is launched reps times back to back (operands that fit the L2 cache are
 * read from it - right for small matrices called in a loop); reps < 0: -reps launches, each after the L2 cache has
 * been flushed by clearing a 256 MiB scratch (right for operands that are streamed from HBM every time; the
 * scratch is allocated and freed inside the call; GRIM_ERR_ALLOC when it cannot be had); 0 = 5.  A set-up call:
 * it synchronises and, with reps < 0, allocates. */
grim_status_t grim_bcr_tune(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, int reps, grim_tune_t* best,
                            float* best_ms, grim_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * Convolution as an implicit-im2col BCR GEMM.  Section 3.1 (CONV as GEMM), Section 4.5
 * ("Computation Transformation": rows of the expanded input whose weight column is pruned are
 * never produced).
 *
 * The handle holds the weight viewed as Cout x (C*KH*KW), K axis flattened as
 * k = (c*KH + kh)*KW + kw.  in: [N, C, H, W], out: [N, Cout, OH, OW] (NCHW, contiguous, DEVICE),
 * OH = (H + 2*pad - KH)/stride + 1, likewise OW.  out = conv(in) + bias, then max(.,0) if
 * GRIM_CONV_RELU.  bias_dev: Cout fp32 DEVICE values or NULL.  in_dtype must equal the
 * handle's dtype; out_dtype GRIM_F32 or (bf16 handles) GRIM_BF16.  Accumulation is fp32.
 */
#define GRIM_CONV_RELU 1u
/* Kernel choice (Section 4.5, per-kernel tuning), normally left to the library: ask for the paired tensor-core kernel
 * (two thread blocks multiply 256 rows x 512 pixels together) or for the single-block one; a kernel that cannot take
 * the request returns GRIM_ERR_UNSUPPORTED.  bf16 handles, 3x3 / stride 1 / pad 1 only. */
#define GRIM_CONV_PAIRED 2u
#define GRIM_CONV_SINGLE 4u
typedef struct {
  int64_t N, C, H, W;
  int32_t KH, KW, stride, pad;
  const float* bias_dev;
  uint32_t flags;
  grim_dtype_t in_dtype, out_dtype;
} grim_conv_desc_t;

grim_status_t grim_bcr_conv2d(grim_bcr_t h, const grim_conv_desc_t* d, const void* in_dev, void* out_dev,
                              grim_stream_t stream);

/* 2x2 / stride-2 max-pool on NCHW DEVICE tensors (H, W even); glue between the conv layers of a
 * VGG-style stack (Section 6.1 evaluates VGG-16), not part of the sparse multiply itself. */
grim_status_t grim_maxpool2x2(const void* in_dev, void* out_dev, int64_t N, int64_t C, int64_t H, int64_t W,
                              grim_dtype_t dtype, grim_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * GRU sequence inference, batch 1.  Section 3.1 (RNN layers are matrix-vector products),
 * Section 6.1 (a 2-layer GRU is the RNN workload).  The paper gives no equations; this is the
 * common variant with gate order r, z, n in the 3H rows:
 *   g = W_ih x_t + b_ih,  q = W_hh h_{t-1} + b_hh
 *   r = sigmoid(g_r + q_r), z = sigmoid(g_z + q_z), n = tanh(g_n + r * q_n)
 *   h_t = (1 - z) * n + z * h_{t-1};   layer l > 0 takes layer l-1's h_t as its x_t.
 *
 * grim_gru_create: W_ih[l] is 3H x in_l, W_hh[l] is 3H x H (fp32 handles packed with the same
 * bh, H a multiple of bh and of 4, else GRIM_ERR_UNSUPPORTED); b_ih_host[l], b_hh_host[l]: 3H fp32 HOST values (copied).  The packed
 * matrices are borrowed: they must outlive the GRU handle.  max_T bounds the sequence length;
 * scratch for the hoisted input projections is allocated here.
 *
 * grim_gru_seq: x_dev [T x in_0], h0_dev [layers x H] or NULL (zeros), y_dev [T x H] receives the
 * last layer's h_t, hT_dev [layers x H] or NULL receives every layer's final state; all fp32
 * DEVICE.  Asynchronous.  The recurrent kernel keeps W_hh on-chip and exchanges h between thread
 * blocks every step; all of its waits are bounded.  If one gives up, the outputs are invalid and
 * grim_gru_status (which synchronises the stream used last) reports GRIM_ERR_TIMEOUT.
 */
grim_status_t grim_gru_create(int layers, const grim_bcr_t* W_ih, const grim_bcr_t* W_hh,
                              const float* const* b_ih_host, const float* const* b_hh_host, int64_t max_T,
                              grim_gru_t* out);
grim_status_t grim_gru_seq(grim_gru_t g, const float* x_dev, int64_t T, const float* h0_dev, float* y_dev,
                           float* hT_dev, grim_stream_t stream);
grim_status_t grim_gru_status(grim_gru_t g);
grim_status_t grim_gru_destroy(grim_gru_t g);

/* One time step for a batch of B independent sequences (Section 6.3 times the GRU at sequence length 1, batch 32): the
 * same equations with the batch as the right-hand side of the two sparse multiplies of every layer.  x_dev [B x in_0],
 * h_dev [layers x B x H] holds every layer's state and is updated in place, y_dev [B x H] or NULL receives the last
 * layer's new state; all fp32 DEVICE, batch-major.  Needs 2 * B <= max_T of grim_gru_create (GRIM_ERR_SHAPE
 * otherwise).  Asynchronous; allocates nothing. */
grim_status_t grim_gru_step(grim_gru_t g, const float* x_dev, int64_t B, float* h_dev, float* y_dev, grim_stream_t stream);

/* Layer pipelining of grim_gru_seq (execution detail, Section 4.2's concern with keeping all units busy; the paper
 * has no multi-layer schedule).  With more than one layer the sequence is cut into `chunks` pieces in time and layer
 * l works on piece k while layer l - 1 works on piece k + 1, each layer on an internal stream ordered by events; the
 * caller's stream continues after the last layer.  Stacks of more than three layers are not pipelined.  chunks = 0 lets the library choose, 1 runs the layers one after the
 * other on the caller's stream, at most 8.  Results do not depend on it. */
grim_status_t grim_gru_set_pipeline(grim_gru_t g, int chunks);

/* grim_gru_seq without any device allocation behind it.  (The paper has no counterpart: this entry
 * point exists for the way the library is deployed, not for the method.)
 *
 * Who needs it: code that runs where the CUDA allocator must not be called - a serving loop that has
 * handed all device memory to its own pool, a real-time audio / control thread that may not take the
 * allocator's locks or tolerate its latency, a process running under a memory budget that was fixed
 * at start-up.  Such a caller builds the GRU handle once during start-up (that step allocates) and
 * afterwards calls this function, which allocates nothing and calls no allocating library routine.
 *
 * Same arguments, results and error codes as grim_gru_seq.  The difference is where the per-call
 * scratch lives (the hoisted pre-activations, T x 3H floats, and for multi-layer models two T x H
 * inter-layer buffers): in one fixed 8 MiB array that is part of the library image and therefore
 * occupies 8 MiB on every GPU that loads the library, until the process exits.
 *   - Limit: round256(T*3H*4) + 2*round256(T*H*4) (second term only for layers > 1) must fit in
 *     8 MiB - e.g. H = 1024, two layers: T <= 409.  Larger requests return GRIM_ERR_UNSUPPORTED
 *     before anything is launched; use grim_gru_seq for those.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current).  Make that first call during start-up, before any CUDA stream capture.  The
 *     address is cached for the life of the process: it does not survive a cudaDeviceReset.
 *   - All calls in the process share the array and it keeps whatever the previous call left there.
 *     Nothing in it has to start at zero: every word the kernels read from it is written earlier in
 *     the same call.  Two calls that overlap on the GPU (different streams or handles) race on it;
 *     serialise them.
 *   - The current device must be the handle's device (GRIM_ERR_INVALID_ARG otherwise). */
grim_status_t grim_gru_seq_static(grim_gru_t g, const float* x_dev, int64_t T, const float* h0_dev, float* y_dev,
                                  float* hT_dev, grim_stream_t stream);

/* Test hook for the bounded waits of the recurrent kernel (no counterpart in the paper): thread
 * block `skip_cta` stays away from the per-step barrier (-1 = normal operation) and a waiting
 * block gives up after `spin_limit` polls (0 = default).  With a block missing, every wait runs
 * out, the kernel returns, and grim_gru_status reports GRIM_ERR_TIMEOUT; nothing waits forever. */
grim_status_t grim_gru_debug_barrier(grim_gru_t g, int skip_cta, unsigned spin_limit);

/* Per-kernel timing of the GRU path (measurement aid, Section 6 reports per-kernel times): when
 * enabled, grim_gru_seq records CUDA events on its stream around the hoisted input projection and
 * around the persistent recurrent kernel of every layer.  grim_gru_profile_read waits for the last
 * call and returns the two sums over layers in milliseconds. */
grim_status_t grim_gru_profile(grim_gru_t g, int enable);
grim_status_t grim_gru_profile_read(grim_gru_t g, float* projection_ms, float* recurrent_ms);

/* Measures the fp32 fused-multiply-add rate of the current device with a register-only micro-kernel (16 independent
 * chains per thread, full occupancy) and returns it in TFLOP/s: the ceiling against which the CUDA-core multiply is
 * reported (measurement aid for Section 6 style reporting; no counterpart in the paper).  Allocates and frees a
 * small device buffer and synchronises `stream`. */
grim_status_t grim_measure_ffma_peak(double* tflops, grim_stream_t stream);

/* Counts kernel launches issued by this library since load (or since the last reset). */
int64_t grim_launch_count(void);
void grim_launch_count_reset(void);

const char* grim_status_string(grim_status_t s);
const char* grim_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GRIM_H_ */
