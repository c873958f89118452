/*
 * tetra.h -- C ABI of the B200 (sm_100a) Tetra decode-and-multiply library.
 *
 * Tetra stores every block of 24 weights as one 48-bit word that names a point
 * of the Leech lattice (Sec. 3 of the paper); the kernels here expand the word
 * inside the matrix-vector product (Sec. 5.1) and never materialise weights.
 *
 * Conventions for every entry point
 *   - returns a tetra_status; never throws, never exits the process;
 *   - "dev" pointers are device memory owned by the caller, "host" pointers are
 *     host memory owned by the caller; nothing is retained after the call
 *     returns except where stated;
 *   - work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream) and the call does not synchronise, except where
 *     stated;
 *   - arguments are validated on the host before anything is launched; a
 *     rejected call launches nothing;
 *   - the entry points may be called from several host threads at once (the
 *     library's one-time set-up per device is guarded); calls that share a
 *     workspace, an output buffer or tetra_gemv_noalloc's scratch array are
 *     ordered by the caller (same stream, or events).
 *
 * Word, file order ("canonical"): six little-endian bytes; fields from the
 * least significant bit: i1[11] i2[11] i3[11] s8[6] b1[1] b2[4] b3[1] p[1] r[1]
 * g[1] (Sec. 3.3, 3.4; the figure that fixes the positions is not printed, so
 * this order is this library's).  A matrix in file order is N rows of
 * nblocks words, tightly packed.
 */
#ifndef TETRA_H
#define TETRA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TETRA_OK = 0,
    TETRA_ERR_NULL = -1,   /* a required pointer is NULL */
    TETRA_ERR_SHAPE = -2,  /* N, K, nblocks or count out of range */
    TETRA_ERR_ALIGN = -3,  /* a pointer is not aligned as documented */
    TETRA_ERR_BATCH = -4,  /* batch outside [1, TETRA_MAX_BATCH] */
    TETRA_ERR_CUDA = -5,   /* a CUDA runtime call or launch failed */
    TETRA_ERR_SIZE = -6,   /* a caller buffer is too small */
    TETRA_ERR_TABLE = -7   /* the table blob was not written by tetra_build_table */
} tetra_status;

enum {
    TETRA_BLOCK = 24,              /* weights per word */
    TETRA_WORD_BYTES = 6,
    TETRA_MAX_BATCH = 16,
    TETRA_PAPER_TABLE_BYTES = 18816, /* 16384 + 2304 + 128, Sec. 3.4 */
    TETRA_NOALLOC_MAX_K = 24576,     /* largest K tetra_gemv_noalloc accepts */
    TETRA_LIST_MAX = 8               /* most matrices in one tetra_gemv_list call */
};

/* Human-readable name of a status code (static storage). */
const char *tetra_status_string(int status);

/* ---- tables (Sec. 3.2-3.4) --------------------------------------------- */

/* Size in bytes of the device table blob tetra_build_table writes: the paper's
 * 18,816-byte tables followed by the two gains and the derived lookup tables
 * the kernels stage in shared memory. */
size_t tetra_table_bytes(void);

/* Builds the decode tables on the host (Golay trellis of Sec. 3.2, rank rows
 * and middle list of Sec. 3.3, 1/sqrt(16 m) of Sec. 3.4) and copies them to
 * table_dev (16-byte aligned, at least tetra_table_bytes() bytes).
 * gain2_host: the two gain values of Eq. (2), or NULL for the defaults
 * {4.3156, 5.4415}.  Synchronises `stream` before returning. */
int tetra_build_table(void *table_dev, size_t bytes, const float *gain2_host, void *stream);

/* Writes the paper-format tables (rows u32 | prefixes | branches u16 | suffixes |
 * 32 floats, all little-endian, TETRA_PAPER_TABLE_BYTES bytes) to host memory.
 * Host-only; for inspection and checks. */
int tetra_table_export(void *blob_host, size_t bytes);

/* ---- decode only (Sec. 3.4, Fig. "decode") ----------------------------- */

/* Decodes nblocks words in file order.  codes_dev: 6*nblocks bytes (2-byte
 * aligned).  y_dev: int8 [nblocks][24] lattice coordinates.  mg_dev (may be
 * NULL): uint8 [nblocks][2] = shell index m, gain bit g.  Bit-exact integers. */
int tetra_decode_blocks(const void *codes_dev, const void *table_dev, int8_t *y_dev,
                        uint8_t *mg_dev, size_t nblocks, void *stream);

/* ---- HBM code layout (Sec. 5.1: the loader only reorders bits and pads) -- */

/* Bytes of the packed device layout of an N x nblocks matrix. */
size_t tetra_codes_bytes(int N, int nblocks);

/* Reorders file-order words (codes_dev, N*nblocks*6 bytes) into the layout the
 * GEMV kernels stream (packed_dev, 16-byte aligned, tetra_codes_bytes bytes).
 * A bijection on each word's 48 bits plus a tiling; no code is expanded.
 * table_dev: a blob written by tetra_build_table (its trellis map is read). */
int tetra_pack_codes(const void *codes_dev, const void *table_dev, void *packed_dev, int N,
                     int nblocks, void *stream);

/* Decodes a packed matrix with the GEMV kernel's own decoder: y_dev int8
 * [N][nblocks][24], mg_dev (may be NULL) uint8 [N][nblocks][2].  Must equal
 * tetra_decode_blocks on the file-order words. */
int tetra_decode_packed(const void *packed_dev, const void *table_dev, int8_t *y_dev,
                        uint8_t *mg_dev, int N, int nblocks, void *stream);

/* ---- decode-and-multiply (Eq. (2), Sec. 5.1) --------------------------- */

/* y[b][n] = row_scales[n] * sum_blk gain[g]/sqrt(16 m) * sum_j Y[n][blk][j] * x[b][24 blk + j]
 * with ceil(K/24) words per row and x read as zero beyond K.
 * codes: packed layout of an N x ceil(K/24) matrix (16-byte aligned).
 * row_scales: float32 [N].  x: float16 [batch][K] (2-byte aligned; 16-byte
 * aligned rows are faster).  y: float32 [batch][N], fully overwritten.
 * 1 <= batch <= 16.  The call takes no scratch memory, so with batch > 1 the
 * vectors are multiplied one after another inside one launch (every word is
 * decoded once per vector); tetra_gemv_batched decodes once for all vectors
 * and is the faster call from two vectors on.
 * Arithmetic: the 24 activations of a block column are held as 24-bit fixed
 * point with a power-of-two step 2^(E-22), 2^E <= max |x_j| < 2^(E+1) over the
 * column; the products with the lattice coordinates and their sum over the
 * block are exact integers, converted once and accumulated in float32 across
 * blocks.  An activation is therefore represented exactly when |x_j| >=
 * 2^(E-12), i.e. within a factor 4096 of its column's largest; a smaller one is
 * rounded to a multiple of the step (at most 2^-23 of the column's largest).
 * Non-finite activations: if any of a block column's 24 activations is NaN or
 * infinite, every output row comes out NaN (every row reads every column); a
 * non-finite value in the unquantized tail propagates by the IEEE rules of
 * float32 multiply-add.  The same holds for every decode-and-multiply entry
 * point below except tetra_gemv_paper_design, which multiplies in float32. */
int tetra_gemv(const void *codes, const float *row_scales, const void *table,
               const void *x, float *y, int N, int K, int batch, void *stream);

/* The paper's rule for K not a multiple of 24 (Sec. 4.1, 5.1): floor(K/24)
 * words per row plus an unquantized float16 tail [N][K mod 24], added after the
 * row-scale multiply.  codes: packed layout of an N x floor(K/24) matrix.
 * tail may be NULL when K mod 24 == 0. */
int tetra_gemv_tail(const void *codes, const float *row_scales, const void *table,
                    const void *x, float *y, int N, int K, int batch,
                    const void *tail, void *stream);

/* One product of a grouped call. Pointers are device pointers as in tetra_gemv_tail. */
typedef struct {
    const void *codes;        /* packed layout, N x floor(K/24) (tail != NULL or K % 24 == 0)
                                 or N x ceil(K/24) (tail == NULL) */
    const float *row_scales;  /* [N] */
    const void *x;            /* float16 [K] */
    const void *tail;         /* float16 [N][K % 24] or NULL */
    float *y;                 /* [N] */
    int32_t N;
    int32_t K;
} tetra_problem;

/* Batch-1 products of a SHORT list of independent matrices (1 <= count <=
 * TETRA_LIST_MAX) in one kernel launch, with no scratch memory and nothing to
 * plan: the call for the matrices of one dependency step of a model (q, k and v
 * of a layer; gate and up), the unit Sec. 5.2 times ("one launch per matrix").
 * The descriptors are read before the call returns.  Everything that does not
 * depend on the activations (decode tables, first code words, row scales) is
 * started before the kernel waits for its predecessor in the stream, so a chain
 * of such calls overlaps each launch's set-up with the previous launch.
 * tetra_gemv and tetra_gemv_tail are this call with one matrix. */
int tetra_gemv_list(const tetra_problem *problems_host, int count, const void *table,
                    void *stream);

/* Batch-1 products of a list of independent matrices from one persistent grid
 * (the tables staged in shared memory once, every warp walking independent
 * eight-row units of the whole list).  The list is planned once and run many
 * times:
 *   tetra_grouped_workspace_bytes  size of the scratch buffer for this list;
 *   tetra_gemv_grouped_plan        copies descriptors and index arrays into it
 *                                  (problems_host is read before the call returns);
 *   tetra_gemv_grouped_run         one step: a small pre-pass kernel rewrites the
 *                                  scratch buffer's fixed-point image of every x,
 *                                  then the persistent kernel computes every y.
 * workspace_dev: 16-byte aligned device memory owned by the caller; it belongs to
 * the plan until the last run using it has completed, and runs that share a
 * workspace must not overlap on the GPU.  The plan in the workspace describes
 * itself (list, mode, index arrays): a planned workspace may be copied to other
 * device memory and run from there, on the device it was planned for.
 * tetra_gemv_grouped_plan copies from host memory it frees before returning:
 * call it outside stream capture (tetra_gemv_grouped_run may be captured).
 * tetra_gemv_grouped = plan + run.  Lists of at most TETRA_LIST_MAX matrices are
 * served faster by tetra_gemv_list. */
size_t tetra_grouped_workspace_bytes(const tetra_problem *problems_host, int count);
int tetra_gemv_grouped_plan(const tetra_problem *problems_host, int count, void *workspace_dev,
                            size_t workspace_bytes, void *stream);
int tetra_gemv_grouped_run(void *workspace_dev, const void *table, void *stream);
int tetra_gemv_grouped(const tetra_problem *problems_host, int count, const void *table,
                       void *workspace_dev, size_t workspace_bytes, void *stream);

/* Several activation vectors at once (1 <= batch <= 16): every block is decoded
 * once and multiplied with all vectors; the contraction over a block's 24
 * coordinates runs on the tensor cores (int8 x int8 -> int32, exact), the
 * per-block scale and the accumulation across blocks in float32.  Same result
 * definition as tetra_gemv_tail.  workspace_dev: 16-byte aligned scratch of at
 * least tetra_batched_workspace_bytes(N, K) bytes (partial results of column
 * ranges, which a second small kernel sums in a fixed order; its contents need
 * no initialisation), private to the call until it completes.  Two kernel
 * launches; the result is bit-identical from run to run.  With one vector
 * the call runs tetra_gemv_tail's kernel instead (one launch, the workspace
 * untouched), which is faster there; two to four vectors run a kernel that
 * feeds the tensor cores from the decoder's registers, five and more one
 * that goes through shared-memory tiles. */
size_t tetra_batched_workspace_bytes(int N, int K);
int tetra_gemv_batched(const void *codes, const float *row_scales, const void *table,
                       const void *x, float *y, int N, int K, int batch, const void *tail,
                       void *workspace_dev, size_t workspace_bytes, void *stream);

/* Encoder search (Sec. 3.1, Eq. (2)).  For each block of 24 float32 weights
 * (w_dev: [nblocks][24]) finds the point of the format's codebook whose
 * direction is closest to the block -- the exact maximum of
 * <w, y> / (|w| |y|) over all 2^47 indices (the paper's own search is not
 * exhaustive; the objective and the codebook are the paper's) -- and the
 * gain bit g that minimises |w - y/|y| gain[g] sigma|^2, with gain[] from the
 * table and sigma = sigma_dev[block] (NULL: 1).  codes_dev receives the words in
 * file order, six bytes per block; cosine_dev (NULL allowed) the attained
 * cosine.  A zero block gives the all-zero word and cosine 0.  Rotation, the
 * error-feedback loop and the choice of sigma (Sec. 3.1, 4.2) are the caller's. */
int tetra_encode_blocks(const float *w_dev, const float *sigma_dev, const void *table_dev,
                        void *codes_dev, float *cosine_dev, size_t nblocks, void *stream);

/* The design the paper describes for its own GPU (Sec. 5.1: a warp per output
 * row, a lane per block, six table loads per block), kept as a comparison arm
 * and a cross-check.  codes: file-order words, row_stride bytes per row
 * (multiple of 2, >= 6*floor(K/24) or 6*ceil(K/24) as in tetra_gemv_tail). */
int tetra_gemv_paper_design(const void *codes, size_t row_stride, const float *row_scales,
                            const void *table, const void *x, float *y, int N, int K,
                            int batch, const void *tail, void *stream);

/* End-to-end convenience: x_host (float16 [batch][K]) is copied to x_stage_dev,
 * the product runs as tetra_gemv_tail, and y is copied from y_stage_dev to
 * y_host (float32 [batch][N]), all on `stream`.  Pinned host buffers make the
 * copies asynchronous.  Does not synchronise. */
int tetra_gemv_hostio(const void *codes, const float *row_scales, const void *table,
                      const void *x_host, float *y_host, void *x_stage_dev, float *y_stage_dev,
                      int N, int K, int batch, const void *tail, void *stream);

/* A planned run with host activations and results: copies x_bytes from x_host to
 * x_dev, runs tetra_gemv_grouped_run, copies y_bytes from y_dev to y_host, all on
 * `stream`.  The planned problems' x and y pointers are expected to point into
 * [x_dev, x_dev + x_bytes) and [y_dev, y_dev + y_bytes).  Does not synchronise.
 * Mapped results: a problem's y may also point into page-locked host memory that
 * the device can address (cudaHostAlloc / cudaHostRegister under unified
 * addressing); the kernels then store the results there directly, while they
 * run.  For a list planned that way pass y_host = y_dev = NULL: only the
 * activations are copied, and the results are in host memory once the stream
 * has passed the run. */
int tetra_gemv_grouped_hostio(void *workspace_dev, const void *table, const void *x_host,
                              void *x_dev, size_t x_bytes, float *y_host, const float *y_dev,
                              size_t y_bytes, void *stream);

/* The batch-1 product of tetra_gemv_tail for callers that cannot allocate
 * device memory (the paper has no counterpart: this is a packaging of the same
 * kernels).  A plug-in inside an application that owns the GPU's memory pool, a
 * control loop that may not touch the allocator, a process with a fixed memory
 * budget: none of them can hand the planned-list kernels the scratch buffer
 * they need, so this entry point keeps that buffer inside the library, as a
 * fixed array of 82,176 bytes in its device image (held by every GPU that
 * loads the library, until the process exits).  The call itself allocates
 * nothing, on the host or on the device.
 *   - Arguments as tetra_gemv_tail with batch = 1; tail == NULL selects the
 *     zero-pad rule.  K > TETRA_NOALLOC_MAX_K returns TETRA_ERR_SIZE.
 *   - The first call on a device looks up the array's device address; make
 *     that call before any stream capture begins on that device.
 *   - All calls share the one array, which keeps whatever the last call wrote.
 *     Nothing in it needs clearing (each call rewrites all it reads), but two
 *     calls that run on the GPU at the same time, on any streams, race on it:
 *     keep calls on one device in stream order, or serialise them.
 *   - K < 24 with a tail (no whole word in a row) returns TETRA_ERR_SHAPE, as in
 *     tetra_gemv_tail.
 *   - Enqueues three kernels on `stream` (the first writes the product's
 *     description into the array from its own parameters, so no host memory is
 *     referenced after the call returns); does not synchronise. */
int tetra_gemv_noalloc(const void *codes, const float *row_scales, const void *table,
                       const void *x, float *y, int N, int K, const void *tail, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TETRA_H */
