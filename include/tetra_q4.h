/*
 * tetra_q4.h -- C ABI for the 4-bit group-quantised matrices of a served model.
 *
 * Besides Tetra blocks, a model file stores some projections as int4 records:
 * 4-bit weights in groups of 128 along a row, with a float16 scale and a
 * float16 offset per group (Sec. 4.1, 4.3).  The embedding table and the
 * output head use the same record with groups of 64 (Sec. 4.4).  The kernel
 * dequantises each weight with its group's scale and offset and accumulates in
 * float32 (Sec. 5.1); embedding rows are dequantised on the fly for the input
 * tokens, and the head is a matrix-vector product over the same table
 * (Sec. 4.4).
 *
 * Conventions are those of tetra.h (status codes, device/host pointers, stream,
 * validation before launch; a rejected call launches nothing).
 *
 * Matrix in file order, as the caller supplies it (the paper leaves these free):
 *   q       uint8   [N][K/2]   byte b of a row holds weight 2b in its low nibble
 *                              and weight 2b+1 in its high nibble, values 0..15;
 *   scale   float16 [N][K/G]   group = k / G;
 *   offset  float16 [N][K/G];
 *   weight  w(n,k) = scale[n][k/G] * q(n,k) + offset[n][k/G].
 * G is 64 or 128 and K a multiple of G (every shape of the three models is).
 */
#ifndef TETRA_Q4_H
#define TETRA_Q4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TETRA_Q4_MAX_BATCH 8
#define TETRA_Q4_MAX_K 65536

/* Device layout.  tetra_q4_pack reorders a file-order matrix once (at load) into
 * the layout the kernels read: rows in strips of 32, and for every (strip,
 * group) one contiguous chunk: 512-byte tiles of 16 rows x 64 weights in which
 * every lane of a warp owns 16 bytes that dequantise, with five logic
 * operations per four registers, straight into tensor-core operand registers,
 * followed by the group's 32 (scale, offset) pairs.  Rows beyond N are zero.  No
 * bits are added except that padding:
 * tetra_q4_packed_bytes = ceil(N/32)*32 * (K/2 + 4*K/G).
 * All three pointers of the source and packed_dev are device memory, 16-byte
 * aligned; packed_bytes must be at least tetra_q4_packed_bytes(N, K, G)
 * (0 is returned for a shape that is rejected). */
size_t tetra_q4_packed_bytes(int N, int K, int G);
int tetra_q4_pack(const void *q_dev, const void *scale_dev, const void *offset_dev, void *packed_dev,
                  size_t packed_bytes, int N, int K, int G, void *stream);

/* y[v][n] = sum_k w(n,k) * x[v][k]  for v < batch (Sec. 5.1), 1 <= batch <=
 * TETRA_Q4_MAX_BATCH.  x_dev: float16 [batch][K], 16-byte aligned; y_dev:
 * float32 [batch][N].  Products of exact float16 values are accumulated in
 * float32 (tensor-core m16n8k16, one accumulator per group, then scale and
 * offset in float32).  One launch, no scratch memory, bit-identical from run
 * to run. */
int tetra_q4_gemv(const void *packed_dev, const void *x_dev, float *y_dev, int N, int K, int G, int batch,
                  void *stream);

/* out[t][k] = float16( fma(scale, q, offset) in float32 ) of row ids[t], for
 * t < count (Sec. 4.4: rows dequantised for the input tokens).  ids_dev: int32
 * [count], every id in [0, N) (an id outside it yields a row of zeros and is
 * not an error the host can see without a copy); out_dev: float16 [count][K],
 * 8-byte aligned. */
int tetra_q4_rows(const void *packed_dev, const int32_t *ids_dev, int count, void *out_dev, int N, int K, int G,
                  void *stream);

/* One product of a list call: packed_dev as written by tetra_q4_pack, x_dev float16 [K] (16-byte
 * aligned), y_dev float32 [N]. */
typedef struct {
    const void *packed;
    const void *x;
    float *y;
    int32_t N;
    int32_t K;
} tetra_q4_problem;

#define TETRA_Q4_LIST_MAX 4096

/* Batch-1 products of a list of independent 4-bit matrices with one group size G (the int4
 * projections of a token pass, Sec. 4.1, 4.3) from one persistent grid: the chunks of all matrices
 * form one stream that the warps cut into equal contiguous ranges, so nothing is paid per matrix.
 * The list is planned once and run many times:
 *   tetra_q4_list_workspace_bytes  size of the scratch buffer (descriptors, per-group sums of the
 *                                  activations, partial strips); 0 for a rejected list;
 *   tetra_q4_list_plan             writes the descriptors (problems_host is read before the call
 *                                  returns; call it outside stream capture);
 *   tetra_q4_list_run              one step, three launches: group sums of every x, the stream, the
 *                                  sum of the strips that two warps share (in warp order).
 * workspace_dev: 256-byte aligned device memory owned by the caller; it belongs to the plan until the
 * last run using it has completed, runs that share it must not overlap on the GPU, and it may be
 * copied to other device memory (the plan describes itself) on the device it was planned for.
 * Same result definition, arithmetic and tolerance as tetra_q4_gemv; bit-identical from run to run. */
size_t tetra_q4_list_workspace_bytes(const tetra_q4_problem *problems_host, int count, int G);
int tetra_q4_list_plan(const tetra_q4_problem *problems_host, int count, int G, void *workspace_dev,
                       size_t workspace_bytes, void *stream);
int tetra_q4_list_run(void *workspace_dev, int G, void *stream);

#ifdef __cplusplus
}
#endif
#endif
