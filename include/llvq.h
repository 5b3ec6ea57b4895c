/*
 * llvq.h -- C ABI of the B200 (sm_100a) LLVQ dequantization library.
 *
 * LLVQ stores every block of 24 weights as one integer index into a union of
 * Leech-lattice shells plus a per-block gain.  This library maps the stored
 * index stream back to weights on the GPU, with no materialised codebook, and
 * fuses that with the decode-time matrix-vector / small-batch matrix product.
 *
 * Conventions common to all entry points
 *   - Pointers named d_* are DEVICE pointers owned by the caller; the library
 *     never allocates, frees or retains them.  `stream` is a cudaStream_t
 *     passed as void* (NULL = default stream).  Work is enqueued on that
 *     stream and the call returns without synchronising, unless stated.
 *   - The compute entry points only enqueue kernels (llvq_gemm_small_batch_noalloc also one memset) and
 *     synchronise nothing, so a sequence of them can be captured into a CUDA graph once each kernel has been
 *     launched at least once outside a capture.  The kernels use programmatic dependent launch: in a stream (or
 *     graph) of them, a kernel's table load overlaps its predecessor's tail; it waits for the predecessor to
 *     finish before it reads any argument buffer.
 *   - Every function returns a status code (LLVQ_OK = 0).  Bad arguments are
 *     rejected on the host before anything is launched.  Nothing throws,
 *     aborts or traps.
 *   - Index stream (App. A: the global integer index I; Sec. 2.2: an index
 *     takes W = ceil(log2 N) bits): field b occupies bits [b*W, (b+1)*W) of a
 *     little-endian bit stream (stream bit t = bit t%8 of byte t/8).  Indices
 *     are 0-based, I in [0, N).  The buffer is 16-byte aligned and
 *     llvq_index_bytes() long (padded with zeros to a multiple of 16 bytes).
 *   - Gains: one IEEE binary16 bit pattern per block (uint16_t), finite.
 *   - A field with I >= N decodes to the zero vector and is counted in a
 *     device-side error counter (see llvq_last_error); it never faults.
 *   - Block layouts of a rows x cols matrix:
 *       LLVQ_LAYOUT_FLAT     block b holds elements 24b .. 24b+23 of the
 *                            row-major flattened matrix; the unused tail of the
 *                            last block is dropped.
 *       LLVQ_LAYOUT_ROWWISE  every row has ceil(cols/24) blocks of its own;
 *                            block r*ceil(cols/24)+c holds columns 24c..24c+23
 *                            of row r; the unused tail of a row's last block is
 *                            dropped (App. C pads K the same way).
 */
#ifndef LLVQ_H
#define LLVQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct llvq_ctx llvq_ctx;   /* opaque: host + device tables of one code; immutable after create */

enum {
    LLVQ_OK = 0,
    LLVQ_EINVAL = 1,        /* null pointer, negative or zero size, unknown enum value    */
    LLVQ_EALIGN = 2,        /* a pointer or leading dimension violates the stated alignment */
    LLVQ_EUNSUPPORTED = 3,  /* a size or code outside what the kernels support            */
    LLVQ_ECUDA = 4,         /* a CUDA runtime call failed                                 */
    LLVQ_EINDEX = 5,        /* reserved: invalid indices are counted, see llvq_last_error */
    LLVQ_ETIMEOUT = 6       /* a bounded device-side wait ran out (flag in llvq_last_error) */
};
enum { LLVQ_LAYOUT_FLAT = 0, LLVQ_LAYOUT_ROWWISE = 1 };
enum { LLVQ_F32 = 0, LLVQ_BF16 = 1 };
enum { LLVQ_FLAG_WAIT_TIMEOUT = 1u,     /* bits in llvq_last_error's flags */
       LLVQ_FLAG_SEARCH_GAVE_UP = 4u }; /* the encoder's search found no point of the code for some input (non-finite input) */
enum { LLVQ_EUCLIDEAN = 0, LLVQ_ANGULAR = 1 };   /* scoring of the encoder's search (Sec. 3.1) */

/*
 * Build the tables of the code  union of Shell(m), m_lo <= m <= m_hi  (Sec. 2.2:
 * Shell(m) = lattice points of squared norm 2m; m_lo = 2 gives the ball cut
 * Lambda_24(m_hi)) and upload them to CUDA device `device`.  Classes, their
 * order, cardinalities A * 2^B * P and cumulative offsets follow Sec. 2.4-2.5
 * and Sec. 3.2.  Supported: 2 <= m_lo <= m_hi <= 53 with N <= 2^72; (2,2),
 * (3,3), (2,13) and (2,53) are the codes the benchmarks use.
 * Allocates the library's own host and device tables; *out is freed by
 * llvq_destroy.  Synchronous.  device < 0 builds a host-only context: the
 * query functions work, every function that would launch returns LLVQ_EINVAL.
 * A context also owns the device scratch (partial sums of rows or row tiles that
 * several thread blocks share, arrival counters) that the fused products keep
 * zero between launches: launches that use the same context must be ordered, on
 * one stream or by events; launches that may overlap need a context each.
 */
int llvq_create(llvq_ctx** out, int m_lo, int m_hi, int device);
void llvq_destroy(llvq_ctx* ctx);

/* W = ceil(log2 N): 18 for (2,2), 24 for (3,3), 48 for (2,13), 72 for (2,53) (Sec. 2.2, Table 1). */
int llvq_index_bits(const llvq_ctx* ctx);
/* N = number of points of the code, as lo_hi[0] + 2^64 * lo_hi[1]. */
int llvq_num_points(const llvq_ctx* ctx, uint64_t lo_hi[2]);
/* Number of classes (Sec. 2.4): 3, 4, 383, 114976 for the four codes above. */
int llvq_num_classes(const llvq_ctx* ctx);
/* Bytes of an index stream of nblocks fields: ceil(nblocks*W/8) rounded up to 16. */
size_t llvq_index_bytes(const llvq_ctx* ctx, uint64_t nblocks);

/*
 * Host-side introspection of the tables (no device work; used to cross-check the
 * table generator).  Class j in global order (Sec. 3.2 (1)-(2)):
 * info = {m, parity (0 even / 1 odd), Golay weight w, sign bits B, number of distinct values};
 * *A, card and offset (as lo, hi) are the quantities of Sec. 2.5 / App. A step 2;
 * values[] / mults[] = distinct absolute values, descending, with multiplicities (24 entries of room).
 */
int llvq_class_info(const llvq_ctx* ctx, int j, int info[5], uint64_t* A, uint64_t card[2], uint64_t offset[2],
                    int values[24], int mults[24]);
/* The 4096 extended-Golay codewords (Sec. 2.3) in table order: by weight, then by value; bit i = coordinate i. */
int llvq_golay_table(const llvq_ctx* ctx, uint32_t out[4096]);

/*
 * Dequantizer, App. A steps 1-4: d_points[b][0..23] = the integer lattice point
 * (coordinates of L^int, |x_i| <= 28) of field b, b < nblocks.
 * d_idx: device, 16-byte aligned.  d_points: device, int8 [nblocks][24], 8-byte aligned.
 */
int llvq_decode_blocks(const llvq_ctx* ctx, const void* d_idx, uint64_t nblocks,
                       int8_t* d_points, void* stream);

/*
 * Shape-gain reconstruction w = g * s (App. E, "Shape-gain"; App. A for s):
 * d_w[r*ld + c] = bf16_rn( float(gain[b]) * float(x[b][j]) ) for the block b and
 * lane j that hold element (r, c) under `layout`; one rounding, to nearest even.
 * d_gain_f16: device, [nblocks] binary16 bits.  d_w_bf16: device, bf16 bits,
 * rows x cols with leading dimension ld >= cols (elements), 2-byte aligned
 * (16-byte aligned base and ld % 8 == 0 select the vectorised store path).
 * FLAT requires ld == cols.
 */
int llvq_dequant_matrix(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16,
                        int64_t rows, int64_t cols, int layout,
                        uint16_t* d_w_bf16, int64_t ld, void* stream);

/*
 * Fused dequantization + matrix-vector product of App. C: y = W x with
 * W (n_out x k_in, ROWWISE blocks) never written to memory.  The weights are
 * the bf16-rounded values llvq_dequant_matrix would produce; products are
 * accumulated in binary32.  d_x_bf16: device, [k_in] bf16 bits.
 * d_y: device, [n_out], float (y_dtype = LLVQ_F32) or bf16 bits (LLVQ_BF16).
 * The order in which partial sums are added is not fixed (shared-memory and global atomics): two calls on the same
 * inputs may differ in the last bits of y.  The same holds for every fused product of this library.
 */
int llvq_gemv(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16,
              int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
              void* d_y, int y_dtype, void* stream);

/*
 * Shape-gain with a projected spherical shape code and a scalar gain codebook (App. E "Shape-gain"; the
 * appendix comparing spherical shaping with shape-gain: C_shape = { x / |x| }, C_gain a small chi(24)-matched
 * codebook, reconstruction = gain * shape), optionally times a high-precision scale per output row (the
 * "0 bit gain" setting: gain_bits = 0, a one-entry codebook and the row scale alone).
 *
 * Stored format: ROWWISE fields of llvq_index_bits(ctx) + gain_bits bits (at most 64 in all), packed like the
 * index stream: the shape index I in the low bits, the gain index k in the gain_bits bits above it.
 * llvq_field_bytes gives the stream length (rounded up to 16 bytes; 0 on bad arguments).
 *
 * Arithmetic, every operation in binary32 and rounded once:
 *     rn  = float( 1 / sqrt(16 m) )           m = shell of the point, |x|^2 = 16 m; formed in binary64
 *     g   = (row_scale[r] * codebook[k]) * rn  row_scale == NULL means 1
 *     w_j = bf16_rn( g * float(x_j) )
 * A field with I >= N decodes to zeros and is counted (see llvq_last_error).
 *
 * d_fields: device, 16-byte aligned.  d_codebook_f32: device, [1 << gain_bits] floats, 0 <= gain_bits <= 8.
 * d_row_scale_f32: device, [rows] ([n_out]) floats, or NULL.  Other arguments as in llvq_dequant_matrix (layout
 * is always ROWWISE) and llvq_gemv.  Codes whose class tables do not fit shared memory ((2,53)) return
 * LLVQ_EUNSUPPORTED.
 */
size_t llvq_field_bytes(const llvq_ctx* ctx, uint64_t nblocks, int gain_bits);
int llvq_dequant_matrix_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32,
                           const float* d_row_scale_f32, int64_t rows, int64_t cols,
                           uint16_t* d_w_bf16, int64_t ld, void* stream);
int llvq_gemv_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32,
                 const float* d_row_scale_f32, int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                 void* d_y, int y_dtype, void* stream);
/* The small-batch product (see llvq_gemm_small_batch for X, Y and batch) with W in the same shape-gain form. */
int llvq_gemm_small_batch_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, const float* d_codebook_f32,
                             const float* d_row_scale_f32, int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                             int batch, uint16_t* d_y_bf16, void* stream);

/*
 * Sorted layout for the fused GEMV: a kernel-private arrangement of the same blocks, made once at load time (the
 * paper fixes no storage layout, only that every block is stored as one integer, Sec. 1; App. A step 5 notes
 * that blocks are independent, which is what makes reordering them legitimate).  llvq_sort_blocks rewrites a
 * ROWWISE index stream for the GPU of this context: the blocks each thread block of the GEMV will own are stored,
 * in segments of up to 65536 blocks, ordered by the form of App. A steps 3-4 their class needs (odd / even with
 * Golay weight 8, 12, 16 / other), its number of unranking steps and the class, every block as a 64-bit entry
 * holding the stored index unchanged (low 48 bits) and its position in the segment (high 16 bits).
 * llvq_gemv_sorted computes the same y = W x as llvq_gemv: all of App. A steps 1-4 still run in the kernel, but the
 * 32 lanes of a warp now execute one form with one trip count and read one class descriptor.
 * The sorted stream takes llvq_sorted_bytes() bytes (8 per block of the 8-row x 4-block units the matrix is padded
 * to; 0 if unsupported: a code with its class tables in shared memory needs at most 1023 classes and fewer than
 * 2^48 - 1 points, which holds for (2,2), (3,3) and (2,13)).  The layout depends on the SM count of the device; use
 * it with the context that produced it.  d_sorted: device, 16-byte aligned.  Out-of-range fields are counted when
 * sorting and decode to zero.  Gains stay in their ROWWISE array.
 * Codes whose class tables stay in global memory (the 72-bit code (2,53)): the three calls work on the layout of
 * llvq_sort_blocks_gemm (96-bit entries in domains of 128 rows x 8 column blocks; llvq_sorted_bytes =
 * llvq_sorted_gemm_bytes, llvq_sort_blocks = llvq_sort_blocks_gemm), which does not depend on the SM count, and
 * llvq_gemv_sorted is the batch-1 case of the sorted small-batch product with the GEMV's output types; it asks for
 * d_x_bf16 16-byte aligned and k_in % 8 == 0 (LLVQ_EALIGN otherwise) and n_out <= 65536.
 */
size_t llvq_sorted_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in);
int llvq_sort_blocks(const llvq_ctx* ctx, const void* d_idx, int64_t n_out, int64_t k_in, void* d_sorted, void* stream);
int llvq_gemv_sorted(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16,
                     int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                     void* d_y, int y_dtype, void* stream);

/*
 * Several independent products y_i = W_i x_i in one launch (App. C's fused product, applied to the matrices of a
 * decoder layer that read the same or unrelated inputs: q, k and v; gate and up).  Blocks, and therefore matrices,
 * are independent (App. A step 5), so the thread blocks take their share of each matrix in turn and the fixed cost
 * of a launch (table staging, first loads, drain) is paid once.  No output may be an input of another matrix of the
 * same call.  descs: HOST array of n_mats (1..8) descriptions; every pointer inside is a device pointer owned by the
 * caller with the alignment llvq_gemv / llvq_gemv_sorted ask for; d_weights is the stored index stream
 * (llvq_gemv_multi) or the stream made by llvq_sort_blocks (llvq_gemv_sorted_multi).  All outputs have type
 * y_dtype.  The descriptions are copied into the launch, nothing is kept.  Results are those of the single calls (the
 * same kernels' code runs per matrix).  LLVQ_EUNSUPPORTED: more than 8 matrices, a code or a k_in the single call does
 * not take in this form either, a matrix with fewer 8-row x 4-block units than the device has SMs, or more than
 * 64 * 65536 output rows in total.
 */
typedef struct {
    const void* d_weights;
    const uint16_t* d_gain_f16;     /* [n_out * ceil(k_in / 24)] ROWWISE */
    int64_t n_out, k_in;
    const uint16_t* d_x_bf16;       /* [k_in] */
    void* d_y;                      /* [n_out] */
} llvq_gemv_desc;
int llvq_gemv_multi(const llvq_ctx* ctx, const llvq_gemv_desc* descs, int n_mats, int y_dtype, void* stream);
int llvq_gemv_sorted_multi(const llvq_ctx* ctx, const llvq_gemv_desc* descs, int n_mats, int y_dtype, void* stream);
/*
 * The same for the shape-gain form: llvq_sort_blocks_sg sorts a stream of fields of llvq_index_bits(ctx) + gain_bits
 * bits (at most 48 in all: the entry keeps the whole field, shape index and gain index), llvq_gemv_sorted_sg computes
 * the y of llvq_gemv_sg from it.  Same size (llvq_sorted_bytes) and the same restrictions as above.
 */
int llvq_sort_blocks_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, int64_t n_out, int64_t k_in,
                        void* d_sorted, void* stream);
int llvq_gemv_sorted_sg(const llvq_ctx* ctx, const void* d_sorted, int gain_bits, const float* d_codebook_f32,
                        const float* d_row_scale_f32, int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                        void* d_y, int y_dtype, void* stream);

/*
 * The same product for a small batch, Y[b][i] = sum_k X[b][k] W[i][k]
 * (App. C's kernel generalised to batch <= 64): the dequantized bf16 tile is
 * fed to the tensor cores, accumulation in binary32.
 * d_x_bf16: device, [batch][k_in] bf16 bits, 16-byte aligned, k_in % 8 == 0.
 * d_y_bf16: device, [batch][n_out] bf16 bits.  1 <= batch <= 64.
 */
int llvq_gemm_small_batch(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16,
                          int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                          int batch, uint16_t* d_y_bf16, void* stream);

/*
 * Sorted layout for the small-batch product (same idea and same licence as llvq_sort_blocks): the blocks of every
 * domain of 128 rows x 8 column blocks are stored ordered by decoder form, unranking steps and class, one 64-bit
 * entry per block (stored index unchanged in the low 48 bits, position in the domain above).
 * llvq_gemm_small_batch_sorted computes the same Y as llvq_gemm_small_batch from that stream and the unchanged
 * ROWWISE gains; all of App. A steps 1-4 run in the kernel.  llvq_sorted_gemm_bytes() gives the stream length (8 bytes
 * per block of the matrix padded to whole domains; 0 if unsupported: same codes as llvq_sort_blocks, plus the one below).
 * Codes whose class tables live in global memory (the 72-bit code, shells 2..53) take 96-bit entries, 12 bytes per
 * block: the index as its two digits in the mixed radix of the class table, i.e. the class (17 bits) and the class-local
 * index I - offset[class] (63 bits; bit 63 marks "no block"), and the position in the domain (10 bits).  App. A step 2
 * (class look-up, a bisection over 128-bit offsets on the stored stream) is thus taken when the layout is made; steps 3-4
 * (the unranking) run in the kernel as before.  The order is by the shape of the unranking: parity (odd first), number
 * of steps, which steps take at most three slots.
 * Out-of-range indices are counted by llvq_sort_blocks_gemm and stored as "no block".
 * d_sorted: device, 16-byte aligned.  Other arguments and limits as in llvq_gemm_small_batch.
 */
size_t llvq_sorted_gemm_bytes(const llvq_ctx* ctx, int64_t n_out, int64_t k_in);
int llvq_sort_blocks_gemm(const llvq_ctx* ctx, const void* d_idx, int64_t n_out, int64_t k_in, void* d_sorted, void* stream);
int llvq_gemm_small_batch_sorted(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16,
                                 int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                                 int batch, uint16_t* d_y_bf16, void* stream);
/* The same for the shape-gain form (fields of llvq_index_bits(ctx) + gain_bits <= 48 bits; see llvq_sort_blocks_sg). */
int llvq_sort_blocks_gemm_sg(const llvq_ctx* ctx, const void* d_fields, int gain_bits, int64_t n_out, int64_t k_in,
                             void* d_sorted, void* stream);
int llvq_gemm_small_batch_sorted_sg(const llvq_ctx* ctx, const void* d_sorted, int gain_bits, const float* d_codebook_f32,
                                    const float* d_row_scale_f32, int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                                    int batch, uint16_t* d_y_bf16, void* stream);

/*
 * llvq_gemm_small_batch for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, same arguments, same result.)
 *
 * Who needs it: code that runs after the application has handed all device memory to its own
 * pool, code inside a latency-critical decode loop where the implicit device synchronisation of
 * cudaMalloc / cudaFree is not acceptable, and plug-ins whose host only lets them launch work.
 * llvq_gemm_small_batch itself takes its split-K scratch from a buffer the context allocated at
 * llvq_create; this variant instead uses a fixed array compiled into the library (1 MiB + 512
 * bytes of device memory on every GPU that loads the library, held until the process exits), and
 * calls no allocating routine at all.
 *
 * Limits: ceil(n_out / 128) <= 128 and  roundup(batch, 16) * roundup(n_out, 128) <= 262144
 * (for example 4096 rows at batch 64, or 16384 rows at batch 16); larger problems return
 * LLVQ_EUNSUPPORTED and launch nothing.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress with that
 * device current); make that first call outside any stream capture.
 * All calls share the one array: each call clears the part it uses on `stream` before the kernel
 * runs, so calls must be ordered on the GPU (same stream, or dependent streams); calls that
 * overlap in time race on the array and give wrong results.
 */
int llvq_gemm_small_batch_noalloc(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16,
                                  int64_t n_out, int64_t k_in, const uint16_t* d_x_bf16,
                                  int batch, uint16_t* d_y_bf16, void* stream);

/*
 * Encoder (Sec. 3.1 "Extending to spherical search", Sec. 3.2 "Indexing scheme"): nearest point of the code to
 * each real vector, and its index.  d_v_f32: device, [nblocks][24] floats in units of the integer coordinates
 * (a point of Shell(m) has squared norm 16 m; the caller applies its own scale).  Outputs: d_points, device,
 * int8 [nblocks][24] (the chosen lattice points) and d_index, device, uint64 [nblocks], 8-byte aligned (their
 * indices, ready for llvq_pack_fields).
 *
 * The paper defers the search itself to the literature.  Here the nearest point of the unbounded lattice is found
 * exactly by decoding all 2 x 4096 cosets (parity, Golay codeword) + 4 Z^24 under the sum rules of Sec. 2.4: a
 * binary32 scan of all cosets, then every coset within rounding distance of the best one again in binary64 (one
 * rounding per operation, sums over the coordinates in order; lowest parity, then lowest codeword position, among
 * equal distances), so the result does not depend on the scan's rounding.  The restriction to the shells of the code:
 *   LLVQ_EUCLIDEAN (spherical shaping, App. E): if the nearest lattice point of the input lies in the code it is the
 *     answer (and then the nearest point of the cut as well).  Otherwise (input outside the ball, or next to the
 *     origin) the input direction is decoded at every shell radius sqrt(16 m), m_lo <= m <= m_hi, and of the
 *     candidates that lie in the code the one nearest to the input wins (first radius on ties): a candidate search,
 *     not an exact one.
 *   LLVQ_ANGULAR (shape-gain, App. E): the same candidates for every input; the one with the largest cosine wins.
 * A zero vector encodes to index 0.  Non-finite inputs encode to index 0 and set LLVQ_FLAG_SEARCH_GAVE_UP.
 * Supported codes: m_lo == 2, m_hi >= 3, indices of at most 64 bits; others return LLVQ_EUNSUPPORTED.
 *
 * llvq_rank_blocks is the indexing step alone (point -> index, the inverse of llvq_decode_blocks): a point that
 * is not in the code gets index 0 and is counted like an out-of-range field (llvq_last_error).
 *
 * llvq_pack_fields writes the stored stream from the indices: field b = d_index[b] | d_gain_index[b] << W
 * (gain_bits = 0: the plain index stream of llvq_index_bytes() bytes, d_gain_index ignored; otherwise the
 * shape-gain fields of llvq_field_bytes() bytes).  d_fields: device, 16-byte aligned.
 */
int llvq_encode_blocks(const llvq_ctx* ctx, const float* d_v_f32, uint64_t nblocks, int metric,
                       int8_t* d_points, uint64_t* d_index, void* stream);
int llvq_rank_blocks(const llvq_ctx* ctx, const int8_t* d_points, uint64_t nblocks, uint64_t* d_index, void* stream);
int llvq_pack_fields(const llvq_ctx* ctx, const uint64_t* d_index, const uint8_t* d_gain_index, int gain_bits,
                     uint64_t nblocks, void* d_fields, void* stream);

/*
 * Row-sharded GEMV over several GPUs, one process per GPU (App. A step 5: blocks are independent, so W splits by
 * output rows with no change to the arithmetic; x is the same on every rank).  A rank owns the band of rows
 * [row0, row0 + n_rows) of W: d_idx / d_gain_f16 (or d_sorted from llvq_sort_blocks, called with n_out = n_rows)
 * describe that band alone, ROWWISE, exactly as llvq_gemv / llvq_gemv_sorted take them.  The kernel writes the band's
 * results into EVERY rank's copy of the full vector: d_y_all is a HOST array of n_dest (1..8) DEVICE pointers, each
 * the start of a full-length y (element type y_dtype) that the calling process can store to - own_slot names this
 * rank's own copy, the others are the peers' exchange buffers opened with llvq_exchange_open (the stores cross
 * NVLink as plain remote writes; nothing is read from a peer).  Row row0 + i of every copy receives what llvq_gemv
 * would have put in y[i].  Copies may be the same pointer only if n_dest = 1.  Everything else (sizes, alignment,
 * errors, summation order) as llvq_gemv / llvq_gemv_sorted.
 * d_flag_words: NULL, or a HOST array of n_dest DEVICE addresses of 32-bit words (4-byte aligned; the entry at own_slot
 * is not read), one in each peer's exchange buffer with this rank as its only writer.  The kernel itself then stores
 * `epoch` there, with release semantics at system scope, once every row of the band is in place in every copy (the
 * last CTA to finish does it; with n_rows = 0 or k_in = 0 a one-warp kernel does) - what llvq_signal_ranks would do
 * in a launch of its own.  The peers see it through llvq_wait_ranks.  One such call at a time per context.  The epoch
 * is an argument of the launch: a captured CUDA graph would replay the same epoch, so these calls are made live.
 */
int llvq_gemv_rowshard(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_rows, int64_t k_in,
                       const uint16_t* d_x_bf16, void* const* d_y_all, int n_dest, int own_slot, int64_t row0,
                       int y_dtype, uint32_t* const* d_flag_words, uint32_t epoch, void* stream);
int llvq_gemv_sorted_rowshard(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16, int64_t n_rows,
                              int64_t k_in, const uint16_t* d_x_bf16, void* const* d_y_all, int n_dest, int own_slot,
                              int64_t row0, int y_dtype, uint32_t* const* d_flag_words, uint32_t epoch, void* stream);

/*
 * The same for the small-batch product: the band's rows are the columns [row0, row0 + n_rows) of every rank's
 * Y [batch][n_out_total] (bf16).  d_y_all lists the starts of those full matrices.  Stream, gains, X, batch and limits
 * as in llvq_gemm_small_batch / llvq_gemm_small_batch_sorted (called with n_out = n_rows), flags as above.
 */
int llvq_gemm_small_batch_rowshard(const llvq_ctx* ctx, const void* d_idx, const uint16_t* d_gain_f16, int64_t n_rows,
                                   int64_t k_in, const uint16_t* d_x_bf16, int batch, void* const* d_y_all, int n_dest,
                                   int own_slot, int64_t row0, int64_t n_out_total, uint32_t* const* d_flag_words,
                                   uint32_t epoch, void* stream);
int llvq_gemm_small_batch_sorted_rowshard(const llvq_ctx* ctx, const void* d_sorted, const uint16_t* d_gain_f16,
                                          int64_t n_rows, int64_t k_in, const uint16_t* d_x_bf16, int batch,
                                          void* const* d_y_all, int n_dest, int own_slot, int64_t row0,
                                          int64_t n_out_total, uint32_t* const* d_flag_words, uint32_t epoch,
                                          void* stream);

/*
 * Exchange buffers for the above (no counterpart in the paper: plumbing between processes).
 * llvq_exchange_create allocates `bytes` of zeroed device memory on the context's device as an allocation of its
 * own (so that it can be exported whole), returns it in *d_buf and writes its inter-process handle
 * (LLVQ_EXCHANGE_HANDLE_BYTES bytes, host) to handle64; the caller carries the handle to the other processes by any
 * host channel.  llvq_exchange_open maps another PROCESS's buffer (same machine, peer access possible) and returns
 * the pointer usable on this context's device; llvq_exchange_close unmaps it; llvq_exchange_destroy frees an own
 * buffer (after every peer has closed it).  These four calls synchronise the device.  LLVQ_ECUDA when the runtime
 * refuses (for instance a handle opened in the process that made it).
 */
#define LLVQ_EXCHANGE_HANDLE_BYTES 64
int llvq_exchange_create(const llvq_ctx* ctx, size_t bytes, void** d_buf, unsigned char* handle64);
int llvq_exchange_destroy(const llvq_ctx* ctx, void* d_buf);
int llvq_exchange_open(const llvq_ctx* ctx, const unsigned char* handle64, void** d_peer_buf);
int llvq_exchange_close(const llvq_ctx* ctx, void* d_peer_buf);

/*
 * llvq_signal_ranks: enqueue, after the kernels already on `stream`, a release store of `epoch` to each of the n
 * (0..8) DEVICE words listed in the HOST array d_flag_words (one word in each peer's exchange buffer, reserved for
 * this rank as the only writer).  Every store those kernels made, remote ones included, is visible to whoever then
 * reads the word with acquire semantics and finds the epoch.
 * llvq_wait_ranks: enqueue a one-warp kernel that waits until the words d_flags[p], p = 0..world-1 except p = skip
 * (pass -1 to wait on all), own DEVICE memory, 4-byte aligned, have reached `epoch` (modular comparison, so epochs may
 * wrap).  The wait is bounded: after max_spins polls (0 = the library's limit of about a second; larger values are
 * clamped to it) the kernel sets LLVQ_FLAG_WAIT_TIMEOUT, which llvq_last_error reports, and returns normally; what
 * follows on the stream then still runs, on incomplete data, so check the flag before trusting a step.
 */
int llvq_signal_ranks(const llvq_ctx* ctx, uint32_t* const* d_flag_words, int n, uint32_t epoch, void* stream);
int llvq_wait_ranks(const llvq_ctx* ctx, const uint32_t* d_flags, int world, int skip, uint32_t epoch,
                    uint32_t max_spins, void* stream);

/*
 * Self-test of the error path every kernel of this library uses for its device-side waits (table copy,
 * tensor-core completion): launches a one-warp kernel that waits, with a small iteration limit, on a barrier
 * nothing arrives at, sees the limit run out, sets LLVQ_FLAG_WAIT_TIMEOUT and returns normally.  Nothing
 * faults or hangs; the context stays usable.  llvq_last_error then reports the flag.  (No counterpart in the
 * paper.)
 */
int llvq_selftest_wait_timeout(llvq_ctx* ctx, void* stream);

/*
 * Synchronises `stream`, then reports and clears the device-side error state:
 * *n_bad_index = number of fields with I >= N seen since the last call,
 * *flags = OR of LLVQ_FLAG_* bits.  Either output pointer may be NULL.
 */
int llvq_last_error(llvq_ctx* ctx, void* stream, uint64_t* n_bad_index, uint32_t* flags);

#ifdef __cplusplus
}
#endif
#endif /* LLVQ_H */
