/*
 * qil - low-bit quantised linear layers for sm_100a (B200), C ABI.
 *
 * The operations are the deployment form of the quantisation the paper applies
 * to its policies: operands of a GEMM are mapped to a 4-bit uniform grid by
 * round-to-nearest (paper Sec. 2.1); the OpenVLA backbone runs 4-bit
 * weight-only linears whose decode stage is memory bound (Sec. 5.4
 * "Implementation", App. A.4.2); the CILRS encoder runs 4-bit weights and 4-bit
 * activations because it is compute bound (Sec. 5.1, App. A.1.2).
 *
 * Conventions
 *   W is [N][K] (out features x in features, K contiguous); x is [M][K];
 *   y[m][n] = sum_k x[m][k] * W_hat[n][k].
 *   Unless a parameter says "host", every pointer is a DEVICE pointer owned by
 *   the caller.  The library never allocates, frees or synchronises (the two
 *   *_host entry points and qil_device_status are the documented exceptions:
 *   they enqueue copies, and qil_device_status waits for its own copy).
 *   Every call validates its arguments on the host first, then enqueues work
 *   on `stream` and returns; nothing throws, aborts or prints.
 *   Tensor base addresses must be 16-byte aligned.
 *
 * The quantiser, as an exact fp32 operation list (the paper names the method,
 * round-to-nearest, without a formula; this is the reading the library fixes):
 *   asymmetric uint4, per (row n, group of group_size consecutive k):
 *     lo = min(0, min w)   hi = max(0, max w)
 *     s  = fp16_rn((hi - lo) / 15)       ; s == 0 -> 1 ; s == inf -> error flag
 *     z  = clamp(rint(-lo / s), 0, 15)   ; stored as fp16 (an integer value)
 *     q  = clamp(rint(w / s) + z, 0, 15) ; dequantised value (q - z) * s
 *   symmetric int4, per (row, group):
 *     a = max |v| ; s = a / 7 ; a == 0 -> s = 1 ; (fp16 scale: round, 0 -> 1, inf -> error flag)
 *     q = clamp(rint(v / s), -8, 7)      ; dequantised value q * s
 *   All divisions are IEEE fp32 divisions, rint is round-half-to-even.
 *
 * Packed layout (canonical): element k of a row sits in 32-bit word k/8 at
 * bits [4*(k%8), 4*(k%8)+3]; signed codes keep their two's-complement nibble.
 */
#ifndef QIL_H_
#define QIL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QIL_OK = 0,
    QIL_ERR_NULL = 1,        /* a required pointer is null */
    QIL_ERR_SHAPE = 2,       /* non-positive size, K % 8 != 0, K % group_size != 0, ... */
    QIL_ERR_ALIGN = 3,       /* a tensor base is not 16-byte aligned */
    QIL_ERR_UNSUPPORTED = 4, /* enum value / combination the library does not implement */
    QIL_ERR_WORKSPACE = 5,   /* workspace missing or too small */
    QIL_ERR_CUDA = 6,        /* the CUDA runtime reported an error at launch */
    QIL_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (read through qil_device_status) */
    QIL_ERR_RANGE = 8        /* a quantisation scale does not fit fp16 (device flag) */
} qil_status;

typedef enum { QIL_F32 = 0, QIL_BF16 = 1, QIL_F16 = 2 } qil_dtype;

/*
 * QIL_LAYOUT_CANONICAL: packed words [N][K/8], row-major.
 * QIL_LAYOUT_TILE16   : the word matrix is cut into tiles of 16 rows x 16 words
 *   (= 128 columns of K).  Tiles are stored one after another, all column tiles
 *   of row-tile 0 first; inside a tile the 16 rows follow each other, 16 words
 *   each.  Word (n, i) is at ((n/16)*(K/128) + i/16)*256 + (n%16)*16 + i%16.
 *   Needs N % 16 == 0 and K % 128 == 0.  A warp of the decode kernel reads one
 *   tile (1 KiB) with two fully coalesced 512-byte loads.
 * QIL_LAYOUT_STREAM128: units for the tensor-memory (tcgen05) decode kernel, built by
 *   qil_pack_stream128_w4.  Unit u = (n/128)*(K/128) + k/128 occupies bytes
 *   [8704 u, 8704 (u+1)): 4 chunks (32 columns of K each) x 128 rows x 16 bytes of
 *   codes - byte b of 32-bit word m of a chunk holds column 8m+b of the chunk in its
 *   low nibble and column 8m+4+b in its high nibble - then 128 pairs {fp16 scale,
 *   fp16 zero}, one per row.  Rows beyond N are zero (N need not be a multiple of
 *   128).  Needs K % 128 == 0 and group_size % 128 == 0.
 */
typedef enum {
    QIL_LAYOUT_CANONICAL = 0,
    QIL_LAYOUT_TILE16 = 1,
    QIL_LAYOUT_STREAM128 = 3
} qil_layout;

typedef struct CUstream_st* qil_stream_t; /* a cudaStream_t */

/* ------------------------------------------------------------------------
 * Weight quantiser (Sec. 2.1 round-to-nearest; 4-bit weights of Sec. 5.4 and
 * Sec. 5.1).  symmetric = 0: uint4 codes 0..15, fp16 scale and fp16 zero point
 * per group (scale_dtype must be QIL_F16, zeros required).  symmetric = 1: int4
 * codes -8..7 stored as int8 in codes[], scale per group in scale_dtype
 * (QIL_F32 or QIL_F16), zeros ignored (may be null).  group_size == K gives one
 * scale per output channel (the paper's channel-wise setting, App. A.1.2).
 *   w      [N][K] of w_dtype          codes  [N][K] one code per byte
 *   scales [N][K/group_size]          zeros  [N][K/group_size] fp16
 *   dev_status: optional device int; QIL_ERR_RANGE is OR-ed into it when a
 *   scale overflows fp16 (the codes of that group are then unspecified).
 * Errors: NULL, SHAPE (sizes <= 0, K % group_size), ALIGN, UNSUPPORTED, CUDA.
 * ---------------------------------------------------------------------- */
qil_status qil_quantize_rtn_w4(const void* w, qil_dtype w_dtype, int N, int K, int group_size,
                               int symmetric, uint8_t* codes, void* scales, qil_dtype scale_dtype,
                               void* zeros, int* dev_status, qil_stream_t stream);

/* Pack 8 codes per 32-bit word (layout rules above); works for unsigned codes
 * and for two's-complement int8 codes alike (the low nibble is kept).
 * Errors: NULL, SHAPE (K % 8; TILE16: N % 16, K % 128), ALIGN, UNSUPPORTED. */
qil_status qil_pack_w4(const uint8_t* codes, int N, int K, qil_layout layout, uint32_t* packed,
                       qil_stream_t stream);
/* Inverse of qil_pack_w4; is_signed != 0 sign-extends each nibble into int8. */
qil_status qil_unpack_w4(const uint32_t* packed, int N, int K, qil_layout layout, int is_signed,
                         uint8_t* codes, qil_stream_t stream);

/* Builds the QIL_LAYOUT_STREAM128 buffer (qil_stream128_w4_bytes(N, K) bytes) from unsigned codes [N][K], fp16
 * scales and fp16 zeros [N][K/group_size].
 * Errors: NULL, SHAPE (N < 1, K % 128, group_size % 128, K % group_size), ALIGN. */
size_t qil_stream128_w4_bytes(int N, int K);
qil_status qil_pack_stream128_w4(const uint8_t* codes, const void* scales, const void* zeros, int N, int K,
                                 int group_size, void* out, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * Weight-only linear, 4-bit weights x bf16 activations (the OpenVLA / Llama-2
 * decode and prefill linears, Sec. 5.4, App. A.4.2): dequantisation is fused
 * into the matmul, accumulation is fp32, the result is rounded to bf16.
 *   x [M][K] bf16   qweight packed per `layout`   scales, zeros [N][K/group_size] fp16
 *   y [M][N] bf16
 * The kernel is chosen from the shape: on the canonical layout with M > 8,
 * K % 64 == 0 and group_size % 64 == 0 the tcgen05 prefill GEMM (weights
 * dequantised to bf16, one rounding per weight; one persistent, cooperative
 * launch whose CTAs take equal ranges of the GEMM's steps; tiles that several
 * CTAs share are added up in a fixed order); else the tensor-core skinny
 * kernel (weights read once, any M handled in slabs of 64 rows) when
 * K % 128 == 0 and group_size % 128 == 0; a general kernel otherwise (any
 * K % 8 == 0, any group_size dividing K, canonical layout only).  With
 * QIL_LAYOUT_STREAM128 (M <= 4) the persistent streaming kernel runs;
 * scales and zeros are part of the buffer, the two arguments are ignored and
 * may be null; the workspace is always needed.  The streaming kernel converts
 * the activations to 16-bit block fixed point (per 128 columns a power-of-two
 * scale, |integer| <= 32639) and accumulates exactly in int32; the conversion
 * error per element is at most 2^-16 of the block maximum.
 * workspace: qil_linear_w4a16_workspace_size() bytes, only touched when the
 * shape needs a split along K or the streaming kernel runs; it must be
 * zero-filled once before first use.  One workspace serves every layout: the
 * streaming kernel's part (a 256-byte header and the slots through which CTAs
 * hand partial row tiles to each other) comes first, the split-K scratch of the
 * skinny kernel after it; each kernel leaves its own part ready for the next
 * call (counters and slot tags back at zero; the header words 1..7 are scratch).
 * Calls that share a workspace must not overlap on the device.  Its first int
 * is a status word: the streaming kernel ORs QIL_ERR_TIMEOUT into it if one of
 * its bounded waits ever runs out (read it with qil_device_status; words 2..5
 * of the workspace then tell where: 1 + CTA, thread, shared-memory address of
 * the barrier or 0, parity; after such an error re-zero the workspace).
 * The streaming kernel is one CTA per SM and its CTAs wait for each other, so
 * it is launched cooperatively: all of them are resident together or the
 * launch is refused (QIL_ERR_UNSUPPORTED), e.g. on a device partition that is
 * smaller than the device.  It should not share the GPU with other kernels.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, CUDA.
 * ---------------------------------------------------------------------- */
size_t qil_linear_w4a16_workspace_size(int M, int N, int K, int group_size);
qil_status qil_linear_w4a16(const void* x, const uint32_t* qweight, const void* scales,
                            const void* zeros, void* y, int M, int N, int K, int group_size,
                            qil_layout layout, void* workspace, size_t workspace_bytes,
                            qil_stream_t stream);

/* -------------------------------------------------------------------------
 * qil_lora_side_add: the low-rank side path of a quantised linear, for
 * adapters that are kept beside the frozen 4-bit base instead of being merged
 * (the paper fine-tunes OpenVLA with QLoRA adapters of rank 32, App. A.1.2):
 *     y[m][n] = bf16( float(y[m][n]) + scale * sum_j (sum_k x[m][k] A[j][k]) B[n][j] )
 *   x [M][K] bf16   A [rank][K] bf16   B [N][rank] bf16   y [M][N] bf16, in place
 * fp32 accumulation; the inner product x . A^T is kept in fp32 in the
 * workspace, as up to 32 partial sums over slices of K that are added in a
 * fixed order (qil_lora_side_workspace_size(M) bytes, no initialisation needed).
 * Call it after the linear that produced y, on the same stream.
 * rank <= 32 (larger: UNSUPPORTED); K even.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, CUDA.
 * ---------------------------------------------------------------------- */
size_t qil_lora_side_workspace_size(int M);
qil_status qil_lora_side_add(const void* x, const void* a, const void* b, void* y, int M, int N, int K,
                             int rank, float scale, void* workspace, size_t workspace_bytes,
                             qil_stream_t stream);

/* -------------------------------------------------------------------------
 * qil_linear_w4a16_swiglu: the gate and up projections of a gated MLP (the
 * Llama-2 backbone of the paper's OpenVLA deployment, App. A.4.2) as ONE
 * weight-only linear with the activation fused into its epilogue:
 *     y[m][i] = silu(x[m] . W_hat[2 i]) * (x[m] . W_hat[2 i + 1]),   silu(g) = g / (1 + exp(-g))
 * Row 2 i of the N weight rows is gate row i, row 2 i + 1 is up row i
 * (group-wise quantisation is per row, so interleaving rows changes no code,
 * scale or zero point).  N must be even.
 *   x [M][K] bf16   qweight, scales, zeros as for qil_linear_w4a16 (canonical layout)
 *   y [M][N / 2] bf16
 * On the shapes the prefill GEMM takes (M > 8, K % 64 == 0, group_size % 64
 * == 0) gate and up products stay in fp32 until the result is rounded to bf16
 * once; on all other shapes the linear is computed as by qil_linear_w4a16 into
 * the workspace (bf16) and a second kernel applies the activation.
 * workspace: qil_linear_w4a16_swiglu_workspace_size() bytes, zero-filled once.
 * Errors: NULL, SHAPE (also odd N), ALIGN, WORKSPACE, UNSUPPORTED, CUDA.
 * ---------------------------------------------------------------------- */
size_t qil_linear_w4a16_swiglu_workspace_size(int M, int N, int K, int group_size);
qil_status qil_linear_w4a16_swiglu(const void* x, const uint32_t* qweight, const void* scales,
                                   const void* zeros, void* y, int M, int N, int K, int group_size,
                                   void* workspace, size_t workspace_bytes, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * qil_linear_w4a16 for callers that must not allocate device memory.  (The paper
 * has no counterpart to this call; it exists for integration reasons only.)
 * Some hosts of this library cannot call cudaMalloc at the point where they run
 * a linear: a real-time control loop that forbids allocation after start-up, a
 * plug-in whose host application owns all device memory, code running inside a
 * region where the allocator may not be entered.  qil_linear_w4a16 needs a
 * caller-allocated workspace whenever the shape is split along K; this variant
 * runs the skinny kernel (or, for shapes outside it, the general kernel, which
 * needs no scratch) with the split-K scratch held in a fixed array of
 * QIL_STATIC_WS_BYTES bytes that is part of the library image (each GPU that
 * loads the library keeps that much memory reserved until the process exits).
 * Arguments as qil_linear_w4a16, minus the workspace.  Two differences from
 * that call: QIL_LAYOUT_STREAM128 is not served (QIL_ERR_UNSUPPORTED: the list
 * kernel's workspace is larger than the array), and on the canonical layout
 * with M > 8 the result is the skinny kernel's (fp32 dequantisation), not the
 * prefill GEMM's (weights rounded to bf16): both are within the tolerance of
 * the linear, but their bits differ.  The array's address is looked up for the
 * device that is current at the call; `stream` must belong to that device.
 *  - Shapes whose split-K scratch (qil_linear_w4a16_static_ws_need) exceeds
 *    QIL_STATIC_WS_BYTES are rejected with QIL_ERR_WORKSPACE; nothing is launched.
 *  - The call allocates and frees nothing.  The first call on each device looks
 *    up the device address of the array (with that device current); make that
 *    first call outside any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's
 *    contents; the call clears the part that has to start at zero itself, on
 *    `stream`.  Two calls that overlap on the GPU (different streams, no
 *    ordering between them) race on the array: order them.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE (shape too large), CUDA.
 * ---------------------------------------------------------------------- */
#define QIL_STATIC_WS_BYTES (4u * 1024u * 1024u)
qil_status qil_linear_w4a16_static_ws(const void* x, const uint32_t* qweight, const void* scales,
                                      const void* zeros, void* y, int M, int N, int K,
                                      int group_size, qil_layout layout, qil_stream_t stream);
/* Bytes of the built-in array that a shape would use (0: the shape needs no scratch). */
size_t qil_linear_w4a16_static_ws_need(int M, int N, int K, int group_size);

/* ------------------------------------------------------------------------
 * A list of weight-only linears run in stream order (one decode pass over the
 * decoder layers, App. A.4.2: q, k, v, o, gate, up, down x layers).  The result
 * is the same as `count` calls of qil_linear_w4a16 in list order.  An entry
 * whose x is written by an earlier entry of the same list must carry
 * QIL_DEP_PREVIOUS in `flags`: it then starts only after every earlier entry has
 * written all of its outputs.  Entries without the flag may overlap with their
 * predecessors (q, k and v of one layer share an input and need no flag) and
 * with each other.  QIL_DEP_NEVER is a diagnostic flag: the entry waits for an
 * event that never happens, so the kernel's bounded wait runs out, the launch
 * ends with QIL_ERR_TIMEOUT in the status word and the outputs of that entry
 * and of all later ones are unspecified (used with qil_set_wait_limit_ns to
 * exercise the error path; the workspace must be re-zeroed afterwards).
 * When every entry uses QIL_LAYOUT_STREAM128, the whole list runs as one
 * persistent kernel.  All pointers inside a descriptor are device
 * pointers; the descriptor array itself is host memory and is consumed before
 * the call returns.  workspace must be as large as the largest
 * qil_linear_w4a16_workspace_size() over the entries (zero-filled once).
 * ---------------------------------------------------------------------- */
typedef struct {
    const void* x;           /* bf16 [M][K] */
    const uint32_t* qweight; /* packed per layout */
    const void* scales;      /* fp16 [N][K/group_size] */
    const void* zeros;       /* fp16 [N][K/group_size] */
    void* y;                 /* bf16 [M][N] */
    int M, N, K, group_size;
    int layout;              /* qil_layout */
    int flags;               /* 0 or QIL_DEP_PREVIOUS */
} qil_linear_desc;
#define QIL_DEP_PREVIOUS 1
#define QIL_DEP_NEVER 2

qil_status qil_linear_w4a16_batch(const qil_linear_desc* descs /*host*/, int count, void* workspace,
                                  size_t workspace_bytes, qil_stream_t stream);

/* Same, with the activations in HOST memory: copies x_bytes from x_host to
 * x_stage (device), runs the list (whose x / y pointers refer into x_stage /
 * y_stage), then copies y_bytes from y_stage to y_host.  All three steps are
 * enqueued on `stream`; the call does not wait.  Use page-locked host buffers
 * for the copies to be asynchronous. */
qil_status qil_linear_w4a16_batch_host(const qil_linear_desc* descs /*host*/, int count,
                                       const void* x_host, void* x_stage, size_t x_bytes,
                                       void* y_host, const void* y_stage, size_t y_bytes,
                                       void* workspace, size_t workspace_bytes, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * 8-bit weight-only linear (the INT8 deployment point of Table "OpenVLA
 * performance", Sec. 5.4): the same round-to-nearest quantiser on 256 levels,
 * and the linear with uint8 codes, one per byte.
 * qil_quantize_rtn_w8: arguments and errors as qil_quantize_rtn_w4.
 *   symmetric = 0: codes 0..255, s = fp16_rn((hi - lo) / 255), z = clamp(rint(-lo / s), 0, 255);
 *   symmetric = 1: codes -128..127 (int8), s = max|v| / 127.
 * qil_linear_w8a16: y[M][N] bf16 = x[M][K] bf16 . dequant(W)^T, fp32 result rounded to bf16.
 *   codes [N][K] uint8 row-major, scales and zeros [N][K/group_size] fp16.
 *   With K % 128 == 0 and group_size % 128 == 0 (and K small enough for the activations of four rows to fit
 *   shared memory: K <= 24576) a streaming kernel runs, four activation rows per pass: it converts the
 *   activations to 16-bit block fixed point per 128 columns (error at most 2^-16 of the block maximum) and
 *   accumulates integer dot products exactly.  Other shapes (K % 16 == 0) use a general kernel.
 *   With M > 8, K % 64 == 0 and group_size % 64 == 0 the tcgen05 prefill GEMM of qil_linear_w4a16 runs on the
 *   8-bit codes (weights dequantised to bf16, one rounding per weight).
 *   workspace: qil_linear_w8a16_workspace_size() bytes (at least 256), zero-filled once; its first int is the
 *   status word (QIL_ERR_TIMEOUT if a bounded wait ran out), its second a counter the list kernel uses between
 *   phases, the rest scratch of the prefill GEMM's split along K.
 * qil_linear_w8a16_batch: a list in stream order, flags as for qil_linear_w4a16_batch (layout must be
 *   QIL_LAYOUT_CANONICAL; desc.qweight points at the uint8 codes).  When every entry fits the streaming kernel
 *   (M <= 4) the list is one cooperative launch of one CTA per SM; rows are dealt out whole, so CTAs exchange
 *   nothing but the phase counter.
 * Errors: NULL, SHAPE (K % 16, K % group_size), ALIGN, UNSUPPORTED, WORKSPACE, CUDA.
 * ---------------------------------------------------------------------- */
qil_status qil_quantize_rtn_w8(const void* w, qil_dtype w_dtype, int N, int K, int group_size,
                               int symmetric, uint8_t* codes, void* scales, qil_dtype scale_dtype,
                               void* zeros, int* dev_status, qil_stream_t stream);
size_t qil_linear_w8a16_workspace_size(int M, int N, int K, int group_size);
qil_status qil_linear_w8a16(const void* x, const uint8_t* qweight, const void* scales, const void* zeros,
                            void* y, int M, int N, int K, int group_size, void* workspace,
                            size_t workspace_bytes, qil_stream_t stream);
qil_status qil_linear_w8a16_batch(const qil_linear_desc* descs /*host*/, int count, void* workspace,
                                  size_t workspace_bytes, qil_stream_t stream);

/* Per-token symmetric int8 activation quantiser of the W8A8 path (Table "CILRS performance", W8A8 row):
 * x [M][K] bf16 -> qx [M][K] int8, scales [M] fp32; divisor 127, clamp to [-128, 127]; static_scale as for
 * qil_quantize_act_a4. */
qil_status qil_quantize_act_a8(const void* x, int M, int K, const float* static_scale /*host*/, int8_t* qx,
                               float* scales, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * Activation quantiser of the W4A4 path (Sec. 5.1: the compute-bound driving
 * policy needs weights and activations in 4 bits): symmetric int4 per row.
 *   x [M][K] bf16 -> qx packed [M][K/8] (canonical), scales [M] fp32.
 * static_scale (host pointer) null: per-row absmax.  Non-null: that one fp32
 * value is used for every row (tensor-wise setting of App. A.1.2) and written
 * to scales[].
 * ---------------------------------------------------------------------- */
qil_status qil_quantize_act_a4(const void* x, int M, int K, const float* static_scale /*host*/,
                               uint32_t* qx, float* scales, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * W4A4 integer GEMM (Sec. 5.1 / Sec. 5.4 autonomous-driving deployment):
 *   acc[m][n] = sum_k qx[m][k] * qw[n][k]   (int32, exact)
 *   y[m][n]   = bf16( float(acc) * (sx[m] * sw[n]) )
 *   qx [M][K/8], qw [N][K/8] canonical packed signed nibbles; sx [M], sw [N] fp32
 *   acc_out: optional [M][N] int32 copy of the raw accumulators.
 * Needs K % 32 == 0 and K < 131072: the kernel works on bytes that are 16 x the
 * codes, its int32 accumulator holds 256 x the sum, and 256 * 64 K must stay
 * below 2^31.
 * workspace: qil_linear_w4a4_workspace_size() bytes, zero-filled once; its first
 * int is a status word that receives QIL_ERR_TIMEOUT if a bounded device-side
 * wait ever runs out (read it with qil_device_status).
 * ---------------------------------------------------------------------- */
size_t qil_linear_w4a4_workspace_size(int M, int N, int K);
qil_status qil_linear_w4a4(const uint32_t* qx, const float* sx, const uint32_t* qw, const float* sw,
                           void* y, int32_t* acc_out, int M, int N, int K, void* workspace,
                           size_t workspace_bytes, qil_stream_t stream);

/* W4A4 GEMM fused with the next layer's activation quantiser (a neighbour of the linear on the W4A4 path: with
 * the paper's tensor-wise static activation scale, App. A.1.2, the next layer's codes can be produced in this
 * layer's epilogue and the bf16 activations never touch memory):
 *   v = fl32(float(acc) * fl32(sx[m] * sw[n]));  v = max(v, 0) if relu;  q = clamp(rint(v / out_scale), -8, 7)
 *   qy [M][N/8]: the codes packed like qx (so that qy is the next call's qx, with sx[m] = out_scale).
 * Needs N % 8 == 0, out_scale > 0; otherwise as qil_linear_w4a4. */
qil_status qil_linear_w4a4_requant(const uint32_t* qx, const float* sx, const uint32_t* qw, const float* sw,
                                   uint32_t* qy, float out_scale, int relu, int M, int N, int K,
                                   void* workspace, size_t workspace_bytes, qil_stream_t stream);

/* 3 x 3 convolution (stride 1, zero padding 1) of the W4A4 conv backbone (the CILRS-style encoder, Sec. 5.1,
 * App. A.1.2) read straight from the int4 feature map, without a materialised im2col matrix: the GEMM's loader
 * computes, for row (b, h, w) and column (3 kh + kw) C + c, the address of channel c of pixel (h + kh - 1, w + kw - 1)
 * or takes zero outside the image.
 *   qx [B][H][W][C/8]   the feature map, NHWC, signed 4-bit codes packed 8 per word along C; one static scale x_scale
 *                       for the whole tensor (the paper's tensor-wise activation setting, App. A.1.2)
 *   qw [Cout][9 C / 8]  filters, column (3 kh + kw) C + c, packed like qx; sw [Cout] fp32 per-filter scales
 * Output, one of (the other pointer null):
 *   y  [B][H][W][Cout] bf16 = float(acc) * (x_scale * sw[n]); acc_out: optional int32 copy of the accumulators;
 *   qy [B][H][W][Cout/8]: the next layer's feature map, quantised in the epilogue as in qil_linear_w4a4_requant
 *      (ReLU if relu, static scale out_scale; Cout % 8 == 0), so that a stack of conv layers never leaves 4 bits.
 * Needs C % 32 == 0 and 9 C < 131072.  workspace: qil_linear_w4a4_workspace_size(B H W, Cout, 9 C) bytes.
 * Errors: NULL (also both or neither output), SHAPE, ALIGN, UNSUPPORTED (out_scale <= 0), WORKSPACE, CUDA. */
qil_status qil_conv3x3_w4a4(const uint32_t* qx, float x_scale, const uint32_t* qw, const float* sw, void* y,
                            int32_t* acc_out, uint32_t* qy, float out_scale, int relu, int B, int H, int W,
                            int C, int Cout, void* workspace, size_t workspace_bytes, qil_stream_t stream);

/* W8A8 integer GEMM (Table "CILRS performance", W8A8 row; Sec. 5.4): as qil_linear_w4a4 with one signed byte per
 * element: qx [M][K], qw [N][K] int8; acc exact in int32 (|acc| <= 2^14 K: K < 131072), K % 16 == 0; the same
 * workspace (qil_linear_w4a4_workspace_size). */
qil_status qil_linear_w8a8(const int8_t* qx, const float* sx, const int8_t* qw, const float* sw, void* y,
                           int32_t* acc_out, int M, int N, int K, void* workspace, size_t workspace_bytes,
                           qil_stream_t stream);

/* A list of independent integer GEMMs in one persistent launch (one CTA per SM walks output tiles of all entries;
 * the conv stages of Sec. 5.1's driving policy are each shorter than the start-up of a kernel).  bits = 4: operands
 * as for qil_linear_w4a4; bits = 8: as for qil_linear_w8a8.  No entry may read another entry's output.  At most 8
 * entries and 1200 output tiles of 128 x 64 per call; larger lists are run entry by entry.  Descriptors are host
 * memory, consumed before the call returns; workspace as for qil_linear_w4a4. */
typedef struct {
    const void* qx;          /* bits 4: packed [M][K/8] uint32; bits 8: int8 [M][K] */
    const float* sx;         /* [M] */
    const void* qw;          /* bits 4: packed [N][K/8]; bits 8: int8 [N][K] */
    const float* sw;         /* [N] */
    void* y;                 /* bf16 [M][N] */
    int32_t* acc_out;        /* optional [M][N] */
    int M, N, K, bits;
} qil_igemm_desc;
qil_status qil_linear_int_batch(const qil_igemm_desc* descs /*host*/, int count, void* workspace,
                                size_t workspace_bytes, qil_stream_t stream);

/* ------------------------------------------------------------------------
 * Helpers
 * ---------------------------------------------------------------------- */
const char* qil_status_string(qil_status s);
int qil_version(void);
/* Copies the device status word to *out (host) and waits for that copy. */
qil_status qil_device_status(const int* dev_status, int* out /*host*/, qil_stream_t stream);
/* Limit of every device-side wait of the streaming list kernel, in nanoseconds, for launches made
 * after the call (process-wide; 0 restores the default of 2 s). */
qil_status qil_set_wait_limit_ns(unsigned long long ns);

/* Measurement helpers (not part of the method): a dense bf16 GEMV
 * y[n] = sum_k x[k] W[n][k] with W bf16 [N][K], the 16-bit baseline the paper's
 * speedups are quoted against (Table "OpenVLA performance"); and a read-only
 * streaming pass over `bytes` bytes that adds every 32-bit word into *sink. */
qil_status qil_ref_gemv_bf16(const void* x, const void* w, void* y, int N, int K, qil_stream_t stream);
qil_status qil_probe_hbm_read(const void* buf, size_t bytes, unsigned int* sink, qil_stream_t stream);
/* Tensor-core roofs: one CTA per SM issues `iters` x 4 tcgen05.mma (128 x 256, K = 32 bytes each) over operand
 * tiles resident in shared memory, kind::i8 resp. kind::f16 with bf16 operands, with a tcgen05.commit every
 * `commit_every` iterations (8 for the roof; 1 shows what a commit per pipeline step costs).  *ops_out (host, optional)
 * receives the operations of the launch (2 per multiply-add); the caller times the launch.  dev_status
 * (device, optional) receives QIL_ERR_TIMEOUT if a bounded wait ran out. */
qil_status qil_probe_mma_i8(int iters, int commit_every, double* ops_out /*host*/, int* dev_status, qil_stream_t stream);
qil_status qil_probe_mma_bf16(int iters, int commit_every, double* ops_out /*host*/, int* dev_status, qil_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* QIL_H_ */
