/*
 * bitlinear.h - C ABI of the B200 (sm_100a) W1.58A8 BitLinear library.
 *
 * The library computes the forward pass of one BitLinear layer of BitNet b1.58
 * (paper Section 2: ternary absmean weights, per-token absmax int8 activations,
 * subln normalisation in front of the projection, no bias; Section 5.1: weights
 * stored packed, four ternary values per byte, unpacked on chip right before the
 * integer matrix product with the 8-bit activations).
 *
 * Conventions for every entry point
 *  - All pointers are DEVICE pointers owned by the caller unless a parameter is
 *    documented as a host pointer.  The library allocates no device memory and
 *    frees none; scratch space is passed in as a workspace.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  Calls only enqueue work on that stream and never synchronise,
 *    except the *_host entry point, which says so.
 *  - Matrices are row-major.  x is [M][K], weights are [N][K] (out x in), y is [M][N].
 *  - Supported shapes: K a multiple of 256 with 256 <= K <= 16384; N a multiple
 *    of 16; M >= 0 (M == 0 is a no-op that returns BITLINEAR_OK).
 *  - Device pointers must be 16-byte aligned.
 *  - Inputs must be finite; NaN/Inf propagate unspecified values but never fault.
 *  - Host-detectable errors are returned before anything is launched.  A failed
 *    launch is reported as BITLINEAR_ERR_CUDA.  Nothing throws, aborts or prints.
 *
 * Numerical definition (bit-exact integer stages; every fp32 operation is one
 * IEEE round-to-nearest-even operation, "Round" is round-half-to-even):
 *   r      = fl32( 1 / sqrt( mean_k(x^2) + rms_eps ) )      (sum of squares in fp64)
 *   yn_k   = fl32( fl32(x_k * r) * g_k )
 *   a      = max( max_k |yn_k|, 1e-5 )
 *   xq_k   = clip( Round( fl32( yn_k * fl32(127 / a) ) ), -128, 127 ),   d = fl32(a / 127)
 *   s_w    = fl32( fl32(mean |W|) + eps_w )                  (mean in fp64)
 *   Wq_nk  = clip( Round( fl32(W_nk / s_w) ), -1, 1 )
 *   acc_mn = sum_k xq_mk * Wq_nk                              (int32, exact)
 *   y_mn   = fl32( fl32( (float)acc_mn * s_w ) * d_m )        (bf16 output: RN-even cast of that)
 *
 * Packed weight layout (2 bits per weight, code c = Wq + 1 in {0,1,2}; 3 is unused)
 *   The [N][K] matrix is cut into tiles of 16 rows x 256 columns, 1024 bytes each,
 *   stored row-block major: tile index = (n / 16) * (K / 256) + (k / 256).
 *   Inside a tile, row r = 8*h + g (h in 0..1, g in 0..7) and column
 *   c = 64*t + 16*i + 4*j + b (t, i, j, b in 0..3) live at
 *       byte  512*h + 64*g + 16*t + 4*i + b,   bits 2*j and 2*j+1.
 *   Hence a 16-byte chunk holds 64 consecutive columns of one row, the 32 lanes of
 *   a warp loading 16 bytes each cover 8 rows x 256 columns of contiguous memory,
 *   a little-endian 32-bit word holds 16 consecutive columns, and
 *   (word >> 2*j) & 0x03030303 yields the codes of four consecutive columns, one
 *   per byte - directly a dot-product-of-four or tensor-core operand.
 *   Kernels accumulate sum_k c*xq and subtract sum_k xq (produced by the
 *   activation quantiser) to recover sum_k Wq*xq.
 *
 * Dense packed weight layout (five ternary values per byte, 1.6 bits per weight; Table 1 of the
 * paper counts the model's memory at about 1.58 bits per weight, and Section 5.1 packs weights
 * to cut the bytes moved per token - the layout itself is this library's)
 *   Byte value: with the codes c_e = Wq + 1 of five weights, digit 0 the most significant,
 *   v = 81*c_0 + 27*c_1 + 9*c_2 + 3*c_3 + c_4 (0..242) and the stored byte is ceil(256 * v / 243),
 *   i.e. the base-3 fraction 0.c_0c_1c_2c_3c_4 scaled to eight bits and rounded up: multiplying the
 *   byte by 3 leaves digit c_0 in bits 8-9 and the fraction of the remaining digits in bits 0-7,
 *   so a decoder peels the digits off with multiplications, no division.  v = floor(243 * B / 256).
 *   Position: K is padded with zero weights to Kp = 320 * ceil(K / 320).  Tiles of 16 rows x 320
 *   columns, 1024 bytes each, row-block major: tile index = (n / 16) * (Kp / 320) + (k / 320).
 *   Inside a tile, row r = 8*h + g and column c = 80*t + 20*i + 4*e + b (t, i, b in 0..3,
 *   e in 0..4) live at byte 512*h + 64*g + 16*t + 4*i + b, base-3 digit e.  Hence a 16-byte chunk
 *   holds 80 consecutive columns of one row, a 32-bit word 20 consecutive columns, and digit e
 *   of the four bytes of a word belongs to four consecutive columns - one dot-product-of-four.
 *   Size: N * Kp / 5 bytes: 418.8 MB for the 210 matrices of the 2B model against 521.0 MB at
 *   four per byte.
 */
#ifndef BITLINEAR_H_
#define BITLINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BITLINEAR_OK = 0,
    BITLINEAR_ERR_NULL = 1,      /* a required pointer is NULL */
    BITLINEAR_ERR_SHAPE = 2,     /* unsupported M, N or K */
    BITLINEAR_ERR_ALIGN = 3,     /* a pointer is not 16-byte aligned */
    BITLINEAR_ERR_WORKSPACE = 4, /* workspace missing or too small */
    BITLINEAR_ERR_DTYPE = 5,     /* unknown dtype code */
    BITLINEAR_ERR_ARCH = 6,      /* the current device is not compute capability 10.x */
    BITLINEAR_ERR_CUDA = 7,      /* a CUDA runtime call or a launch failed */
    BITLINEAR_ERR_TIMEOUT = 8    /* a bounded device-side wait ran out (see bitlinear_poll_status) */
} bitlinear_status;

/* dtype codes */
#define BITLINEAR_F32 0
#define BITLINEAR_BF16 1

/* Layout of a packed weight matrix (field w_format of bitlinear_problem). */
#define BITLINEAR_WEIGHTS_2BIT 0   /* four values per byte, from bitlinear_pack_weights */
#define BITLINEAR_WEIGHTS_DENSE5 1 /* five values per byte, from bitlinear_pack_weights5 */

/* Which contraction kernel bitlinear_matmul_q / bitlinear_forward use. */
#define BITLINEAR_PATH_AUTO 0  /* decode kernel for M <= 16, tensor-core kernel above */
#define BITLINEAR_PATH_GEMV 1  /* force the streaming decode kernel (any M, in chunks of 16 tokens) */
#define BITLINEAR_PATH_GEMM 2  /* force the tcgen05 tensor-core kernel (needs N % 128 == 0) */

/* Human-readable name of a status code (static storage, never NULL). */
const char* bitlinear_status_string(int status);

/* Library version, major*10000 + minor*100 + patch. */
int bitlinear_version(void);

/* Bytes of the packed form of an [N][K] ternary matrix: N*K/4 (Section 5.1: four values per
 * byte).  Returns 0 for an unsupported shape. */
size_t bitlinear_packed_bytes(int N, int K);

/* Workspace bytes bitlinear_pack_weights needs for an [N][K] matrix (fp64 partial sums of the
 * absmean reduction).  Returns 0 for an unsupported shape. */
size_t bitlinear_pack_workspace_bytes(int N, int K);

/* Workspace bytes bitlinear_forward needs: int8 activations [M][K], the per-token scale and
 * code sum, and, when the tensor-core path can be taken (M > 16 or a forced path), the scratch
 * of bitlinear_matmul_workspace_bytes.  Returns 0 for an unsupported shape. */
size_t bitlinear_workspace_bytes(int M, int N, int K);

/* Workspace bytes bitlinear_matmul_q needs: for the tensor-core path one byte per weight (the
 * codes 0/1/2 expanded into the shared-memory images of the kernel's 256 x 128 tiles, N rounded up
 * to whole tiles) plus a small launch table; 0 when only the decode kernel can be taken, i.e.
 * M <= 16 and path AUTO or GEMV. */
size_t bitlinear_matmul_workspace_bytes(int M, int N, int K, int path);

/*
 * Offline weight quantiser and packer (Section 2, "Weight Quantization": absmean scheme onto
 * {-1,0,+1}; Section 5.1: four ternary values per byte kept in HBM).
 *   W          in : [N][K] master weights, fp32 (w_dtype 0) or bf16 (w_dtype 1).
 *   eps_w      in : added to mean|W| to form the scale s_w.
 *   packed_out out: bitlinear_packed_bytes(N,K) bytes in the layout described above.
 *   s_w_out    out: one fp32 on the device, the dequantisation scale mean|W| + eps_w.
 *   ws / ws_bytes : scratch of at least bitlinear_pack_workspace_bytes(N,K).
 * The reduction order is fixed, so the result is deterministic run to run.
 */
int bitlinear_pack_weights(const void* W, int w_dtype, int N, int K, float eps_w, void* packed_out,
                           float* s_w_out, void* ws, size_t ws_bytes, void* stream);

/* Test hook: expand a packed matrix back to int8 values in {-1,0,1}, [N][K] row-major. */
int bitlinear_unpack_weights(const void* packed, int N, int K, int8_t* wq_out, void* stream);

/*
 * The same quantiser writing the dense layout, five ternary values per byte (Table 1: about 1.58
 * bits per weight; Section 5.1: packing exists to move fewer bytes).  Arguments as
 * bitlinear_pack_weights; packed5_out holds bitlinear_packed5_bytes(N,K) = N * Kp / 5 bytes,
 * Kp = K rounded up to a multiple of 320 (0 for an unsupported shape).  The scale and the ternary
 * values are identical to those of bitlinear_pack_weights; only the storage differs.  Dense
 * matrices are consumed by bitlinear_forward_batch (w_format = BITLINEAR_WEIGHTS_DENSE5) for
 * problems of at most 16 tokens.
 */
size_t bitlinear_packed5_bytes(int N, int K);
int bitlinear_pack_weights5(const void* W, int w_dtype, int N, int K, float eps_w, void* packed5_out,
                            float* s_w_out, void* ws, size_t ws_bytes, void* stream);
/* Test hook: expand a dense matrix back to int8 values in {-1,0,1}, [N][K] row-major (padding dropped). */
int bitlinear_unpack_weights5(const void* packed5, int N, int K, int8_t* wq_out, void* stream);

/*
 * Fused RMSNorm + per-token absmax int8 quantiser (Section 2, "Activation Quantization" and
 * "Normalization": the subln norm feeding each BitLinear, 8-bit absmax per token).
 *   x_bf16   in : [M][K] bf16.
 *   gain     in : [K] bf16 RMSNorm gain, or NULL for all ones.
 *   xq_out   out: [M][K] int8 codes.
 *   d_out    out: [M] fp32 dequantisation scale a/127 of each token.
 *   xsum_out out: [M] int32 sum of each token's codes (the contraction kernels need it); nullable.
 */
int bitlinear_quant_act(const void* x_bf16, const void* gain, float rms_eps, int M, int K,
                        int8_t* xq_out, float* d_out, int32_t* xsum_out, void* stream);

/*
 * The same quantiser with the squared-ReLU gate of the feed-forward block in front (Section 2: ReLU^2 replaces SwiGLU;
 * the down projection is a BitLinear, so its subln norm and its 8-bit quantiser follow the gate directly).  One launch
 * computes f = bf16( fl32( fl32(r * r) * up ) ), r = max(gate, 0), and quantises f exactly as bitlinear_quant_act does.
 *   gate, up   in : [M][F] fp32 (outputs of the gate and up projections).
 *   x_out_bf16 out: nullable; [M][F] bf16, receives f.
 *   gain, xq_out, d_out, xsum_out: as in bitlinear_quant_act, with K = F.
 */
int bitlinear_quant_act_relu2(const float* gate, const float* up, const void* gain, float rms_eps, int M, int F,
                              void* x_out_bf16, int8_t* xq_out, float* d_out, int32_t* xsum_out, void* stream);

/*
 * Ternary x int8 contraction over packed weights with the dequantising epilogue
 * (Section 5.1: packed weights are loaded from HBM, unpacked on chip and multiplied with the
 * 8-bit activations; Section 2 fixes the two scales the epilogue undoes).
 *   xq, d, xsum in : outputs of bitlinear_quant_act (all three required).
 *   packed, s_w in : outputs of bitlinear_pack_weights (s_w on the device).
 *   y_out      out : [M][N] fp32 (y_dtype 0) or bf16 (y_dtype 1).
 *   acc_out    out : nullable; [M][N] int32 raw accumulators sum_k xq*Wq, for parity checks.
 *   path           : BITLINEAR_PATH_*.
 *   ws / ws_bytes  : scratch of at least bitlinear_matmul_workspace_bytes(M,N,K,path); may be
 *                    NULL when that is 0.
 */
int bitlinear_matmul_q(const int8_t* xq, const float* d, const int32_t* xsum, const void* packed,
                       const float* s_w, int M, int N, int K, void* y_out, int y_dtype,
                       int32_t* acc_out, int path, void* ws, size_t ws_bytes, void* stream);

/*
 * The whole BitLinear forward: bitlinear_quant_act followed by bitlinear_matmul_q (path AUTO)
 * on the same stream (Section 2: norm -> activation quantiser -> W1.58A8 product -> rescale).
 * At one token the two steps are one launch (every CTA quantises the row while its share of the
 * packed weights is on its way from HBM); the result is the same, bit for bit.
 *   ws / ws_bytes : scratch of at least bitlinear_workspace_bytes(M,N,K).
 */
int bitlinear_forward(const void* x_bf16, const void* gain, float rms_eps, const void* packed,
                      const float* s_w, int M, int N, int K, void* y_out, int y_dtype, void* ws,
                      size_t ws_bytes, void* stream);

/*
 * The BitLinear forward as it runs in training (Section 2: the weights are quantised to 1.58 bits during the forward
 * pass; Section 1: the released bf16 checkpoint is the master weight, used for training only): the absmean scale and
 * the ternary codes are formed from the master weights on the fly, then the forward above runs on them.
 *   W, w_dtype  in : master weights [N][K] row-major, BITLINEAR_F32 or BITLINEAR_BF16, device, 16-byte aligned.
 *   eps_w       in : added to mean|W| to form the scale.
 *   packed_out out : nullable; bitlinear_packed_bytes(N,K) bytes: the packed weights this call used (byte for byte what
 *                    bitlinear_pack_weights writes - the inference artefact of the same step).
 *   s_w_out    out : nullable; one fp32 on the device, the scale.
 *   ws / ws_bytes  : device scratch of at least bitlinear_forward_master_workspace_bytes(M,N,K) (0 for an
 *                    unsupported shape); holds the reduction partials, the packed weights and the forward's scratch.
 * Three steps on `stream`: the absmean reduction (fixed order, deterministic), the quantise-and-pack pass, the forward.
 * Everything else as bitlinear_forward.  The backward pass is not part of this library (the paper does not describe it).
 */
size_t bitlinear_forward_master_workspace_bytes(int M, int N, int K);
int bitlinear_forward_master(const void* x_bf16, const void* gain, float rms_eps, const void* W, int w_dtype, float eps_w,
                             int M, int N, int K, void* y_out, int y_dtype, void* packed_out, float* s_w_out, void* ws,
                             size_t ws_bytes, void* stream);

/*
 * bitlinear_forward for callers whose activations live in HOST memory: copies x (host, ideally
 * pinned) into the workspace, runs the forward, copies y back to the host buffer and
 * SYNCHRONISES the stream before returning.
 *   x_host  in : host pointer, [M][K] bf16.      y_host out: host pointer, [M][N] of y_dtype.
 *   gain, packed, s_w, ws: device pointers as in bitlinear_forward;
 *   ws_bytes >= bitlinear_workspace_bytes(M,N,K) + bitlinear_host_staging_bytes(M,N,K,y_dtype).
 */
size_t bitlinear_host_staging_bytes(int M, int N, int K, int y_dtype);
int bitlinear_forward_host(const void* x_host, const void* gain, float rms_eps, const void* packed,
                           const float* s_w, int M, int N, int K, void* y_host, int y_dtype, void* ws,
                           size_t ws_bytes, void* stream);

/*
 * Batched forward: `count` independent BitLinear forwards in a handful of launches.
 *
 * Problems of at most 16 tokens (the decode regime of Section 5.1, where the cost is the packed
 * weight bytes streamed from HBM) take two launches together: one fused RMSNorm+quantiser launch
 * over every token, then one persistent kernel that streams the packed weights of all of them
 * back to back (dot-products-of-four when every such problem has one token; int8 mma.sync fed
 * from the same stream when none has more than 8; otherwise tcgen05, with the codes unpacked in
 * registers and handed over in tensor memory).  A call whose
 * problems all have one token and read the same input row the same way - a level of a decoder
 * layer: q/k/v, o, gate/up or down - is ONE launch: every CTA quantises the row itself while its
 * share of the packed weights is on its way (up to four problems in the 2-bit layout; otherwise the
 * streaming kernel without a quantiser launch in front).  Problems of 17 to
 * 96 tokens (K <= 8192) are cut into 16-token problems for that same decode kernel: streaming the
 * packed weights once per 16 tokens is measured faster there than a tensor-core tile that is mostly
 * padding.  Longer problems (prefill; N must be a multiple of 128) take two launches together: the
 * quantiser and one persistent tcgen05 kernel that runs every tile of every matmul and expands the
 * packed weights into tensor-core tile images in shared memory as it goes (on a device with an odd
 * number of SMs, where CTA pairs cannot cover the chip, a separate expansion launch into ws comes
 * first); problems that name the same x, gain, rms_eps, M and K (q/k/v or gate/up of a layer) share
 * one quantised copy.
 * All kinds may be mixed in one call.
 * Weights in the dense layout (w_format = BITLINEAR_WEIGHTS_DENSE5, Table 1 / Section 5.1) are accepted for
 * problems of at most 16 tokens; all such problems of a call must use the same layout.  Their kernel is the
 * one-token streaming kernel with the base-3 digits peeled off in registers; a problem of M tokens streams its
 * weights M times, so this layout trades speed at M > 1 for 20 % less memory.
 *   problems : HOST array of `count` descriptors; the pointers inside are DEVICE pointers with the
 *              meaning, layout and alignment of the bitlinear_forward arguments.  K <= 8192 for
 *              problems of at most 16 tokens.  Problems with M == 0 are skipped.  Outputs must not
 *              alias inputs of other problems of the same call (they run concurrently).
 *   flags    : 0, or an OR of BITLINEAR_BATCH_REUSE_PLAN (the previous call on this workspace had
 *              exactly the same descriptors, and the packed weights, their scales and the gains
 *              have not been written since - the steady state of a decode loop: skips
 *              re-uploading the decode plan and, when the library still remembers what it derived
 *              from these descriptors for this workspace (a small per-process table keyed by the
 *              workspace address and a hash of the descriptors), planning on the host altogether;
 *              and a call that is a single launch (one token, one
 *              shared input row) may begin fetching weights while the launch before it on the
 *              stream is still running) and
 *              BITLINEAR_BATCH_REUSE_ACT (the inputs are unchanged as well: skips the quantiser
 *              launches and reuses their results in ws), BITLINEAR_BATCH_REUSE_WEIGHTS (same
 *              descriptors and same packed matrices: skips the expansion of the prefill problems).
 *   ws       : device scratch of at least bitlinear_batch_workspace_bytes(problems, count); it
 *              holds the uploaded plan, the quantised activations and the expanded weights of the
 *              prefill problems, so a call must not overlap another call that uses the same
 *              workspace.
 */
typedef struct bitlinear_problem {
    const void* x;      /* [M][K] bf16 (another operand where x_op says so) */
    const void* gain;   /* [K] bf16 or NULL */
    const void* packed; /* packed weights of an [N][K] matrix */
    const float* s_w;   /* its scale */
    void* y;            /* [M][N] */
    int M, N, K;
    int y_dtype;        /* BITLINEAR_F32 or BITLINEAR_BF16 */
    float rms_eps;
    int w_format;       /* layout of `packed`: BITLINEAR_WEIGHTS_2BIT (0) or BITLINEAR_WEIGHTS_DENSE5 (1) */
    /* The element-wise step of a decoder layer that sits in front of this BitLinear, fused into its quantiser launch
     * (Section 2: squared-ReLU feed-forward block, residual connections; the subln norm then applies to the result).
     * Same arithmetic as the bitlinear_glue_* calls below: one fp32 operation per step, one bf16 rounding.
     *   BITLINEAR_X_PLAIN (0)        x is the input, bf16 [M][K]; x2 and x_out are ignored.
     *   BITLINEAR_X_RELU2 (1)        x = gate, x2 = up, both fp32 [M][K]:   input = bf16(max(gate,0)^2 * up)
     *   BITLINEAR_X_RESIDUAL (2)     x = h bf16 [M][K], x2 = y fp32 [M][K]: input = bf16(h + y)
     *   BITLINEAR_X_ATTN_STANDIN (3) x = q fp32 [M][K], x2 = v fp32 [M][K / x_arg1], x_arg0 = head_dim (a multiple
     *                                of 8), x_arg1 = query heads per KV head: input = q + v of the matching KV head
     *                                (a stand-in for attention, which is not a BitLinear)
     * x_out: nullable bf16 [M][K] that receives the input so formed (the new hidden state after a residual); it must
     * not alias x.  Problems of a call that name the same x, x2, x_op, gain, rms_eps, M and K share one quantised copy. */
    int x_op;
    int x_arg0, x_arg1;
    int reserved;       /* set to 0 */
    const void* x2;
    void* x_out;
} bitlinear_problem;

#define BITLINEAR_X_PLAIN 0
#define BITLINEAR_X_RELU2 1
#define BITLINEAR_X_RESIDUAL 2
#define BITLINEAR_X_ATTN_STANDIN 3

#define BITLINEAR_BATCH_REUSE_PLAN 1 /* descriptors unchanged since the previous call on this workspace */
#define BITLINEAR_BATCH_REUSE_ACT 2  /* inputs x unchanged too: skip the quantiser launch, reuse its results in ws */
#define BITLINEAR_BATCH_REUSE_WEIGHTS 4 /* same packed matrices as the previous call on this workspace: the byte codes the
                                           prefill problems were expanded to are still in ws and are not expanded again
                                           (prefill is compute-bound: a caller with memory to spare keeps one workspace
                                           per layer and pays the expansion once, not per call) */

size_t bitlinear_batch_workspace_bytes(const bitlinear_problem* problems, int count);
int bitlinear_forward_batch(const bitlinear_problem* problems, int count, int flags, void* ws, size_t ws_bytes,
                            void* stream);

/*
 * Parity hook: bitlinear_forward_batch that also stores the raw int32 accumulators sum_k xq*Wq of the contraction
 * (Section 5.1: the integer product of unpacked ternary weights and 8-bit activations).
 *   acc_out : HOST array of `count` DEVICE pointers, entry i nullable or [M][N] int32 for problem i.
 * Available where the persistent streaming kernels run the problem: calls in the 2-bit layout whose decode-sized
 * problems all have at most 8 tokens, and problems of up to 16 tokens in the dense layout; BITLINEAR_ERR_SHAPE for a
 * non-NULL entry anywhere else.
 */
int bitlinear_forward_batch_acc(const bitlinear_problem* problems, int count, int flags, int32_t* const* acc_out,
                                void* ws, size_t ws_bytes, void* stream);

/*
 * bitlinear_forward_batch for callers whose activations live in HOST memory.  The x pointers of the
 * descriptors point into one device arena x_dev and the y pointers into one device arena y_dev;
 * the call copies x_host (host, ideally pinned, x_bytes) into x_dev, runs the batch, copies y_dev
 * (y_bytes) into y_host and SYNCHRONISES the stream before returning.
 * A call of at least 24 decode-sized problems (M <= 16, plain inputs) whose operands lie in both arenas in the order
 * of the problems runs as three segments of about equal packed bytes, two of them on streams of the library's own
 * (created on first use, one set per device) that start after the caller's earlier work and that the caller's stream
 * waits for: one segment's copies then run beside another's kernels.  Every byte of both arenas is still copied
 * exactly once and the results are those of the unsegmented call.  Each segment keeps its own plan in its slice of ws
 * (bitlinear_batch_workspace_bytes covers that), so BITLINEAR_BATCH_REUSE_PLAN here refers to an earlier call of
 * THIS function on the same ws, not to an earlier bitlinear_forward_batch.
 */
int bitlinear_forward_batch_host(const bitlinear_problem* problems, int count, int flags, const void* x_host,
                                 void* x_dev, size_t x_bytes, const void* y_dev, void* y_host, size_t y_bytes,
                                 void* ws, size_t ws_bytes, void* stream);

/*
 * Element-wise glue between the BitLinear matmuls of a decoder layer, for chained decode runs (Section 2: squared
 * ReLU replaces SwiGLU in the feed-forward block; residual connections of the Transformer).  Inputs that come out of
 * a BitLinear are fp32 [M][*]; every result is rounded once to bf16 (round to nearest even) because it feeds the next
 * BitLinear.  Each arithmetic step is one fp32 operation.
 *   relu2_mul    : u = bf16( fl32( fl32(r*r) * up ) ), r = max(gate, 0);          gate, up [M][F] -> u [M][F]
 *   residual_add : h = bf16( fl32( float(h) + y ) ) in place;                       h bf16 [M][N], y fp32 [M][N]
 *   attn_standin : NOT attention (attention is not a BitLinear and is outside this library): a fixed mixing of the
 *                  q and v projections that keeps the data dependence of a layer,
 *                  o_in[m][h*D + j] = bf16( fl32( q[m][h*D + j] + v[m][(h / (n_q/n_kv))*D + j] ) ).
 */
int bitlinear_glue_relu2_mul(const float* gate, const float* up, void* u_bf16, int M, int F, void* stream);
int bitlinear_glue_residual_add(void* h_bf16, const float* y, int M, int N, void* stream);
int bitlinear_glue_attn_standin(const float* q, const float* v, void* o_in_bf16, int M, int n_q_heads, int n_kv_heads,
                                int head_dim, void* stream);

/*
 * One decoded token through a stack of decoder layers in ONE persistent cooperative kernel (Section 2: every linear
 * map of a layer is a BitLinear; squared-ReLU feed-forward block; Section 5.1: decode is bound by the packed weight
 * bytes).  Per layer, with the glue steps defined above:
 *     q,k,v = BitLinear(h);  a = attn_standin(q, v);  h = residual_add(h, BitLinear_o(a));
 *     g,u   = BitLinear_gate/up(h);  f = relu2_mul(g, u);  h = residual_add(h, BitLinear_down(f)).
 * The result is bit-identical to issuing those calls one by one.  The kernel keeps every SM busy for the whole token:
 * a level's weight rows are split over the SMs, prefetched into shared memory one level ahead, and levels are
 * separated by grid barriers instead of kernel boundaries.
 *   layers   : HOST array of n_layers descriptors; pointers inside are DEVICE pointers: packed / s_w of the seven
 *              matrices in the order q,k,v,o,gate,up,down, and the bf16 RMSNorm gains of the four BitLinear inputs
 *              (of {q,k,v}, o, {gate,up}, down; NULL = ones).
 *   dims     : hidden = n_q_heads * head_dim; head_dim a multiple of 4; hidden and ffn multiples of 256, at most
 *              8192; one token.
 *   h_bf16   : [hidden] bf16, in and out.      k_out : nullable, [n_kv_heads*head_dim] fp32, the last layer's k.
 *   flags    : 0 or BITLINEAR_BATCH_REUSE_PLAN (the layer table uploaded by the previous call on ws is still valid).
 *   ws       : at least bitlinear_decode_chain_workspace_bytes(...); calls on one workspace must not overlap.
 * Needs a device that supports cooperative launches with one CTA per SM free (else BITLINEAR_ERR_CUDA).
 */
typedef struct bitlinear_chain_layer {
    const void* packed[7];
    const float* s_w[7];
    const void* gain[4];
} bitlinear_chain_layer;
size_t bitlinear_decode_chain_workspace_bytes(int n_layers, int hidden, int ffn, int n_q_heads, int n_kv_heads,
                                              int head_dim);
int bitlinear_decode_chain(const bitlinear_chain_layer* layers, int n_layers, int hidden, int ffn, int n_q_heads,
                           int n_kv_heads, int head_dim, float rms_eps, void* h_bf16, float* k_out, int flags, void* ws,
                           size_t ws_bytes, void* stream);

/*
 * bitlinear_forward for decode-sized calls by code that cannot allocate device memory.
 * (No counterpart in the paper: this is a convenience of the library.)
 *
 * Who needs it: an operator plug-in that receives only its input and output buffers, code that
 * runs after a framework's pool has claimed the whole device, a serving loop whose steady state
 * must not touch an allocator.  Such callers cannot provide the workspace bitlinear_forward asks
 * for, and the library itself never calls cudaMalloc.  Here the workspace is a fixed array inside
 * the library image instead: bitlinear_static_scratch_bytes() bytes (262,656) that every GPU which
 * loads the library holds until the process exits.  The call allocates and frees nothing.
 *
 *   Arguments as bitlinear_forward, without ws.  Limits: M <= BITLINEAR_STATIC_MAX_TOKENS and
 *   K <= BITLINEAR_STATIC_MAX_K; anything larger returns BITLINEAR_ERR_WORKSPACE before a launch.
 *   The result is the same as bitlinear_forward's for the same arguments (same kernels).
 *   The first call on each device looks up the array's device address (with that device current)
 *   and caches it; make that first call outside any stream capture.
 *   All calls on a device share the one array.  Each call rewrites every element it later reads,
 *   so leftovers of earlier calls are harmless, but two calls that overlap on the GPU (different
 *   streams, no ordering between them) race on it: serialise them.
 */
#define BITLINEAR_STATIC_MAX_TOKENS 16
#define BITLINEAR_STATIC_MAX_K 16384
size_t bitlinear_static_scratch_bytes(void);
int bitlinear_forward_static(const void* x_bf16, const void* gain, float rms_eps, const void* packed,
                             const float* s_w, int M, int N, int K, void* y_out, int y_dtype, void* stream);

/* Reads and clears the sticky device-side status word of the current device: BITLINEAR_OK,
 * BITLINEAR_ERR_TIMEOUT if a kernel gave up a bounded wait since the last poll, or
 * BITLINEAR_ERR_WORKSPACE if a batch call with BITLINEAR_BATCH_REUSE_PLAN found that the plan in
 * its workspace was no longer the one it had uploaded (the call then computed nothing).
 * Synchronises `stream` first. */
int bitlinear_poll_status(void* stream);

/*
 * The rest of a decode step around the BitLinear layers.  The paper names these parts without formulas (Section 2:
 * rotary position embeddings; a Transformer decoder; a tokenizer with 128,256 entries, hence an embedding table and an
 * output head of that many rows); the definitions taken are the textbook ones, stated here.  None is a BitLinear: they
 * exist so that a whole decoded token can be run and timed on the device.
 *
 * bitlinear_rope_kv: rotary embedding of the q and k projections and append of k, v to the cache.
 *   q [M][n_q*D], k, v [M][n_kv*D] fp32 (BitLinear outputs); positions [M] int32 (device); seq_ids [M] int32 (device)
 *   or NULL (one sequence).  Coordinate i of a head is paired with i + D/2, angle = position * rope_base^(-2i/D):
 *   (x_i, x_j) -> (x_i cos - x_j sin, x_j cos + x_i sin); angles in fp64, rotation in fp32, results rounded to bf16.
 *   q_out bf16 [M][n_q*D]; caches bf16 [n_seq][n_kv][t_max][D] (the rows of one KV head of one sequence are
 *   contiguous, so that attention streams a head's keys as one run of memory): row positions[m] of every head of
 *   sequence seq_ids[m] receives the rotated k and the unrotated v (positions outside 0 .. t_max-1 and sequences
 *   outside 0 .. n_seq-1 are not stored).  D a multiple of 8.
 * bitlinear_attention_decode: one query token per row against the first lengths[m] cache rows of its sequence.
 *   Query head h reads key/value head h / (n_q / n_kv); scores q.k / sqrt(D), softmax over the rows, weighted sum of
 *   the values, fp32 arithmetic, bf16 output [M][n_q*D] (the input of the o projection; zeros for a length <= 0 or
 *   a sequence outside 0 .. n_seq-1, lengths above t_max are taken as t_max).  D = 64 or 128, n_q / n_kv <= 8,
 *   n_seq * n_kv * t_max <= 2^30, M <= 65535, all pointers 16-byte aligned; the caches are read through tensor maps
 *   encoded per call from their addresses and n_seq, t_max.  ws (device, 16-byte aligned, contents need not
 *   survive the call) at least bitlinear_attention_workspace_bytes(...) bytes (0 for unsupported sizes): up to 64
 *   partial results per token and query head.
 *   A copy that does not land within the wait limit ends the call's kernels and sets BITLINEAR_ERR_TIMEOUT in the
 *   status word (bitlinear_poll_status).
 * bitlinear_rope_table: table_out (device, fp32 [t_max][D/2][2], 16-byte aligned) receives (cos, sin) of
 *   position * rope_base^(-2i/D) for every cache position and pair i, from the same fp64 angle as bitlinear_rope_kv.
 *   D = 64 or 128.  Built once per (rope_base, D, t_max).
 * bitlinear_attention_decode_append: bitlinear_rope_kv followed by bitlinear_attention_decode in the attention
 *   launches themselves (one launch per layer fewer), for the usual decode step in which token m is the newest row
 *   of its sequence: its position is lengths[m] - 1.  q, k, v fp32 as for bitlinear_rope_kv (16-byte aligned);
 *   rope_table from bitlinear_rope_table with the same D and a t_max at least this call's; the caches receive the
 *   rotated k and the unrotated v at row lengths[m] - 1 (the same bits bitlinear_rope_kv stores) and the token
 *   attends to rows 0 .. lengths[m] - 1, its own included; out as for bitlinear_attention_decode, the same bits as the
 *   two-call route.  A length outside 1 .. t_max or a sequence outside 0 .. n_seq-1 stores nothing and gives a zero
 *   row.  The tokens of one call must belong to DIFFERENT sequences (a token does not see rows stored by another
 *   token of the same call; use the two-call route for that); this is not checked.  Other limits, the workspace and
 *   the status word as for bitlinear_attention_decode.
 * bitlinear_lm_head: logits[m][v] = sum_k x[m][k] * table[v][k], x bf16 [M][K] (M <= 16), table bf16 [V][K], fp32
 *   accumulation and output [M][V].  The table is streamed once per call (bf16 tensor-core products, which are exact,
 *   accumulated in fp32).  K a multiple of 8; x is staged in shared memory, so K <= 7168 (BITLINEAR_ERR_SHAPE beyond).
 * bitlinear_embed: out[m] = table[ids[m]] (bf16 rows; ids outside 0 .. V-1 are clamped).
 */
int bitlinear_rope_kv(const float* q, const float* k, const float* v, const int32_t* positions, const int32_t* seq_ids, int M,
                      int n_q_heads, int n_kv_heads, int head_dim, float rope_base, void* q_out_bf16, void* k_cache_bf16,
                      void* v_cache_bf16, int n_seq, int t_max, void* stream);
size_t bitlinear_attention_workspace_bytes(int M, int n_q_heads, int n_kv_heads, int head_dim, int t_max);
int bitlinear_attention_decode(const void* q_bf16, const void* k_cache_bf16, const void* v_cache_bf16, const int32_t* lengths,
                               const int32_t* seq_ids, int M, int n_q_heads, int n_kv_heads, int head_dim, int n_seq, int t_max,
                               void* out_bf16, void* ws, size_t ws_bytes, void* stream);
int bitlinear_rope_table(float rope_base, int head_dim, int t_max, float* table_out, void* stream);
int bitlinear_attention_decode_append(const float* q, const float* k, const float* v, const float* rope_table, void* k_cache_bf16,
                                      void* v_cache_bf16, const int32_t* lengths, const int32_t* seq_ids, int M, int n_q_heads,
                                      int n_kv_heads, int head_dim, int n_seq, int t_max, void* out_bf16, void* ws, size_t ws_bytes,
                                      void* stream);
int bitlinear_lm_head(const void* x_bf16, const void* table_bf16, int M, int V, int K, float* logits, void* stream);
int bitlinear_embed(const int32_t* ids, const void* table_bf16, int M, int V, int K, void* out_bf16, void* stream);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper: every kernel of this library waits on
 * barriers - for copies, for other warps, for other CTAs - and every such wait has a time limit, 2 s in production).
 * Launches one small CTA that waits, with a limit of limit_us microseconds (1 .. 100000), on a barrier nobody arrives
 * on.  The kernel gives up by itself, the context stays usable, and the next bitlinear_poll_status reports
 * BITLINEAR_ERR_TIMEOUT once.  Nothing else is touched.
 */
int bitlinear_selftest_wait_timeout(unsigned limit_us, void* stream);

/*
 * Measurement aid (no counterpart in the paper): the rate at which this GPU executes the int8 tensor-core
 * instruction the prefill contraction is made of.  Launches, on every SM, n_mma_per_sm (1 .. 4,000,000)
 * tcgen05.mma kind::i8 operations of 128 x 256 x 32 on operands that stay in shared memory - no global traffic, no
 * epilogue - and returns at once; *ops_out (HOST pointer, nullable) receives the integer operations of the launch,
 * 2 per multiply-accumulate.  Time the launch with events on `stream`: operations / time is the int8 peak the
 * benchmark reports prefill fractions against.
 */
int bitlinear_probe_int8_mma_rate(int n_mma_per_sm, double* ops_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BITLINEAR_H_ */
