/*
 * goq.h - C ABI of libgoq: the linear-layer inner product against dual-basis Power-of-Two
 * (PoT) weights of GoQuant (arxiv 2605.26092), hand-written CUDA for sm_100a.
 *
 * A weight row is cut into macro-blocks ("groups") of `group` consecutive input channels
 * (paper Section 3.1, N = 128 there). Each group is stored as
 *      w_hat = c1 * b1 + c2 * b2,   <b1, b2> = 0                        (Section 3.1)
 *   b1  one `wbits`-bit PoT code per weight on the asymmetric lattice of Section 3.2
 *       (code c: sign = c >> (wbits-1), e = c & emax, emax = 2^(wbits-1) - 1,
 *        value = (-1)^sign 2^-e, except c == emax which is 0);
 *   b2  never stored: a 6-bit record per 8 weights (2-bit pattern s-1, four pair-sign flags)
 *       tells how to derive it from b1 by the Strided Dual-Exchange of Section 3.3, Theorem 1:
 *       for each pair (i, j = i XOR s), i < j:  y_i = -eta x_j,  y_j = eta x_i.
 *       Record byte: bits[1:0] = s-1; bit 2+p = 1 iff eta of the p-th pair (pairs in ascending
 *       order of their lower index) is -1;
 *   c1, c2  one fp16 pair per (row, group) (Section 3.4).
 *
 * The layer itself is Eq. 4 of Section 3.5 read per group:
 *      y[m,n] = sum_j ( c1[n,j] * sum_{k in j} b1[n,k] x[m,k] + c2[n,j] * sum_{k in j} b2[n,k] x[m,k] )
 * The two inner sums use PoT operands only; the coefficient multiply sits outside them.
 *
 * Conventions for every call
 *   - W is [n_out][k_in] (row n = output channel). k_in % group == 0, group % 8 == 0.
 *   - All pointers are DEVICE pointers unless a parameter says "host". The caller owns every
 *     buffer; the library allocates nothing, frees nothing and keeps no pointer after return.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream). Calls enqueue work
 *     and return; they do not synchronise.
 *   - Argument errors are found on the host before any launch and returned as a status; nothing
 *     is printed, nothing aborts. A failed launch returns GOQ_ERR_CUDA.
 *   - The library runs on compute capability 10.x only (GOQ_ERR_ARCH otherwise). There is no
 *     CPU path.
 */
#ifndef GOQ_H
#define GOQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GOQ_OK = 0,
    GOQ_ERR_INVALID_ARG = 1,    /* NULL pointer, bad size, bad enum */
    GOQ_ERR_UNSUPPORTED = 2,    /* valid request this build has no kernel for */
    GOQ_ERR_ALIGNMENT = 3,      /* pointer not aligned as documented */
    GOQ_ERR_WORKSPACE = 4,      /* workspace or output buffer too small */
    GOQ_ERR_OVERFLOW_BOUND = 5, /* integer path: static int32 bound k_in*127*127*2^emax exceeded */
    GOQ_ERR_ARCH = 6,           /* current device is not sm_100 */
    GOQ_ERR_CUDA = 7,           /* CUDA runtime reported an error */
    GOQ_ERR_TIMEOUT = 8         /* a bounded device-side wait expired (reported through a status word) */
} goq_status;

typedef enum { GOQ_BF16 = 0, GOQ_F32 = 1, GOQ_I8 = 2 } goq_dtype;
typedef enum { GOQ_OP_GEMV = 0, GOQ_OP_GEMM = 1 } goq_op;

#define GOQ_LAYOUT_TILE16 1 /* dual-basis weights w_hat = c1 b1 + c2 b2; see goq_pack */
/* Single-basis weights w_hat = c1 b1 (Section 3.1, the K = 1 row of the basis-dimension ablation) in the same packed
 * format: goq_pack and goq_quantize_geo store zero records and c2 = 0, so every kernel evaluates c1 b1, and the decode
 * GEMV skips the second basis altogether (algorithmic bits per weight: wbits + 16/group). */
#define GOQ_LAYOUT_TILE16_K1 2

typedef struct {
    int32_t n_out;  /* output channels N */
    int32_t k_in;   /* input channels K */
    int32_t group;  /* macro-block size g: multiple of 8 that divides 128, or 128 (8,16,32,64,128) */
    int32_t wbits;  /* 2, 3 or 4 */
    int32_t layout; /* GOQ_LAYOUT_TILE16 or GOQ_LAYOUT_TILE16_K1 */
} goq_desc;

/* Text for a status code (static string, never NULL). */
const char* goq_status_string(goq_status s);

/* Bytes of the packed buffer for this descriptor; 0 if the descriptor is invalid.
 * Storage arithmetic of Section 3.3 step 3 (6 record bits per 8 weights) plus codes and coefficients. */
size_t goq_packed_bytes(const goq_desc* desc);

/* Algorithmic bytes of the same weights: n_out*k_in*(wbits + 0.75)/8 + n_out*(k_in/group)*4.
 * This is the figure roofline numbers are quoted against; the packed buffer may be larger. */
size_t goq_algorithmic_bytes(const goq_desc* desc);

/* Scratch bytes goq_gemv / goq_gemm need for `m` activation rows (may be 0). Every kernel keeps its counters in
 * the same leading area and leaves them zero, and nothing else in the buffer is carried from one call to the
 * next: one buffer of the largest size, initialised once, can serve calls for different layers, ops and m, as
 * long as those calls cannot overlap on the GPU. */
size_t goq_workspace_bytes(const goq_desc* desc, int op, int m);

/* Zero-fill a scratch buffer (asynchronous on `stream`). A scratch buffer must be initialised once
 * before its first use; every call leaves it ready for the next one. One buffer may serve any number
 * of calls that run one after another on a stream; calls that may overlap need separate buffers. */
goq_status goq_workspace_init(void* ws, size_t ws_bytes, void* stream);

/* Read the device-side status word of a scratch buffer after synchronising `stream`:
 * GOQ_OK, or GOQ_ERR_TIMEOUT if a kernel gave up on a bounded wait. Its outputs are then undefined and counters in
 * the buffer may be left non-zero: zero-fill it again (goq_workspace_init) before the next call that uses it. */
goq_status goq_workspace_status(const void* ws, void* stream, int* status_out);

/* goq_pack - re-tile quantizer output into the layout the kernels stream (Sections 3.2-3.4 give
 * the fields; the layout is this library's own).
 *   codes     [n_out][k_in] uint8, one code per weight, value < 2^wbits
 *   meta      [n_out][k_in/8] uint8, 6-bit exchange record per micro-block
 *   coef_f16  [n_out][k_in/group][2] IEEE fp16 bit patterns (c1, c2)
 *   packed    out, goq_packed_bytes(desc) bytes, 128-byte aligned
 * Layout GOQ_LAYOUT_TILE16: rows padded to a multiple of 16 and k to a multiple of 128 with
 * zero-valued weights; one 32-bit word per micro-block (8 nibbles = 8 codes, record bits in the
 * nibbles' spare top bits for wbits <= 3, in a side byte plane for wbits = 4); words ordered so
 * that the 32 lanes of a warp read 512 contiguous bytes per 128-bit load; coefficient pairs in a
 * second plane, 64 contiguous bytes per (16-row tile, group). */
goq_status goq_pack(const goq_desc* desc, const uint8_t* codes, const uint8_t* meta,
                    const uint16_t* coef_f16, void* packed, size_t packed_bytes, void* stream);

/* goq_unpack - inverse of goq_pack plus the in-register derivation of b2, for tests.
 *   codes_b1  out [n_out][k_in] uint8: the stored code of b1
 *   codes_b2  out [n_out][k_in] uint8: b2 as (sign << 3) | e, or 0x80 for a zero (b2 can take the
 *             value +2^-emax that b1's code cannot express; Section 3.3 on separate sign and magnitude)
 *   coef_f16  out [n_out][k_in/group][2]
 * Any output pointer may be NULL to skip it. */
goq_status goq_unpack(const goq_desc* desc, const void* packed, uint8_t* codes_b1, uint8_t* codes_b2,
                      uint16_t* coef_f16, void* stream);

/* goq_gemv - decode-time layer for a small batch (Eq. 4, float activations).
 *   x_bf16   [batch][k_in] bf16, 16-byte aligned, batch in 1..16
 *   y        out [batch][n_out], y_dtype GOQ_BF16 or GOQ_F32
 *   ws       scratch of goq_workspace_bytes(desc, GOQ_OP_GEMV, batch) bytes, 256-byte aligned,
 *            initialised once with goq_workspace_init (may be NULL if the size is 0)
 * Each PoT term is applied to the activation as an exponent shift; sums are fp32. Up to 4 tokens
 * whose activations fit the chain kernel's staging buffer run as a one-linear goq_gemv_sequence
 * (integer operands: same rounding and saturation of non-finite activations as stated there);
 * the other cases take the bf16-operand streaming kernel.
 * Stream order: the streaming kernel starts fetching `packed` before earlier work on the stream has
 * finished (programmatic dependent launch), so the packed weights must not be written by work that
 * is still in flight on the stream when the call is issued (synchronise after goq_pack, or put
 * other work in between). x and y follow plain stream order. */
goq_status goq_gemv(const goq_desc* desc, const void* packed, const void* x_bf16, int batch, void* y,
                    int y_dtype, void* ws, size_t ws_bytes, void* stream);

/* goq_gemm - the same layer for m activation rows.
 *  x_dtype GOQ_BF16: x [m][k_in] bf16; y out [m][n_out] (GOQ_BF16 or GOQ_F32); sx, cq, sc, acc unused (NULL).
 *      ws: goq_workspace_bytes(desc, GOQ_OP_GEMM, m) bytes, 256-byte aligned, initialised once with
 *      goq_workspace_init. From 33 rows on the tensor-core kernel runs: it keeps an fp16 copy of x (each row scaled by
 *      a power of two, undone in the output) in ws, so the size grows with m * k_in, and it rounds c1*b1 + c2*b2 once
 *      to fp16 (normwise output error about 1.5e-4 to 2.5e-4). The coefficients of every output channel are scaled by a
 *      power of two taken from the channel's largest |c1|, |c2| before that rounding and the output is scaled back, so
 *      the result does not depend on the magnitude of the weights; inside one channel, coefficients more than 2^13
 *      below the channel's largest lose precision to fp16's range.
 *  x_dtype GOQ_I8 (Eq. 4 with integer X~ and c~; left shifts x~ << (emax-e), exact int32):
 *      x    [m][k_in] int8         sx [m] fp32 per-token scale
 *      cq   [n_out][k_in/group][2] int8 integer coefficients,  sc [n_out][2] fp32 their per-channel scales
 *      acc  out, optional: [2][m][n_out] int32, ACC_b[m][n] = sum_j cq[n][j][b] * sum_{k in j} x[m][k] * (2^emax b_b[n][k])
 *      y    out, optional: [m][n_out] = sx[m] * 2^-emax * (sc[n][0]*ACC_1 + sc[n][1]*ACC_2)
 *    At least one of acc, y must be given. Returns GOQ_ERR_OVERFLOW_BOUND if k_in*127*127*2^emax >= 2^31 (W3: k_in up
 *    to 16642; W4, emax = 7: k_in up to 1040). wbits = 4 and groups of 16 run on the packed-dot-product kernel, wbits <= 3
 *    with groups of 32 or more on the int8 tensor-core kernel. */
goq_status goq_gemm(const goq_desc* desc, const void* packed, const void* x, int m, int x_dtype,
                    const float* sx, const int8_t* cq, const float* sc, void* y, int y_dtype,
                    int32_t* acc, void* ws, size_t ws_bytes, void* stream);

/* goq_quantize_activations - the activation quantizer of Section 3.5 (X~ and s_x of Eq. 4): per-token symmetric
 * b_a-bit integers in int8 containers, q_max = 2^(abits-1) - 1, s_x[m] = max_k |x[m,k]| / q_max (1 for an all-zero
 * token), x~ = clamp(rne(x / s_x), +-q_max), evaluated in float64 (round half to even). abits = 8 is the W/A8 setting,
 * 6 and 4 the A6 / A4 settings of the accuracy tables; the integer layer (goq_gemm with GOQ_I8) takes any of them.
 *   x      [m][k] GOQ_F32 or GOQ_BF16        xq  out [m][k] int8        sx  out [m] fp32        abits in 2..8
 *   amax   optional [m] fp32: the tokens' largest magnitudes if the caller already has them (goq_gemm_i8_requant records
 *          them in its epilogue); the kernel then reads x once instead of twice. NULL: computed here. */
goq_status goq_quantize_activations(const void* x, int x_dtype, int m, int k, int abits, const float* amax, int8_t* xq,
                                    float* sx, void* stream);

/* goq_gemm_i8_requant - the integer layer of goq_gemm (x_dtype GOQ_I8) followed by the "global rescaling or
 * requantization" of Section 3.5, after Eq. 4: y = sx * 2^-emax * (sc1 ACC_1 + sc2 ACC_2) as fp32, the per-token
 * largest |y| recorded by the GEMM's epilogue, and - when yq, sy are given - y requantised to the next layer's int8
 * activations with goq_quantize_activations' arithmetic (one more kernel that reads y once).
 *   x, sx, cq, sc as in goq_gemm;  y out [m][n_out] fp32;  amax out [m] fp32 (cleared by the call);
 *   yq out [m][n_out] int8 and sy out [m] fp32, both or neither. */
goq_status goq_gemm_i8_requant(const goq_desc* desc, const void* packed, const int8_t* x, int m, const float* sx,
                               const int8_t* cq, const float* sc, float* y, float* amax, int8_t* yq, float* sy, void* stream);

/* goq_quantize_geo - the GEO-mode quantizer on the device (Sections 3.2-3.4): b1 = Q(w / ||w||_inf) on the asymmetric
 * lattice (nearest state, ties to the smaller magnitude), residual r = w - c1 b1 (Eq. 1), per micro-block
 * d = x_i r_j - x_j r_i, eta* = sgn d (+1 at 0), A_s = sum |d|, s* = first maximiser (Section 3.3, steps 1-3),
 * c1 = <w,b1>/||b1||^2, c2 = <w,b2>/||b2||^2 (Eq. 2), rounded to fp16. float64 arithmetic; one warp per macro-block.
 * With layout GOQ_LAYOUT_TILE16_K1 only b1 and c1 are computed (records 0, c2 = 0).
 *   w      [n_out][k_in] fp32, 16-byte aligned (finite values)
 *   codes, meta, coef_f16   out, in goq_pack's input format (codes 4-byte aligned) */
goq_status goq_quantize_geo(const goq_desc* desc, const float* w, uint8_t* codes, uint8_t* meta, uint16_t* coef_f16,
                            void* stream);

/* goq_solve_ref - REF-mode coefficients (Section 3.4, Eq. 3): per row and macro-block, with X_q the calibration inputs
 * restricted to the macro-block's channels, A = [X_q b1, X_q b2], Y = X_q w:  c* = (A^T A + lambda I)^-1 A^T Y.
 *   w [n_out][k_in] fp32; codes, meta as produced by goq_quantize_geo; x_calib [m][k_in] fp32 (m observations);
 *   lambda >= 0 (the paper uses 1e-4);  coef_f16 out [n_out][k_in/group][2];  c_f64 optional out, the unrounded pairs. */
goq_status goq_solve_ref(const goq_desc* desc, const float* w, const uint8_t* codes, const uint8_t* meta,
                         const float* x_calib, int m, double lambda, uint16_t* coef_f16, double* c_f64, void* stream);

/* goq_gemv_host - goq_gemv for callers whose activations live in host memory (Eq. 4, as goq_gemv).
 *   x_host   HOST [batch][k_in] bf16 (pinned memory makes the copy asynchronous)
 *   y_host   HOST out [batch][n_out]
 *   x_stage, y_stage  DEVICE staging buffers of batch*k_in*2 and batch*n_out*sizeof(y_dtype) bytes
 * Enqueues copy-in, the kernel and copy-out on `stream`; the caller synchronises the stream
 * before reading y_host. */
goq_status goq_gemv_host(const goq_desc* desc, const void* packed, const void* x_host, int batch,
                         void* y_host, int y_dtype, void* x_stage, void* y_stage, void* ws,
                         size_t ws_bytes, void* stream);

/* goq_gemv_static - goq_gemv without a scratch argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a packaging convenience of this library, not part of the method.)
 * Who needs it: code that runs inside a serving engine or plugin host which already owns all device memory
 * through its own arena; latency-critical decode loops that must not risk the device-wide synchronisation
 * cudaMalloc/cudaFree imply; plain C callers with no device allocator of their own. The scratch lives in a
 * fixed array inside the library image (GOQ_STATIC_SCRATCH_BYTES per GPU that loads the library, held until
 * the process exits); nothing is allocated or freed by this call, by any CUDA call it makes, or through torch.
 *   Arguments as goq_gemv; always the bf16-operand streaming kernel (goq_gemv takes the integer-operand form for
 *   up to 4 tokens, so the two can differ in the last bits, both far inside the stated tolerance).
 *   Limits: configurations goq_gemv serves with its scratch-free kernels (group < 32, wbits = 4, more than
 *   16384 row tiles) return GOQ_ERR_UNSUPPORTED here and nothing is launched - use goq_gemv for them. Every layer
 *   the streaming kernel does take fits the array (status word, tile counters, 1 MiB of parked partial sums);
 *   GOQ_ERR_WORKSPACE is reserved for a build whose array is smaller than that.
 *   Status: a kernel that gave up on a bounded wait writes GOQ_ERR_TIMEOUT into the array's first word; read it
 *   with goq_gemv_static_status (which synchronises the stream) BEFORE the next goq_gemv_static call on the
 *   device, because every call clears the word.
 *   First call on each device: looks up the array's device address (once per device, with that device
 *   current). Make that first call outside any stream capture.
 *   Sharing: every call on a device uses the same array. The call clears the part that must start at zero
 *   and the kernel leaves the rest in a state the next call can overwrite, so calls issued one after another
 *   on one stream are fine. Calls that can overlap on the GPU (different streams, or different host threads
 *   feeding different streams) race on the array and corrupt each other's results: serialise them or give
 *   the others their own scratch through goq_gemv. */
#define GOQ_STATIC_SCRATCH_BYTES (2u * 1024u * 1024u)
goq_status goq_gemv_static(const goq_desc* desc, const void* packed, const void* x_bf16, int batch, void* y,
                           int y_dtype, void* stream);
/* Device-side status word of the built-in scratch array of the current device, read after synchronising `stream`
 * (the paper has no counterpart; allocates nothing: the word is copied through the array's cached address). */
goq_status goq_gemv_static_status(void* stream, int* status_out);

/* goq_gemv_sequence: a chain of decode GEMVs (Eq. 4, one call of goq_gemv each) executed by ONE persistent
 * cooperative kernel, in order. Results are those of calling goq_gemv item by item on one stream; what changes
 * is the cost: no launch, prologue or first-byte latency per linear, and the weight stream never stops at a
 * boundary between linears. The kernel computes with integer operands: the activations of each token and
 * 128-wide k-block become 16-bit fixed point (exact for every element within 2^-7 of the block's largest
 * magnitude, rounded at 2^-15 of it below; measured normwise error ~1e-5 or less), the PoT weights times 2^emax
 * are small integers, sums are exact in int32 and the coefficient multiply is fp32. Non-finite activations are
 * not propagated (they saturate).
 *   items    HOST array of n_items entries (read during the call, not kept):
 *            desc, packed, x_bf16 [batch][k_in], y [batch][n_out], y_dtype as in goq_gemv, all device pointers;
 *            depends != 0 : the kernel waits until every earlier item of the sequence is complete (all SMs) before it
 *                           reads this item's x - a full barrier, whatever the buffers;
 *            depends == 0 : the library orders the item from the address ranges alone. Activations that lie inside
 *                           ONE earlier item's bf16 output (the whole output with the same batch, or for batch 1 any
 *                           slice of it that starts at a multiple of 8 channels) are taken as soon as the producer's
 *                           16-channel tiles that hold them are finished, wherever on the GPU that happened: the
 *                           fastest way to chain linears. Any other overlap of this item's x or y with the x or y of
 *                           earlier items (an fp32 producer, an input that spans two outputs, an output buffer used
 *                           twice) is detected too and handled as if depends were set. Items that overlap nothing
 *                           run without waiting.
 *            Give every item of a chain its own output buffer: writing an earlier item's output (or input) buffer
 *            again forces the full barrier.
 *   Constraints (else GOQ_ERR_UNSUPPORTED): every item has the same wbits (2 or 3) and group (32, 64, 128),
 *   batch <= 8, k_in <= 12288, and the staged activations (2 * batch * (round_up(k_in, 128) + 32) bytes) fit in
 *   shared memory beside two 16-record stages of the weight stream (about 180 KB: batch 8 up to k_in = 11008).
 *   ws       goq_sequence_workspace_bytes(n_items) bytes (about 0.5 MB per item: the parts of tiles shared between SMs
 *            and the copies of bf16 outputs that later items read), 256-byte aligned, zero-filled once with
 *            goq_workspace_init; every call leaves it ready for the next one. Its first word is the status word
 *            (goq_workspace_status): after GOQ_ERR_TIMEOUT the outputs are undefined and the buffer must be
 *            zero-filled again before it is reused.
 * Sequences longer than GOQ_SEQUENCE_MAX_ITEMS are split into several launches. The device must support
 * cooperative launches (every sm_100 device does); the grid is one CTA per SM, all resident. */
typedef struct {
    goq_desc desc;
    const void* packed;
    const void* x_bf16;
    void* y;
    int32_t batch;
    int32_t y_dtype;
    int32_t depends;
} goq_gemv_item;
#define GOQ_SEQUENCE_MAX_ITEMS 256
size_t goq_sequence_workspace_bytes(int n_items);
goq_status goq_gemv_sequence(const goq_gemv_item* items, int n_items, void* ws, size_t ws_bytes, void* stream);

/* goq_sequence_order: how goq_gemv_sequence will order each item of `items` (host only: nothing is launched, no pointer
 * is dereferenced; the paper has no counterpart). kind_out[i] receives GOQ_ORDER_NONE (the item waits for nothing),
 * GOQ_ORDER_DATA (it reads an earlier item's bf16 output as that item's 16-channel tiles are finished; source_out[i], if
 * given, receives that item's index, else -1) or GOQ_ORDER_BARRIER (it waits until every earlier item is complete).
 * Item 0 and the first item of every further GOQ_SEQUENCE_MAX_ITEMS items (a new launch) are GOQ_ORDER_NONE. */
#define GOQ_ORDER_NONE 0
#define GOQ_ORDER_DATA 1
#define GOQ_ORDER_BARRIER 2
goq_status goq_sequence_order(const goq_gemv_item* items, int n_items, int32_t* kind_out, int32_t* source_out);

/* goq_gemv_sequence_host: goq_gemv_sequence for callers whose activations and results live in HOST memory.
 * All activations of the sequence sit in one host block and all outputs in another; the call enqueues, on `stream`,
 *   one copy x_host -> x_stage (x_bytes), the sequence kernel, one copy y_stage -> y_host (y_bytes).
 *   items     as in goq_gemv_sequence; every items[i].x_bf16 must point inside [x_stage, x_stage + x_bytes) or, for
 *             an item fed by an earlier item, inside [y_stage, y_stage + y_bytes); every items[i].y inside the y block
 *             (else GOQ_ERR_INVALID_ARG). The layout of the two blocks is the caller's.
 *   x_host, y_host   host pointers (pinned memory makes the copies asynchronous); x_stage, y_stage device blocks.
 * Asynchronous like every other entry point: y_host is valid once the stream has been synchronised. */
goq_status goq_gemv_sequence_host(const goq_gemv_item* items, int n_items, const void* x_host, void* x_stage,
                                  size_t x_bytes, void* y_host, void* y_stage, size_t y_bytes, void* ws,
                                  size_t ws_bytes, void* stream);

/* The cudaError_t value behind the most recent GOQ_ERR_CUDA returned in this process (0 if none). */
int goq_last_cuda_error(void);

/* Force a kernel variant (benchmarks and tests only): 0 = automatic, 1 = scalar exponent-add
 * kernel, 2 = tensor-core fragment kernel, 3 = streaming tensor-core kernel. Process-wide. Returns the
 * previous value. */
int goq_set_gemv_variant(int variant);

/* Bound, in polls, of every device-side wait of goq_gemv_sequence (tests only; 0 restores the kernel's own bound).
 * With a bound of a few polls a dependent chain gives up at once: the call returns GOQ_OK (it only enqueues), the
 * status word then reads GOQ_ERR_TIMEOUT, the context stays usable. Process-wide. Returns the previous value. */
int goq_set_wait_limit(int polls);

#ifdef __cplusplus
}
#endif
#endif /* GOQ_H */
