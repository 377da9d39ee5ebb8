/* stb.h - C ABI of the N:M structured-binary linear layer y = W^ x on NVIDIA B200 (sm_100a).
 *
 * The layer follows STBLLM (arXiv 2408.01803): of every M = 8 consecutive input columns of
 * an output row exactly N weights are kept (Section 3.3); a kept weight is +-1 times an
 * fp16 scale (Eq. 1); within every block of 128 input columns the kept weights of a row are
 * split into a dense, an intermediate and a sparse region with one scale each (Section 3.4,
 * "Non-Salient Part"; Algorithm 2, Trisection) and the kept weights of the block's salient
 * columns carry a second, residual +-1 term with its own scale (Eq. 4; Algorithm 2,
 * Res_Approx).  In fp32 a kept weight is  s * a_region,  a kept salient weight is
 * fl32(s1 * a_sal1 + s2 * a_sal2), a dropped weight is 0.
 *
 * All entry points are asynchronous on the CUDA stream they are given (a cudaStream_t passed
 * as void*; NULL = the default stream) unless stated otherwise.  Every data pointer is a
 * DEVICE pointer owned by the caller unless its comment says HOST.  The library allocates no
 * device memory.  Its global state is: constant lookup tables in device memory; per-process,
 * per-device caches on the host (which kernels already had their shared-memory limit raised on a
 * device, the device address of the array below, the driver entry point that encodes tensor maps);
 * and the one 8 MiB device array of stb_gemm_noalloc, which that entry point alone writes.
 * Argument errors are returned
 * synchronously and launch nothing; conditions only the device can see (a corrupt logical
 * layer, a bounded wait that ran out) are written to the caller's `dev_status` word (device
 * memory, int32, may be NULL, must be zeroed by the caller) and are read by the caller after
 * it has synchronised the stream.  Nothing traps, aborts or prints.
 */
#ifndef STB_H_
#define STB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum stb_status {
  STB_OK = 0,
  STB_ERR_ARG = 1,          /* null pointer, negative size, bad leading dimension */
  STB_ERR_SHAPE = 2,        /* n < 1, m < 128 or m not a multiple of 128 */
  STB_ERR_NM = 3,           /* N outside 1..8 */
  STB_ERR_SIZE = 4,         /* buffer or workspace too small, batch outside its range */
  STB_ERR_UNSUPPORTED = 5,  /* dtype or mode this build does not provide */
  STB_ERR_CORRUPT = 6,      /* device: logical layer or packed header fails validation */
  STB_ERR_TIMEOUT = 7,      /* device: a bounded wait on an mbarrier ran out */
  STB_ERR_CUDA = 8          /* a CUDA runtime call failed (launch error) */
} stb_status;

typedef enum stb_dtype { STB_F16 = 0, STB_BF16 = 1, STB_F32 = 2 } stb_dtype;

/* Logical (unpacked) layer: the quantizer's output, one field per piece of information of
 * Sections 3.3-3.4.  n output rows, m input columns, N kept of every 8.
 *   keep    [n][m/8]      bit c (LSB first) of a byte: column 8g+c of group g is kept;
 *                         every byte has exactly N bits set               (Section 3.3)
 *   sign    [n][m/8]      bit k: sign of the k-th kept weight of the group in ascending
 *                         column order, 1 = +1, 0 = -1; bits >= N are zero       (Eq. 1-2)
 *   region  [n][m/8]      2 bits per kept weight, same rank order: 0 dense, 1 intermediate,
 *                         2 sparse (Algorithm 2, Trisection), 3 = the column is salient
 *   sign2   [n][m/128]    bit t: residual sign (Eq. 4) of the kept weight in the t-th
 *                         salient column (ascending) of the block; 0 where that weight is
 *                         dropped; bits >= number of salient columns are zero
 *   salient [m/128][2]    128-bit mask of the block's salient columns, word 0 = columns
 *                         0..63; at most 32 bits set                  (Algorithm 2, Salient)
 *   scale   [n][m/128][5] fp16 bit patterns a_dense, a_inter, a_sparse, a_sal1, a_sal2
 */
typedef struct stb_logical {
  int n, m, N;
  const uint8_t *keep;
  const uint8_t *sign;
  const uint16_t *region;
  const uint32_t *sign2;
  const uint64_t *salient;
  const uint16_t *scale;
} stb_logical;

/* HOST struct filled by stb_packed_info. */
typedef struct stb_info {
  int n, m, N;
  int status;             /* what the pack kernels found: STB_OK or STB_ERR_CORRUPT */
  uint64_t used_bytes;    /* header + tables + all tiles + residual codes */
  uint64_t stream_bytes;  /* tiles and residual codes: the bytes one GEMV pass streams from HBM:
                             26 + 6 N bytes per row and block, plus one byte per four salient
                             columns (rounded up) of the block; rows padded to a multiple of 32 */
} stb_info;

/* How a step forms its input.  STB_IN_PLAIN: x = in.  STB_IN_SILU_MUL: x = fp16(silu(in) * in2),
 * silu(v) = v / (1 + exp(-v)), evaluated in fp32: the gated activation that sits between the gate / up and
 * the down projection of a LLaMA MLP (every FFN linear is structured-binary, Section 3; the activation
 * between them is not part of the layer), applied while the down projection stages its activations, so that
 * no extra pass over them is needed.  Only stb_layer_stack_resident takes STB_IN_SILU_MUL. */
typedef enum stb_input { STB_IN_PLAIN = 0, STB_IN_SILU_MUL = 1 } stb_input;

/* One step of stb_layer_stack: out[batch][n] = layer(x[batch][m]).  HOST struct. */
typedef struct stb_step {
  const void *packed;
  int n, m, N;
  const void *in;   /* fp16 [batch][ldin]  */
  void *out;        /* fp32 or fp16 [batch][ldout], see odt */
  stb_dtype odt;    /* STB_F32 or STB_F16 (fp32 sum rounded to nearest even) */
  int batch;
  size_t ldin, ldout;
  const void *in2;  /* fp16 [batch][ldin], 16-byte aligned: second input of STB_IN_SILU_MUL, else NULL */
  stb_input input;
} stb_step;

/* Upper bound of the packed size of an n x m layer at N:8 (the packed size depends on the
 * number of salient columns of every block, at most 8 bytes per row and block for 32 of them;
 * this is the size with all of them).  *bytes is HOST memory.  Synchronous, no CUDA call. */
int stb_pack_size(int n, int m, int N, size_t *bytes);

/* Fused pack / transpose: logical arrays -> the streaming layout read by stb_gemv and
 * stb_gemm (the counterpart of the paper's matrix compression and value compression steps,
 * Appendix C).  The packed buffer must be 256-byte aligned and hold stb_pack_size bytes.
 * Validates on the device that every keep byte has N bits, that sign / region / sign2 carry
 * no bits beyond their fields, that region 3 marks exactly the kept weights of salient
 * columns and that no block has more than 32 salient columns; a violation stores
 * STB_ERR_CORRUPT in *dev_status and in the packed header (the packed data is then not to be
 * used).  Two small launches on `stream`. */
int stb_pack(const stb_logical *L, void *packed, size_t packed_bytes, int *dev_status,
             void *stream);

/* Reads the packed header back (SYNCHRONOUS: waits for `stream`, copies 64 bytes to the
 * host).  Not for the hot path. */
int stb_packed_info(const void *packed, stb_info *info, void *stream);

/* Parity hook: decode the packed layer to a dense row-major matrix W[n][ldw].
 * dt = STB_F32: exactly the fp32 definition at the top of this file.
 * dt = STB_F16 / STB_BF16: that fp32 value rounded to nearest even. */
int stb_dequant(const void *packed, int n, int m, int N, void *W, stb_dtype dt, size_t ldw,
                void *stream);

/* Decode GEMV, batch 1..64:  y[t][i] = sum_j W^[i][j] * x[t][j],  fp32 accumulation.
 * x: fp16 [batch][ldx] (ldx >= m, ldx a multiple of 8, x 16-byte aligned); y: [batch][ldy]
 * (ldy >= n) in fp32 (ydt = STB_F32) or fp16 (STB_F16: the fp32 sum rounded to nearest even,
 * for chaining layers).  The memory-bound case of the paper's Appendix C.2 (decoding stage,
 * N = batch). */
int stb_gemv(const void *packed, int n, int m, int N, const void *x, int batch, size_t ldx,
             void *y, stb_dtype ydt, size_t ldy, int *dev_status, void *stream);

/* Self-test of the bounded device-side waits (Appendix C describes no counterpart; this is the
 * library's failure detection).  Launches the stb_gemv kernel for these arguments (N = 4, 5, 6;
 * other N give STB_ERR_UNSUPPORTED) with its weight copies switched off and its wait limit cut
 * to about 50 microseconds: every warp's wait for its first tiles runs out, the kernel returns
 * normally and *dev_status (required) becomes STB_ERR_TIMEOUT; y receives meaningless values.
 * Nothing faults or hangs, and the next ordinary call works as usual. */
int stb_gemv_wait_selftest(const void *packed, int n, int m, int N, const void *x, int batch,
                           size_t ldx, void *y, stb_dtype ydt, size_t ldy, int *dev_status,
                           void *stream);

/* Bytes of workspace stb_gemm wants for T tokens.  HOST result.  The workspace always holds the
 * activations of the residual slots, gathered per call (T x m / 4 bf16: room for 32 salient columns in
 * every block).  Beyond that, two cases add fp32 partial tiles: few output tiles (every tile is then
 * split along K and the partial tiles are summed afterwards: required), and many output tiles whose
 * last wave of 148 would be small (only that wave's tiles are split: optional, without it those tiles
 * run unsplit).  stb_gemm_workspace gives the size with the optional part, stb_gemm_workspace_min the
 * size stb_gemm cannot do without. */
int stb_gemm_workspace(int n, int m, int N, int T, size_t *bytes);
int stb_gemm_workspace_min(int n, int m, int N, int T, size_t *bytes);

/* Prefill GEMM:  Y[t][i] = sum_j W^[i][j] * X[t][j]  on the tensor cores (tcgen05, fp32
 * accumulation in tensor memory); W^ is decoded tile by tile to bf16 (RN-even): a kept weight is
 * s bf16(a_region), a kept salient weight s1 bf16(a_sal1) + s2 bf16(a_sal2) with the second term
 * multiplied in as extra K (Eq. 4: the two binarizations of a salient weight are two terms).
 * X: bf16 [T][ldx]; Y: fp32 or bf16 [T][ldy] (ydt).  The compute-bound case of Appendix C.2
 * (prefilling stage, N = sequence length x batch).  ws / ws_bytes: caller-owned workspace, 256-byte
 * aligned, of at least stb_gemm_workspace_min bytes (else STB_ERR_SIZE); with stb_gemm_workspace
 * bytes the optional split is used too.  Three launches at most: gather, GEMM, sum of partial tiles. */
int stb_gemm(const void *packed, int n, int m, int N, const void *X, int T, size_t ldx, void *Y,
             stb_dtype ydt, size_t ldy, void *ws, size_t ws_bytes, int *dev_status,
             void *stream);

/* The same product for fp16 activations: X fp16 [T][ldx], Y fp32 or fp16 (ydt = STB_F32 / STB_F16); W^ is decoded to
 * fp16 with its scales as stored (no rounding: a kept weight is s a_region exactly, a salient one s1 a_sal1 + s2 a_sal2 as
 * two terms of the sum), so the result is the one stb_gemv defines.  Meant for decode batches beyond what the GEMV
 * kernels do well (Appendix C.2 between its two stages: tens of tokens): for T <= 64 the CTA tile is 128 rows x 64 tokens
 * (one accumulator of 64 TMEM columns per MMA-issuing lane), K is split into the number of parts that makes waves of
 * 148 CTAs x (a CTA's fixed cost + its blocks) smallest, and the kernel runs at the speed of its decode warps; for T > 64 it is stb_gemm's tiling.  The workspace (stb_gemm_f16_workspace bytes, 256-byte
 * aligned; the gathered residual activations and the fp32 partial tiles) is required.  Errors as stb_gemm. */
int stb_gemm_f16_workspace(int n, int m, int N, int T, size_t *bytes);
int stb_gemm_f16(const void *packed, int n, int m, int N, const void *X, int T, size_t ldx, void *Y,
                 stb_dtype ydt, size_t ldy, void *ws, size_t ws_bytes, int *dev_status,
                 void *stream);

/* stb_gemm without a workspace argument (the paper has no counterpart: this entry point exists
 * for the integration, not for the method).  Some hosts of this library may not allocate device
 * memory while they run: a serving process that gave its whole memory budget to one arena at
 * start-up, or a latency-critical loop in which a cudaMalloc (which synchronises the device)
 * is forbidden.  For them stb_gemm's workspace (gathered residual activations, split-K partial
 * sums) is a fixed 8 MiB array that is part of the library image: every GPU that loads the library holds these 8 MiB until the process
 * exits.  Same arguments, results and errors as stb_gemm, except:
 *   - a call whose required workspace (see stb_gemm_workspace_min) exceeds 8 MiB returns
 *     STB_ERR_SIZE and launches nothing (use stb_gemm with your own workspace for it); an
 *     optional split is used only if its partial tiles fit the array too;
 *   - the first call on each device looks the array's device address up (with that device
 *     current); make that first call outside any stream capture;
 *   - all calls share the one array.  It keeps whatever the last call left there; nothing in
 *     it has to start at zero, because every call writes what it reads there before reading it.
 *     Two calls that may run on the GPU at the same time (different streams) would overwrite
 *     each other's partial sums: keep calls of this entry point on one stream, or order them.
 * It calls no allocation routine of CUDA or of any library. */
int stb_gemm_noalloc(const void *packed, int n, int m, int N, const void *X, int T, size_t ldx,
                     void *Y, stb_dtype ydt, size_t ldy, int *dev_status, void *stream);

/* Runs `count` GEMV steps in order on one stream; every step carries its own N (layer-wise
 * N:M assignment, Section 3.3).  steps is a HOST array.  Launches only. */
int stb_layer_stack(const stb_step *steps, int count, int *dev_status, void *stream);

/* stb_layer_stack as ONE resident kernel (Section 3.3: per-layer N:M; Appendix C.2: decoding is
 * memory-bound, so the weight stream must not stop between layers).  One CTA per SM stays on the
 * machine for the whole list: consecutive steps that read the same activations (q / k / v,
 * gate / up) are dealt to the SMs together in equal shares of 32 x 128 tiles, every warp keeps
 * streaming packed weights across layer boundaries, and a layer that reads an earlier layer's
 * output starts its arithmetic when a counter in the workspace says that every earlier step
 * is complete (bounded poll; STB_ERR_TIMEOUT through *dev_status).  Results are reproducible:
 * every sum has a fixed order.  Steps must have N = 4, 5 or 6 and batch <= 8, else
 * STB_ERR_UNSUPPORTED (use stb_layer_stack).  Lists of more than 64 groups of same-input steps
 * run as several launches.
 * ws: caller-owned DEVICE workspace of stb_layer_stack_resident_workspace bytes, 256-byte
 * aligned, ZEROED by the caller before its first use; every call leaves its counters zero
 * again (also after a wait that ran out), so the same workspace serves call after call without
 * being cleared; the rest of it holds partial sums that are written before they are read.
 * Calls that share a workspace must not overlap on the GPU.
 * The launch is cooperative: it fails with STB_ERR_CUDA when the GPU cannot hold one 512-thread
 * CTA per SM at once. */
int stb_layer_stack_resident_workspace(const stb_step *steps, int count, size_t *bytes);
int stb_layer_stack_resident(const stb_step *steps, int count, void *ws, size_t ws_bytes,
                             int *dev_status, void *stream);

/* stb_layer_stack_host through the resident kernel (same copies before and after). */
int stb_layer_stack_resident_host(const stb_step *steps, int count, void *ws, size_t ws_bytes,
                                  const void *in_host, size_t in_bytes, void *out_host,
                                  size_t out_bytes, int *dev_status, void *stream);

/* Self-test of the resident kernel's bounded waits, in the manner of stb_gemv_wait_selftest:
 * weight copies off, wait limit about 50 microseconds.  *dev_status (required) becomes
 * STB_ERR_TIMEOUT, every CTA leaves, the workspace is zero again; outputs are meaningless. */
int stb_layer_stack_resident_wait_selftest(const stb_step *steps, int count, void *ws,
                                           size_t ws_bytes, int *dev_status, void *stream);

/* Integrity check of packed layers (the paper has no counterpart): sums[i] (DEVICE, 64-bit, one per step)
 * becomes the XOR of all 32-bit words of step i's tiles and residual streams, i.e. of the bytes
 * [tiles offset, used_bytes) of its packed buffer -- everything a decode pass streams.  Only `packed`, n, m,
 * N, batch and the pointers' validity of a step are looked at.  The layers are walked exactly as
 * stb_layer_stack_resident walks them (same dealing to the SMs, same rings and bulk copies), without
 * the arithmetic: its running time is what that way of streaming costs by itself.  One launch per 64
 * groups of steps, plus a memset of sums. */
int stb_layer_stack_checksum(const stb_step *steps, int count, unsigned long long *sums,
                             int *dev_status, void *stream);

/* stb_layer_stack for a caller whose activations live in HOST memory: copies in_bytes from
 * in_host (HOST, pinned for the copy to be asynchronous) into steps[0].in, runs the steps,
 * then copies out_bytes from steps[count-1].out to out_host (HOST).  The device buffers named
 * in the steps stay caller-owned staging; everything is queued on `stream` and the caller
 * synchronises it before reading out_host.  Same per-layer N rule (Section 3.3). */
int stb_layer_stack_host(const stb_step *steps, int count, const void *in_host, size_t in_bytes,
                         void *out_host, size_t out_bytes, int *dev_status, void *stream);

/* The quantizer on the GPU: Standardized Importance (Eq. 3), N of 8 per group (Section 3.3), the salient-column
 * search and the break-point search of Algorithm 2 (32 candidate columns, 160 grid points, sigma = 2), residual
 * binarization (Eq. 4) and trisection: the block loop of Algorithm 1 without its Hessian update (column score with
 * the diagonal h_jj = 2 ||X_:,j||^2; lambda < 0 selects 0.01 mean_j h_jj).  W: dense fp16 [n][ldw]; xnorm: float64
 * [m], the column norms of the calibration activations; out: a stb_logical whose n, m, N match and whose six DEVICE
 * arrays (sizes as documented at stb_logical) are WRITTEN here, ready for stb_pack.  float64 throughout; sums that
 * are not exact are taken in the order of the definition, so the result does not depend on the launch shape.
 * ws: DEVICE workspace of stb_quantize_workspace bytes, 256-byte aligned.  About a dozen launches on `stream`. */
int stb_quantize_workspace(int n, int m, size_t *bytes);
int stb_quantize(const void *W, size_t ldw, const double *xnorm, int n, int m, int N, double lambda,
                 const stb_logical *out, void *ws, size_t ws_bytes, void *stream);

/* Layer-wise N:M assignment (Section 3.3): more important layers, by the L2 norm of their weights, keep more of
 * every 8.  stb_weight_sumsq adds the sum of squares of a dense fp16 matrix W[n][ldw] (DEVICE, 16-byte aligned, ldw a
 * multiple of 8) to *sumsq (DEVICE float64, zeroed by the caller; one launch).  stb_allocate_nm is HOST arithmetic on
 * the layers' sums of squares copied back: alpha_i = omega_i / sum_k omega_k with omega = sqrt(sum of squares),
 * N_i = 8 (alpha_i + (1 - alpha_i) r_target) rounded to nearest (ties to even) and kept inside 1..8.  As printed in the
 * paper the ratio never falls below r_target. */
int stb_weight_sumsq(const void *W, int n, int m, size_t ldw, double *sumsq, void *stream);
int stb_allocate_nm(const double *sumsq, int layers, double r_target, int *N_out);

/* Static string for a status code. */
const char *stb_status_str(int status);

#ifdef __cplusplus
}
#endif
#endif /* STB_H_ */
