/*
 * eora_linear.h -- C ABI of the EoRA compensated linear layer for NVIDIA B200 (sm_100a).
 *
 * The operation (paper Eq. 4 / Algorithm 1 step 7, written row-vector style):
 *
 *     Y = X . deq(Wq) + (X . A) . B
 *
 *   X  [M][d_in]      activations (fp16 or bf16), row-major
 *   Wq [d_in][d_out]  frozen compressed backbone: group-wise asymmetric 3/4-bit codes
 *                     (paper Section 4.1 "asymmetric quantization"; group size 128 in the
 *                     group-wise appendix) or 2:4 structured-sparse fp16 (Section 1 / 4.2)
 *   A  [d_in][rank], B [rank][d_out]   the EoRA low-rank residual (Algorithm 1 output), in
 *                     fp16 or quantised to 4-bit group-wise / 8-bit per-channel (Section 4.5)
 *   Y  [M][d_out]     written once (Section 4.5: the output shared by the backbone product and
 *                     the product with B never leaves the chip in between)
 *
 * The paper's column-vector form  W^ X + B' A X  maps as d_in = k, d_out = d, A = A_paper^T,
 * B = B'_paper^T.
 *
 * All pointers are DEVICE pointers unless a parameter is named *_host.  Nothing here is a
 * torch type.  Every function returns an int status (0 = EORA_OK, negative = error); nothing
 * throws, aborts or traps.  The library targets one GPU; there is no CPU fallback.
 *
 * Interchange layout of the weights handed to eora_linear_create (all little-endian):
 *   b-bit codes (b = w_bits = 3 or 4): LSB-first bit stream along d_in for each column n;
 *       the code of (k, n) is stream bits [b*k, b*k+b); word i of the stream is
 *       w_codes[i * d_out + n]  (uint32 [b*d_in/32][d_out]).  For b = 4: 8 codes per uint32,
 *       code k%8 in bits 4*(k%8).  For b = 3: 32 codes per 3 words, codes 10 and 21 straddle.
 *   scales: fp16 [d_in/w_group][d_out].
 *   zeros : the same b-bit stream along n for each group row: uint32 [d_in/w_group][b*d_out/32];
 *       the stored value is the zero-point itself;  w = (q - z) * s.
 *   fp16 A: [d_in][rank] row-major; fp16 B: [rank][d_out] row-major.
 *   4-bit A (ab_format 1): a [d_in x rank] weight in the layout above (codes uint32 [d_in/8][rank],
 *       scales fp16 [d_in/ab_group][rank], zeros uint32 [d_in/ab_group][rank/8]); 4-bit B: a
 *       [rank x d_out] weight with groups of min(ab_group, rank) along rank.
 *   8-bit A/B (ab_format 2): uint8 codes [d_in][rank] / [rank][d_out], one fp16 scale and one
 *       uint8 zero per column (rank of them for A, d_out for B).
 *   2:4 backbone (w_format 1): w_codes = fp16 values [d_out][d_in/2] (the two kept values of each
 *       quad of consecutive k in increasing-k order), w_zeros = uint32 meta [d_out][d_in/32]:
 *       quad j owns nibble (meta[n][j/8] >> 4*(j%8)) & 0xF = p0 | p1<<2, 0 <= p0 < p1 <= 3;
 *       w_scales is unused (may be NULL).
 *   2:4 + 4-bit backbone (w_format 2; the appendix on sparsity & quantisation error compensation prunes to 2:4
 *       and quantises to 4 bits): the d_in/2 kept values of every column are a 4-bit group-wise matrix
 *       [d_in/2][d_out] in the code layout above (w_codes uint32 [d_in/16][d_out]); w_group counts ORIGINAL
 *       reduction elements, so a group holds w_group/2 kept values: w_scales fp16 [d_in/w_group][d_out],
 *       w_zeros uint32 [d_in/w_group][d_out/8]; w_meta = the 2:4 position words uint32 [d_out][d_in/32] as
 *       for w_format 1.  w[4j+p0][n] = (q[2j][n] - z) * s, w[4j+p1][n] = (q[2j+1][n] - z) * s, others 0.
 */
#ifndef EORA_LINEAR_H_
#define EORA_LINEAR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eora_linear* eora_linear_t;   /* opaque handle, owned by the library */

enum {
  EORA_OK = 0,
  EORA_ERR_NULL_ARG = -1,
  EORA_ERR_BAD_SHAPE = -2,
  EORA_ERR_UNSUPPORTED = -3,
  EORA_ERR_MISALIGNED = -4,
  EORA_ERR_M_TOO_LARGE = -5,
  EORA_ERR_CUDA = -6,
  EORA_ERR_DEVICE_TIMEOUT = -7
};

enum { EORA_W_QUANT = 0, EORA_W_SPARSE24 = 1, EORA_W_SPARSE24_Q4 = 2 };
enum { EORA_AB_F16 = 0, EORA_AB_Q4 = 1, EORA_AB_Q8 = 2, EORA_AB_Q3 = 3 };
enum { EORA_X_F16 = 0, EORA_X_BF16 = 1 };
enum { EORA_Y_F16 = 0, EORA_Y_BF16 = 1, EORA_Y_F32 = 2 };
/* kernel families reported by eora_linear_path */
enum { EORA_PATH_GENERIC = 0, EORA_PATH_DECODE = 1, EORA_PATH_PREFILL = 2 };
/* kernel_policy */
enum { EORA_POLICY_AUTO = 0, EORA_POLICY_GENERIC = 1, EORA_POLICY_TMEM_DECODE = 2 };

/* Plain-old-data, caller-owned, copied by create. */
typedef struct {
  int32_t d_in;        /* K; multiple of 128 */
  int32_t d_out;       /* N; multiple of 32 */
  int32_t rank;        /* r >= 0, multiple of 8 (0 = no adapter: the plain compressed layer) */
  int32_t w_format;    /* EORA_W_QUANT, EORA_W_SPARSE24 or EORA_W_SPARSE24_Q4 */
  int32_t w_bits;      /* 3 or 4 (EORA_W_QUANT); 4 (EORA_W_SPARSE24_Q4) */
  int32_t w_group;     /* group size along d_in: multiple of 64 dividing d_in (d_in = channel-wise) */
  int32_t ab_format;   /* EORA_AB_F16 / EORA_AB_Q4 / EORA_AB_Q8 / EORA_AB_Q3 */
  int32_t ab_group;    /* group size for EORA_AB_Q4 / _Q3 (128); B uses min(ab_group, rank) */
  int32_t x_dtype;     /* EORA_X_F16 or EORA_X_BF16 */
  int32_t y_dtype;     /* EORA_Y_F16, EORA_Y_BF16 or EORA_Y_F32 */
  int32_t max_m;       /* largest M forward will be called with (sizes the scratch memory) */
  int32_t kernel_policy; /* EORA_POLICY_AUTO; EORA_POLICY_GENERIC forces the simple kernels; EORA_POLICY_TMEM_DECODE: as AUTO, but M <= 64
                            goes to the tensor-memory decode kernels where they serve the layer (see eora_linear_forward) */
} eora_linear_config;

/* Device pointers, interchange layout (see the top of this file); 16-byte aligned. */
typedef struct {
  const void* w_codes;   /* codes, or 2:4 values */
  const void* w_scales;  /* fp16 scales (NULL for 2:4) */
  const void* w_zeros;   /* packed zero-points, or 2:4 metadata */
  const void* a;         /* fp16 A, or its codes */
  const void* a_scales;  /* NULL when ab_format == EORA_AB_F16 */
  const void* a_zeros;
  const void* b;
  const void* b_scales;
  const void* b_zeros;
  const void* w_meta;    /* 2:4 position words of EORA_W_SPARSE24_Q4; unused (may be NULL) otherwise */
} eora_linear_weights;

/*
 * Build a layer (Eq. 4 operands).  Reads the caller's weight buffers on `stream` (a cudaStream_t,
 * may be NULL for the default stream), re-tiles them into library-owned device memory laid out
 * for 128-bit loads, and allocates the scratch memory forward needs.  The call synchronises
 * `stream` before returning, so the caller may free its buffers afterwards.  The handle is
 * immutable; it owns scratch memory, so two forwards on the same handle must not overlap on the
 * GPU (stream order is enough).  Errors: NULL_ARG, BAD_SHAPE, UNSUPPORTED, MISALIGNED, CUDA;
 * on error *out is NULL and nothing is leaked.
 */
int eora_linear_create(const eora_linear_config* cfg, const eora_linear_weights* w,
                       void* stream, eora_linear_t* out);

/*
 * Y[M][d_out] = X[M][d_in] . deq(Wq) + (X . A) . B   (Eq. 4), enqueued on `stream`.
 * x, y: device pointers, row-major, 16-byte aligned, caller-owned; 1 <= m <= max_m; m == 0 is a
 * no-op returning EORA_OK.  Never synchronises and never allocates.  The current device must be the one
 * the handle was created on (EORA_ERR_UNSUPPORTED otherwise).  M <= 8 runs the decode
 * kernel family (one streaming pass over the weights), M > 8 the tensor-core (tcgen05) family, which
 * for up to 64 tokens splits the reduction axis of a tile over several thread blocks (fp32 sums in the
 * handle's scratch, restored by the block that completes a tile); handles that the tensor-core family
 * does not serve run ceil(M / 8) decode passes up to M = 64 (eora_linear_path reports the choice).
 * Asynchronous device-side
 * problems (a bounded wait that ran out) are latched in a status word readable with
 * eora_linear_last_device_status after the caller has synchronised.
 */
int eora_linear_forward(eora_linear_t h, const void* x, int32_t m, void* y, void* stream);

/*
 * Fused layers.  The compensation of Eq. 4 is applied to every compressed linear layer of a model
 * (Section 3), and several of them read the same activations: q/k/v of an attention block, gate/up
 * of an MLP.  eora_linear_create_fused builds ONE handle for n_layers (2..4) such layers, given as
 * arrays of configs and weights; they must agree in everything but d_out (same d_in, rank, formats,
 * groups, dtypes, max_m, policy AUTO; any backbone format).  eora_linear_forward_fused computes
 *     ys[i][M][d_out_i] = X . deq(Wq_i) + (X . A_i) . B_i      for every layer i
 * with ONE kernel launch for up to eight tokens: X is read once, and the launch latency is paid once.
 * ys: host array of n_layers device pointers (16-byte aligned, caller-owned).  M <= 8: the decode
 * family; more tokens: the tensor-core family (two launches, the first for t = X . A of all layers) if
 * every d_out_i is a multiple of 128 (and the group size of 64), else ceil(M / 8) decode passes up to
 * M = 64.  max_m > 64 therefore needs the tensor-core family: create returns EORA_ERR_UNSUPPORTED
 * otherwise.  eora_linear_forward / _forward_host on it return
 * EORA_ERR_UNSUPPORTED, everything else (destroy, launches, last_device_status, dump of the
 * stacked matrices) works as for a plain handle.  Errors as for create / forward.
 */
int eora_linear_create_fused(const eora_linear_config* cfgs, const eora_linear_weights* weights, int32_t n_layers,
                             void* stream, eora_linear_t* out);
int eora_linear_forward_fused(eora_linear_t h, const void* x, int32_t m, void* const* ys, void* stream);
/*
 * Several adapters on one backbone.  The paper stores the compensation apart from the compressed
 * weights so that task-specific low-rank modules can be switched on and off (Sections 1 and 3); a
 * server decoding several requests at once needs a different module per token.
 * eora_linear_create_multi builds one handle from the layer's config and n_adapters (1..8) weight
 * structs: the backbone is taken from weights[0], adapter j (A_j, B_j and their scales / zeros) from
 * weights[j]; all adapters have the config's rank and format.  eora_linear_forward_multi computes
 *     y[i] = x[i] . deq(Wq) + (x[i] . A_j) . B_j   with j = adapter_ids[i],   or without the second
 * term if adapter_ids[i] is negative (or not below n_adapters),
 * for M <= max_m <= 64 tokens in one launch per eight tokens.  adapter_ids: HOST array of m int32,
 * read before the call returns.  Decode family only; eora_linear_forward on such a handle returns
 * EORA_ERR_UNSUPPORTED.  Cost: every adapter's A and B are streamed once per launch whatever the ids.
 */
int eora_linear_create_multi(const eora_linear_config* cfg, const eora_linear_weights* weights, int32_t n_adapters,
                             void* stream, eora_linear_t* out);
int eora_linear_forward_multi(eora_linear_t h, const void* x, int32_t m, const int32_t* adapter_ids, void* y, void* stream);

/* The fused forward for activations in HOST memory (see eora_linear_forward_host): ys_host is a host array
 * of n_layers host pointers; synchronises `stream` before returning. */
int eora_linear_forward_fused_host(eora_linear_t h, const void* x_host, int32_t m, void* const* ys_host, void* stream);

/*
 * The same forward for callers whose activations live in HOST memory: copies x_host (pinned or
 * pageable, [m][d_in]) to a library-owned device staging buffer, runs the forward, copies the
 * result back to y_host ([m][d_out]) and synchronises `stream` before returning.  When y_host is
 * page-locked memory mapped into the device's address space (cudaHostAlloc / cudaHostRegister) and
 * m <= 64, the kernel stores the result there itself and the copy back is skipped; the bytes
 * crossing the link are the same.
 */
int eora_linear_forward_host(eora_linear_t h, const void* x_host, int32_t m, void* y_host, void* stream);

/*
 * The host-buffer forwards without the synchronisation at the end: the copy of x_host, the launch(es) and the copy (or
 * the kernel's own stores) into y_host / ys_host are enqueued on `stream` and the call returns.  x_host must stay
 * unchanged and y_host unread until the caller has synchronised the stream; both should be page-locked (pageable
 * memory makes the copies synchronous).  The staging buffers belong to the handle, so calls on ONE handle must use
 * one stream (they are then ordered); different handles are independent.  A token's worth of layers can so be
 * enqueued back to back and synchronised once.
 */
int eora_linear_forward_host_async(eora_linear_t h, const void* x_host, int32_t m, void* y_host, void* stream);
int eora_linear_forward_fused_host_async(eora_linear_t h, const void* x_host, int32_t m, void* const* ys_host, void* stream);

/* Free everything the handle owns.  NULL is a no-op.  The caller must have synchronised. */
int eora_linear_destroy(eora_linear_t h);

/* Which kernel family (EORA_PATH_*) forward would run for this m; negative status on error. */
int eora_linear_path(eora_linear_t h, int32_t m);

/* How many of this library's kernels one forward(m) launches; negative status on error. */
int eora_linear_launches(eora_linear_t h, int32_t m);

/*
 * Debug read-back of the library's internal (re-tiled) copy, for bit-exact unpack / dequant
 * checks of steps a1/a2:  what = 0: backbone codes as int32 [d_in][d_out] (quantised backbones);
 * 1: backbone dequantised to fp32 [d_in][d_out], exactly (float)(q - z) * (float)s, or the
 * expanded 2:4 matrix; 2: A as fp32 [d_in][rank]; 3: B as fp32 [rank][d_out].
 * `out` is a device buffer of that size; enqueued on `stream`.
 */
int eora_linear_dump(eora_linear_t h, int32_t what, void* out, void* stream);

/*
 * Status word latched by the kernels (0 = fine, EORA_ERR_DEVICE_TIMEOUT = a bounded wait ran
 * out).  Reads device memory with a blocking copy: call after synchronising.  Clears the word; if it was
 * not zero, the handle's scratch (partial sums, t, tickets) is put back to its between-calls state as well, so
 * that the handle stays usable (the outputs of the call that timed out are undefined).
 */
int eora_linear_last_device_status(eora_linear_t h);

/*
 * Diagnostics.  eora_linear_decode_grid: how many CTAs a decode forward(m) launches (0 if m is
 * not served by the decode family); each CTA has sixteen warps.  eora_linear_set_trace: give the
 * handle a caller-owned device buffer (or NULL to switch tracing off).  A decode forward then
 * records four %globaltimer values (nanoseconds) per warp, at uint64 index
 * 4 * (16 * cta + warp) + k:  k = 0 kernel entry, 1 dependency wait over, 2 first share of the
 * backbone done, 3 all work of the warp done; the buffer must hold 64 * grid values.  A prefill
 * forward records, for CTA (0, 0) only, four clock64 values per 64-element k-block (token tile
 * requested / first weight tile dequantised / token tile seen by the MMA warp / MMAs issued) at
 * index 4 * k_block + k, k_block < nkb = d_in / 64 + (rank padded to 128) / 64, and one more row at
 * k_block = nkb: kernel entry / set-up done / accumulators complete / epilogue done; the buffer
 * must hold 4 * ((d_in + rank) / 64 + 4) values.  Tracing costs time; leave it off in production.
 */
int eora_linear_decode_grid(eora_linear_t h, int32_t m);
int eora_linear_set_trace(eora_linear_t h, void* trace_buf);

/*
 * The same layer for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a deployment convenience of the library.)
 *
 * Everything else in this header works on a handle, and eora_linear_create calls cudaMalloc.  Code
 * that runs after another framework has taken all device memory into its own pool, code in a
 * latency-critical loop that must not risk the stall an allocation can cause, or a plug-in that is
 * only ever handed buffers and a stream, cannot do that.  This call needs no handle: it reads the
 * weights directly from the caller's buffers in the interchange layout (top of this file) and keeps
 * its only scratch, t = X.A as fp32, in a fixed array of EORA_NOALLOC_MAX_T_ELEMS floats (256 KB)
 * that is part of the library image: every GPU that loads the library holds it until the process
 * exits.  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Supported: quantised backbone (3/4-bit), fp16 A and B (or rank 0), any x/y dtype of the config;
 * cfg->max_m and cfg->kernel_policy are ignored.  m * cfg->rank must not exceed
 * EORA_NOALLOC_MAX_T_ELEMS, otherwise EORA_ERR_M_TOO_LARGE is returned and nothing is launched.
 * Other errors as for create / forward.  It runs two simple kernels and is much slower than the
 * handle-based forward.
 *
 * The first call on a device looks up the device address of the scratch array
 * (cudaGetSymbolAddress) with that device current; make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps whatever the previous call left in it; each
 * call overwrites the part it uses before reading it, so nothing has to be cleared, but two calls
 * that overlap on the GPU (different streams) race on it: keep them in stream order.
 */
#define EORA_NOALLOC_MAX_T_ELEMS 65536
int eora_linear_forward_noalloc(const eora_linear_config* cfg, const eora_linear_weights* w, const void* x,
                                int32_t m, void* y, void* stream);

/*
 * Bytes of device memory the handle owns: the re-tiled weights; the scratch the kernels need (partial sums, t, tickets:
 * a few hundred KB to a few MB); and the staging buffers of the *_host entry points, [max_m][d_in] + [max_m][d_out],
 * which are allocated by the first *_host call on the handle (0 before that): a model whose activations stay on the
 * device keeps the memory saving that compression buys (paper Section 4.5, the model-size table).
 */
int64_t eora_linear_weight_bytes(eora_linear_t h);
int64_t eora_linear_scratch_bytes(eora_linear_t h);
int64_t eora_linear_staging_bytes(eora_linear_t h);

/*
 * Diagnostics.  The one wait between thread blocks that Eq. 4 imposes (the product with B needs all of t = X.A) is bounded:
 * a kernel that waits longer than the limit latches EORA_ERR_DEVICE_TIMEOUT, lets its copies in flight land and
 * returns by itself; the outputs of that call are undefined, and eora_linear_last_device_status puts the handle's scratch
 * back so that the next forward is correct.  Default (and ns == 0): one second.  A test sets it to a few nanoseconds to see
 * the timeout path end to end; nothing hangs or faults in it.
 */
int eora_linear_set_wait_limit(eora_linear_t h, uint64_t ns);
/*
 * Self-test of that path: enqueues a one-warp kernel that leaves a partial sum, a partial t and a ticket in the handle's
 * scratch (what a kernel that gives up leaves behind) and then waits, bounded by the handle's limit, for a count nobody
 * raises.  After synchronising, eora_linear_last_device_status must report EORA_ERR_DEVICE_TIMEOUT, and the next forward
 * must be correct again.  Nothing faults or hangs: the wait returns by itself.
 */
int eora_linear_selftest_wait_timeout(eora_linear_t h, void* stream);

/* Human-readable name of a status code; never NULL. */
const char* eora_status_string(int status);

/* Library version: major*10000 + minor*100 + patch. */
int eora_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EORA_LINEAR_H_ */
