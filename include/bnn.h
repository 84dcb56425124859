/*
 * bnn.h -- C ABI of the B200 (sm_100a) forward pass of a feed-forward acoustic-model DNN
 * with binary (+-1) weights and activations (Lu, arXiv 1706.09453).
 *
 * Every step of the forward pass runs in this library's own CUDA kernels; there is no CPU
 * path.  The library never allocates or frees, and only bnn_device_status synchronises: the
 * caller owns every buffer and work is enqueued on `stream` (a cudaStream_t passed as void*;
 * NULL = default stream).  A process may drive several devices; each call works on the device
 * that is current when it is made.
 *
 * Unless an argument is marked HOST, every pointer is a DEVICE pointer.
 *
 * Storage conventions (the paper fixes none; these are this library's):
 *   - real matrices are fp32 row-major with a row pitch `ld*` in floats;
 *   - a binarised matrix stores one bit per element: bit = 1 <=> +1, bit = 0 <=> -1;
 *     element k of a row is bit k%32 of the 32-bit word k/32 (LSB first);
 *   - packed rows have a pitch `ld*p` in 32-bit words which is a multiple of 4, and packed
 *     base pointers are 16-byte aligned, so every row starts on a 16-byte boundary;
 *   - kernels that WRITE a packed row write words 0 .. ceil(K/32)-1 with the unused high
 *     bits of the last word zero; pitch words beyond that are left untouched;
 *   - kernels that READ a packed row ignore bits at positions >= K.
 *
 * Every entry point returns a bnn_status.  Arguments are validated on the host before any
 * launch; a rejected call launches nothing.  Nothing throws or aborts across this ABI.
 */
#ifndef BNN_H_
#define BNN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BNN_API __attribute__((visibility("default")))
#else
#define BNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BNN_OK = 0,
    BNN_ERR_NULL = 1,        /* a required pointer is NULL */
    BNN_ERR_SHAPE = 2,       /* a size is < 1, too large, or a pitch is smaller than its row */
    BNN_ERR_ALIGN = 3,       /* base pointer or pitch breaks the alignment rules above */
    BNN_ERR_UNSUPPORTED = 4, /* a combination of options this library does not implement */
    BNN_ERR_WORKSPACE = 5,   /* workspace missing or too small */
    BNN_ERR_CUDA = 6,        /* the CUDA runtime reported an error at launch */
    BNN_ERR_TIMEOUT = 7      /* a bounded wait inside a kernel ran out: see bnn_device_status */
} bnn_status;

/* Value of Sign at zero.  Eq. 3 of the paper gives +1 for x > 0 and -1 for everything else, i.e.
 * BNN_SIGN_ZERO_NEG.  BNN_SIGN_ZERO_POS is the other common convention (x >= 0 -> +1).
 * NaN maps to -1 in both modes (every comparison with NaN is false). */
typedef enum { BNN_SIGN_ZERO_POS = 0, BNN_SIGN_ZERO_NEG = 1 } bnn_sign_mode;

/* What a stored bit of a binarised ACTIVATION matrix stands for in the layer that reads it.
 * The paper works with the pair (-1,+1) and also reports binary activations in (0,1), which it
 * likens to a Sigmoid with a hard step (Section 3.2, Table 3; Section 3.3, Table 4).  The decision that
 * sets the bit is the same in both (pre-activation positive, or zero under
 * BNN_SIGN_ZERO_POS); only the value the next layer multiplies differs.  Weights are always
 * (-1,+1): the paper's (0,1) weights did not train (Table 3). */
typedef enum { BNN_VALUES_PM1 = 0, BNN_VALUES_01 = 1 } bnn_act_values;

/* What happens to a pre-activation after the per-unit affine (Eq. 2, h = f(h_hat)). */
typedef enum {
    BNN_ACT_NONE = 0,      /* write the value itself */
    BNN_ACT_SIGN_PACK = 1, /* f = Sign (Algorithm 2), written as packed bits */
    BNN_ACT_HARDTANH = 2,  /* f = clamp to [-1, 1], written as fp32 */
    BNN_ACT_SIGMOID = 3    /* f = 1 / (1 + exp(-x)), written as fp32: the real-valued hidden units of
                              the paper's networks (Section 3; Table 2 keeps them on the first and
                              last hidden layer) */
} bnn_act;

/*
 * Epilogue of a GEMM: the per-unit affine y_hat[n] = scale[n]*y[n] + shift[n] (Eq. 1 has
 * only the bias r_l, i.e. scale = 1; a per-unit scale covers a folded normalisation), and
 * the activation.  The affine is ONE fused multiply-add in fp32.
 *
 *   scale, shift : [N] or NULL (NULL scale = 1, NULL shift = 0); used by bnn_signw_gemm.
 *   thr, flip    : used by bnn_xnor_gemm with BNN_ACT_SIGN_PACK.  Because the integer dot
 *                  product d takes few values and d -> fma(scale, d, shift) is monotone,
 *                  Sign(fma(scale[n], d, shift[n])) == ((d >= thr[n]) XOR flipbit[n]);
 *                  bnn_fold_thresholds computes thr [N] and flip [ceil(N/32)] (bit n%32 of
 *                  word n/32) so that this holds for EVERY integer d in [-K, K].
 *   out_bits     : [M][ldob] packed result of BNN_ACT_SIGN_PACK.
 *   sign_mode    : convention for Sign(0) (bnn_signw_gemm; the integer path has it folded
 *                  into thr).
 */
typedef struct bnn_epilogue {
    int act;
    int sign_mode;
    const float* scale;
    const float* shift;
    const int32_t* thr;
    const uint32_t* flip;
    uint32_t* out_bits;
    int ldob;
} bnn_epilogue;

/* ------------------------------------------------------------------------------------
 * Binarisation, Eq. 3 (w^b = Sign(w), Algorithm 1 forward, first statement of the loop).
 * W : fp32 [N][ldw] real-valued weights.   Wp : uint32 [N][ldwp] packed signs (written).
 * Errors: NULL -> BNN_ERR_NULL; N,K < 1, ldw < K, ldwp < ceil(K/32) -> BNN_ERR_SHAPE;
 * ldwp % 4 != 0 or Wp not 16-byte aligned -> BNN_ERR_ALIGN.
 */
BNN_API int bnn_pack_weights(const float* W, int N, int K, int ldw, uint32_t* Wp, int ldwp,
                     int sign_mode, void* stream);

/* Same operation on a matrix of activations (Section 2.2 applies Eq. 3 to activations).
 * X : fp32 [M][ldx].   Ap : uint32 [M][ldap] (written).  Errors as bnn_pack_weights. */
BNN_API int bnn_binarize_pack(const float* X, int M, int K, int ldx, uint32_t* Ap, int ldap,
                      int sign_mode, void* stream);

/* ------------------------------------------------------------------------------------
 * Fold the affine + Sign of a binary hidden layer into integer thresholds (see
 * bnn_epilogue).  scale, shift : [N] or NULL.  K : fan-in of the layer (d ranges over
 * [-K, K]).  thr : int32 [N] (written).  flip : uint32 [ceil(N/32)] (written).
 * The paper has no counterpart: it evaluates Sign(w h + r) directly (Algorithm 2).
 */
BNN_API int bnn_fold_thresholds(const float* scale, const float* shift, int N, int K, int sign_mode,
                        int32_t* thr, uint32_t* flip, void* stream);

/* ------------------------------------------------------------------------------------
 * Binary weights AND binary activations (Section 2.3): the product of Eq. 1 without the
 * bias, d[m][n] = sum_k a[m][k]*w[n][k] with a, w in {-1,+1}
 *             = K - 2*popcount(a_bits XOR w_bits).
 * Ap : [M][ldap] packed activations.  Wp : [N][ldwp] packed weights.  1 <= K <= 2^24.
 * C  : int32 [M][ldc] receives d, or NULL.
 * epi: NULL, or act = BNN_ACT_SIGN_PACK with thr, flip, out_bits set: the next layer's
 *      packed input h = Sign(scale*d + shift) (Eq. 2 with f = Sign) is written without the
 *      integers ever leaving the chip.  At least one of C and epi must be given.
 * Errors: as above; epi->act other than NONE / SIGN_PACK -> BNN_ERR_UNSUPPORTED.
 */
BNN_API int bnn_xnor_gemm(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp,
                  int M, int N, int K, int32_t* C, int ldc,
                  const bnn_epilogue* epi, void* stream);

/* One-time preparation of a binary layer's weights for the tensor cores, and the product of
 * bnn_xnor_gemm on the prepared form.  The tensor cores multiply nothing narrower than 4-bit
 * numbers, so every +-1 has to be widened to 4 bits on its way to them; a layer's weights are
 * the same for every batch, so bnn_xnor_prepare widens them once, into an image laid out in
 * the order the tensor core reads shared memory (4 bits per weight, rounded up to tiles of
 * 192 units x 256 inputs), and bnn_xnor_gemm_prepared streams that image with bulk copies
 * instead of widening the weights again for every tile of frames.  Same integers, same bits.
 * The packed matrix Wp stays the model's stored form (1 bit per weight, the paper's memory
 * argument); the image is a cache that can be rebuilt from it at any time.
 *   prepared : device buffer, 256-byte aligned, at least bnn_xnor_prepared_bytes(N, K) bytes;
 *              written by bnn_xnor_prepare, read by bnn_xnor_gemm_prepared with the SAME N, K.
 *   K <= 2^22 (larger K: BNN_ERR_UNSUPPORTED; use bnn_xnor_gemm).  Other arguments and errors
 *   as bnn_xnor_gemm; a short buffer -> BNN_ERR_WORKSPACE.
 * The paper has no counterpart (it leaves efficient binary products to hardware; Section 3). */
BNN_API size_t bnn_xnor_prepared_bytes(int N, int K);
BNN_API int bnn_xnor_prepare(const uint32_t* Wp, int ldwp, int N, int K,
                             void* prepared, size_t prepared_bytes, void* stream);
BNN_API int bnn_xnor_gemm_prepared(const uint32_t* Ap, int ldap, const void* prepared,
                                   int M, int N, int K, int32_t* C, int ldc,
                                   const bnn_epilogue* epi, void* stream);

/* The product of bnn_xnor_gemm for activations in (0,1) (Section 3.2):
 * d[m][n] = sum_k h[m][k]*w[n][k] with h in {0,1}, w in {-1,+1}
 *         = 2*popcount(h_bits AND w_bits) - popcount(h_bits).
 * Hp : [M][ldhp] packed activations (bit = value).  Wp : [N][ldwp] packed weights, or NULL when
 * `prepared` (the bnn_xnor_prepare image of the same weights) is given; with both, the library
 * picks the faster kernel.  C, epi, errors: as bnn_xnor_gemm (the thresholds of
 * bnn_fold_thresholds apply unchanged: d still lies in [-K, K]). */
BNN_API int bnn_gemm01(const uint32_t* Hp, int ldhp, const uint32_t* Wp, int ldwp, const void* prepared,
                       int M, int N, int K, int32_t* C, int ldc,
                       const bnn_epilogue* epi, void* stream);

/* ------------------------------------------------------------------------------------
 * Binary weights against real-valued activations (Section 2.1; Algorithm 1 forward):
 * y[m][n] = sum_k w^b[n][k]*x[m][k] -- additions and subtractions only -- followed by the
 * epilogue: y_hat = fma(scale[n], y, shift[n]); then
 *   BNN_ACT_NONE      : Y[m][n] = y_hat
 *   BNN_ACT_HARDTANH  : Y[m][n] = min(max(y_hat, -1), 1)
 *   BNN_ACT_SIGN_PACK : out_bits <- Sign(y_hat)   (Y may be NULL; if given it gets y_hat)
 * X : fp32 [M][ldx].  Wp : [N][ldwp].  Y : fp32 [M][ldy] or NULL.  epi NULL = no affine,
 * BNN_ACT_NONE.  Accumulation is fp32.
 */
BNN_API int bnn_signw_gemm(const float* X, int ldx, const uint32_t* Wp, int ldwp,
                   int M, int N, int K, float* Y, int ldy,
                   const bnn_epilogue* epi, void* stream);

/* bnn_signw_gemm with scratch.  With `workspace` (device, 256-byte aligned, at least
 * bnn_signw_workspace_bytes(M, K) bytes) the real operand is split into its bf16 terms once
 * per call, into an image laid out in the order the tensor core reads it, and the GEMM streams
 * that image with bulk copies: 2-4x faster than bnn_signw_gemm on the tensor path.  Without
 * workspace (NULL, or too small) it behaves exactly like bnn_signw_gemm.  Same results within
 * the same bound.  The paper has no counterpart. */
BNN_API size_t bnn_signw_workspace_bytes(int M, int K);
BNN_API int bnn_signw_gemm_ws(const float* X, int ldx, const uint32_t* Wp, int ldwp,
                              int M, int N, int K, float* Y, int ldy,
                              const bnn_epilogue* epi, void* workspace, size_t workspace_bytes,
                              void* stream);

/* ------------------------------------------------------------------------------------
 * Top layer (Section 2.3: the Softmax layer keeps real-valued weights; Algorithm 2, the
 * branch l = L): z[m][c] = sum_n Wout[c][n]*h[m][n] + b[c], logp = z - logsumexp_c(z).
 * Exactly one of Hp (packed +-1 activations [M][ldhp]) and Hf (fp32 [M][ldhf]) is given.
 * Wout : fp32 [C][ldw].  b : [C] or NULL.  logp : fp32 [M][ldo] (written; holds the raw
 * logits between the two internal passes).  log_softmax = 0 leaves the logits z.
 * prepared : NULL, or the image bnn_output_prepare made from the SAME Wout; with it and
 * packed activations the product runs on the tensor cores, otherwise on the FP32 pipe.
 */
BNN_API int bnn_output_layer(const uint32_t* Hp, int ldhp, const float* Hf, int ldhf,
                     const float* Wout, int ldw, const float* b, const void* prepared,
                     int M, int C, int H, float* logp, int ldo, int log_softmax,
                     void* stream);

/* bnn_output_layer on packed activations that stand for (0,1) (Section 3.2); other arguments
 * as there. */
BNN_API int bnn_output_layer01(const uint32_t* Hp, int ldhp, const float* Wout, int ldw,
                               const float* b, const void* prepared, int M, int C, int H,
                               float* logp, int ldo, int log_softmax, void* stream);

/* bnn_output_layer on fp32 activations (the last hidden layer of a binary-weights-only network,
 * Algorithm 1) with scratch.  With `prepared` and a `workspace` (device, 256-byte aligned) of at
 * least bnn_output_workspace_bytes(M, H) bytes the product runs on the tensor cores: the
 * activations are split once per call into two fp16 terms (scratch image), the weights are the
 * two fp16 terms of `prepared`, three MMAs per step:
 *   |z - exact| <= ~3 * 2^-22 * sum_h |Hf[m][h]| |Wout[c][h]|  (+ fp32 accumulation rounding).
 * Activations must be finite with |Hf| < 65504 (hardtanh outputs lie in [-1, 1]).  Without
 * `prepared` or with too little workspace it behaves exactly like bnn_output_layer (FP32 pipe). */
BNN_API size_t bnn_output_workspace_bytes(int M, int H);
BNN_API int bnn_output_layer_ws(const float* Hf, int ldhf, const float* Wout, int ldw,
                                const float* b, const void* prepared, int M, int C, int H,
                                float* logp, int ldo, int log_softmax,
                                void* workspace, size_t workspace_bytes, void* stream);

/* A hidden layer with real-valued weights (Eq. 1-2): Y = f(Hf W^T + bias), f = BNN_ACT_SIGMOID,
 * BNN_ACT_HARDTANH or BNN_ACT_NONE.  Hf : fp32 [M][ldhf].  W : fp32 [N][ldw].  Y : fp32 [M][ldy].
 * With `prepared` (bnn_output_prepare image of W) and `workspace` (bnn_output_workspace_bytes(M, K)
 * bytes, 256-byte aligned) it runs on the tensor cores like bnn_output_layer_ws, same bound before
 * f; otherwise on the FP32 pipe. */
BNN_API int bnn_real_layer(const float* Hf, int ldhf, const float* W, int ldw, const float* bias,
                           const void* prepared, int M, int N, int K, float* Y, int ldy, int act,
                           void* workspace, size_t workspace_bytes, void* stream);

/* Sigmoid units on a binary layer: Y[m][n] = Sigmoid(fma(scale[n], D[m][n], shift[n])) for the
 * integer dot products D of bnn_xnor_gemm (the last hidden layer of the paper's mixed networks,
 * Table 2).  scale, shift : [N] or NULL.  Y may be the same buffer as D when ldy == ldd.  The
 * affine is the same single fp32 fused multiply-add as in the Sign layers. */
BNN_API int bnn_affine_sigmoid_i32(const int32_t* D, int ldd, const float* scale, const float* shift,
                                   int M, int N, float* Y, int ldy, void* stream);

/* One-time preparation of the top layer's weights for the tensor cores: each class row is
 * scaled by a power of two and split into two fp16 terms (about 22 significant bits), stored
 * in the order the MMA reads shared memory.  prepared : device buffer, 256-byte aligned, of
 * at least bnn_output_prepared_bytes(C, H) bytes.  The paper has no counterpart (it keeps
 * this layer in full precision; Section 2.3). */
BNN_API size_t bnn_output_prepared_bytes(int C, int H);
BNN_API int bnn_output_prepare(const float* Wout, int ldw, int C, int H,
                               void* prepared, size_t prepared_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Whole forward pass: the loops "for l = 1 to L" of Algorithms 1 and 2.
 */
typedef enum {
    BNN_LAYER_SIGNW = 0,   /* +-1 weights x real input (first layer; every hidden layer of
                              a binary-weights-only network) */
    BNN_LAYER_XNOR = 1,    /* +-1 weights x +-1 activations */
    BNN_LAYER_REAL_OUT = 2,/* real-valued top layer + log-softmax; must be last */
    BNN_LAYER_REAL = 3     /* real-valued weights x real input + bias, SIGMOID or HARDTANH units: the
                              input layer the paper keeps real-valued in its best systems (Table 2) */
} bnn_layer_kind;

typedef struct bnn_layer {
    int kind;
    int K, N;              /* fan-in, fan-out */
    const uint32_t* Wp;    /* SIGNW, XNOR: packed weights [N][ldwp] */
    int ldwp;
    const float* W;        /* REAL_OUT, REAL: fp32 weights [N][ldw] */
    int ldw;
    const void* W_prepared;/* REAL_OUT, REAL: bnn_output_prepare image of W, or NULL;
                              XNOR: bnn_xnor_prepare image of Wp, or NULL */
    const float* scale;    /* SIGNW: per-unit scale or NULL */
    const float* shift;    /* SIGNW: per-unit shift or NULL; REAL_OUT, REAL: bias or NULL;
                              XNOR with SIGMOID units: scale and shift of the affine */
    const int32_t* thr;    /* XNOR: folded thresholds [N] */
    const uint32_t* flip;  /* XNOR: [ceil(N/32)] */
    int act;               /* SIGNW: SIGN_PACK, HARDTANH or SIGMOID; XNOR: SIGN_PACK (thr, flip) or
                              SIGMOID (scale, shift; fp32 output); REAL: SIGMOID or HARDTANH */
} bnn_layer;

typedef struct bnn_model {
    int n_layers;
    int sign_mode;
    const bnn_layer* layers; /* HOST array of n_layers entries (device pointers inside) */
    int act_values;          /* bnn_act_values of every BNN_ACT_SIGN_PACK activation */
    /* Front and back of a hybrid acoustic model, both optional (0, 0, NULL = off).
     * splice_left/right: the network's input is a window of splice_left + 1 + splice_right
     * consecutive feature frames (Section 3: 11 frames of 40 filter-bank features).  With a
     * window, X holds ONE frame per row, K_0 / (left + right + 1) features wide, and input row m
     * of the first layer is the concatenation of rows m - left .. m + right of X, rows outside
     * [0, M) replaced by the nearest one (one call = one utterance or chunk of it).  The window
     * is formed while the first layer loads its input, so the spliced matrix never exists in
     * memory; this needs the full bnn_forward_workspace_bytes workspace (else
     * BNN_ERR_WORKSPACE).  The paper only says that the features are spliced; the edge rule is
     * this library's.
     * log_prior: device [C] or NULL; subtracted from every row of log-probabilities, which turns
     * the state posteriors into the scaled likelihoods a hybrid HMM decoder consumes
     * (the paper decodes with Kaldi, Section 3; it does not print this step). */
    int splice_left, splice_right;
    const float* log_prior;
} bnn_model;

/* Bytes of scratch for M frames.  bnn_forward_workspace_bytes is what makes bnn_forward
 * fastest: two ping-pong activation buffers, the arrival counters of binary hidden layers that
 * run as one launch (a few bytes per 128 frames and layer) and of the log-softmax that follows the
 * top layer's kernel (4 bytes per 512 frames), and room for the split-activation
 * images: of the widest sign-weight layer (see bnn_signw_gemm_ws; two of them when such layers
 * follow one another, because each writes the next one's image while it reads its own) or of a
 * real-valued layer fed with fp32 activations (see bnn_output_layer_ws).
 * bnn_forward_min_workspace_bytes is the least it accepts (the two buffers and the counters;
 * sign-weight layers then split their activations inside the GEMM and hand on fp32 rows). */
BNN_API size_t bnn_forward_workspace_bytes(const bnn_model* model, int M);
BNN_API size_t bnn_forward_min_workspace_bytes(const bnn_model* model, int M);

/*
 * model : HOST struct.  X : fp32 [M][ldx] spliced features h_0.  logp : fp32 [M][ldo].
 * workspace : device scratch, 256-byte aligned, >= bnn_forward_min_workspace_bytes(model, M);
 *   give bnn_forward_workspace_bytes(model, M) for the fastest path.
 * layer_out : HOST array of n_layers-1 device pointers or NULL; a non-NULL entry l makes
 *   hidden layer l write its output there instead of into the workspace (packed bits with
 *   pitch bnn_packed_pitch(N_l) words, or fp32 [M][N_l] for HARDTANH layers), which lets a
 *   caller inspect every layer at no cost.
 * Layer kinds must chain: a layer with SIGN_PACK units feeds XNOR or REAL_OUT; a layer with
 * fp32 units (HARDTANH, SIGMOID) feeds SIGNW, REAL or REAL_OUT; the last layer is REAL_OUT.
 * Otherwise BNN_ERR_UNSUPPORTED.  The paper's mixed topology (Table 2) is
 * REAL+SIGMOID -> SIGNW+SIGN_PACK -> XNOR+SIGN_PACK ... -> XNOR+SIGMOID -> REAL_OUT.
 */
BNN_API int bnn_forward(const bnn_model* model, const float* X, int ldx, int M,
                float* logp, int ldo, void* workspace, size_t workspace_bytes,
                void* const* layer_out, void* stream);

/* The forward pass for callers that cannot allocate device memory -- for instance a
 * real-time decoding thread (cudaMalloc stalls the whole device), a plug-in whose host
 * program fixes its memory budget at start-up, or a process that has given all device memory
 * to another pool.  Same result as bnn_forward, but the scratch is a fixed array of
 * BNN_STATIC_WORKSPACE_BYTES inside the library image instead of a caller buffer; every GPU
 * that loads the library holds those bytes until the process exits.  The paper has no
 * counterpart.
 *   - Inputs and outputs (model, X, logp) are still the caller's.
 *   - Limit: bnn_forward_min_workspace_bytes(model, M) must not exceed the array; otherwise the
 *     call launches nothing and returns BNN_ERR_WORKSPACE.  (For a 2048-wide network 8 MiB holds
 *     16379 frames of binary activations -- the activation buffers plus the counters of the stacked
 *     binary layers and of the log-softmax that follows the top layer -- or 511 frames of fp32 hardtanh activations.)
 *   - This call makes no cudaMalloc/cudaFree and uses no allocating library routine.
 *   - The first call on each device looks up the array's device address (with that device
 *     current), and the CUDA runtime may load this library's device code -- the array with it --
 *     only then; make that first call at start-up, outside of any stream capture.  From then on a
 *     call leaves the device's free memory exactly as it found it.
 *   - All calls share the one array, which keeps whatever the last call left in it (nothing
 *     needs clearing: each layer only reads what the previous layer wrote in the same call).
 *     Two calls whose kernels can overlap on the GPU -- different streams, or several host
 *     threads -- race on it: run them one after the other. */
#define BNN_STATIC_WORKSPACE_BYTES (8u << 20)
BNN_API int bnn_forward_static(const bnn_model* model, const float* X, int ldx, int M,
                               float* logp, int ldo, void* stream);

/* bnn_forward that also records events on `stream` so a caller can time each layer where it
 * runs.  events : HOST array of n_layers+2 cudaEvent_t (NULL entries skipped): events[l] is
 * recorded before layer l, events[n_layers] after the last kernel, events[n_layers+1]
 * between the top layer's GEMM and its log-softmax.  The paper has no counterpart. */
BNN_API int bnn_forward_events(const bnn_model* model, const float* X, int ldx, int M,
                               float* logp, int ldo, void* workspace, size_t workspace_bytes,
                               void* const* layer_out, void* const* events, void* stream);

/* Process-wide choice of kernels; bnn_set_option returns the previous value or -1 for an
 * unknown option/value.  Every choice computes the same function (integers identical, floats
 * within the documented bounds); the options exist so that the paths can be measured against
 * each other.
 *   BNN_OPT_XNOR_PATH  : BNN_PATH_AUTO | BNN_PATH_CUDA_CORE (XOR/popcount on the integer
 *                        pipes) | BNN_PATH_TENSOR (tcgen05; needs K <= 2^22, larger K falls
 *                        back to popcount).  AUTO = TENSOR, the faster one on B200.
 *   BNN_OPT_REAL_PATH  : same values, for bnn_signw_gemm and bnn_output_layer: FP32 pipe or
 *                        tcgen05 with split bf16/fp16 operands.  AUTO = TENSOR.
 *   BNN_OPT_SIGNW_TERMS: 2 (default) or 3 bf16 terms for the real operand of bnn_signw_gemm
 *                        on the tensor path: |error| <= 2^-17 sum|x_i| with 2, fp32-exact
 *                        products with 3.
 *   BNN_OPT_XNOR_PREPARED: which kernel bnn_xnor_gemm_prepared (and bnn_forward on prepared
 *                        layers) runs for a fused Sign layer: BNN_PREPARED_STREAM reads the
 *                        weight image from L2 for every tile of frames; BNN_PREPARED_RESIDENT
 *                        keeps a tile of units' weights in shared memory for the whole launch
 *                        (needs K <= 3072; other shapes stream); AUTO picks by shape (resident for
 *                        K <= 2048; for a single layer of larger fan-in the kernel that widens the packed
 *                        weights on the fly; runs of equal layers, see BNN_OPT_XNOR_STACK, are resident
 *                        up to K = 3072).
 *   BNN_OPT_SMALL_BATCH: 1 (default) lets bnn_forward run batches of up to 16 frames -- the
 *                        matrix-vector regime the paper has in mind for embedded recognisers
 *                        (Section 1) -- on kernels that spread each layer's weights over all SMs,
 *                        one warp per output unit, on the integer / FP32 pipes, instead of the
 *                        tiled tensor-core kernels (about 4x lower latency); 0 turns that off.
 *                        Integers and bits are identical; the fp32 sums differ by rounding order.
 *   BNN_OPT_XNOR_STACK : 1 (default) lets bnn_forward run consecutive binary hidden layers of one
 *                        shape with prepared weights (the loop over l of Algorithm 2's forward pass)
 *                        as ONE launch, in which a layer's frame tiles start as soon as the layer
 *                        before has stored them; 0 launches one kernel per layer.  Same bits.  The CTAs
 *                        of such a launch wait for one another, so all of them (one per SM at most)
 *                        must be resident together: a caller that runs several forward passes on ONE
 *                        device at the same time (several streams or threads), whose kernels could share
 *                        the SMs between them, should set 0; otherwise such a launch may give up on a
 *                        bounded wait (status word set, see bnn_device_status) instead of finishing.
 *   BNN_OPT_SOFTMAX_FOLLOW: 1 (default) lets bnn_forward launch the log-softmax of a tensor-core top layer
 *                        on packed activations BEHIND that layer's kernel instead of after it: the
 *                        log-softmax kernel shares the SMs with the (tensor-pipe-bound) GEMM and takes every
 *                        512 frames as soon as all their logits are stored, so that only the last frames are
 *                        left when the GEMM ends.  Same log-probabilities.  Its waits are bounded like all
 *                        others (BNN_OPT_WAIT_LIMIT_US).  0 runs the two kernels one after the other; so does
 *                        bnn_forward_events, whose per-layer events need them apart.
 *   BNN_OPT_WAIT_LIMIT_US: how long a kernel may wait on one of its internal barriers or counters before
 *                        it gives up (see bnn_device_status), in microseconds at a nominal 2 GHz SM
 *                        clock; default 1 000 000, minimum 1.  Applies to launches made after the call. */
typedef enum { BNN_OPT_XNOR_PATH = 0, BNN_OPT_REAL_PATH = 1, BNN_OPT_SIGNW_TERMS = 2,
               BNN_OPT_XNOR_PREPARED = 3, BNN_OPT_SMALL_BATCH = 4, BNN_OPT_XNOR_STACK = 5,
               BNN_OPT_WAIT_LIMIT_US = 6, BNN_OPT_SOFTMAX_FOLLOW = 7 } bnn_option;
typedef enum { BNN_PATH_AUTO = 0, BNN_PATH_CUDA_CORE = 1, BNN_PATH_TENSOR = 2 } bnn_path;
typedef enum { BNN_PREPARED_AUTO = 0, BNN_PREPARED_STREAM = 1, BNN_PREPARED_RESIDENT = 2 } bnn_prepared_kernel;
BNN_API int bnn_set_option(int option, int value);

/* Give-up path (the paper has no counterpart).  The tensor-core kernels bound every wait they
 * perform -- on a pipeline barrier, on another CTA's progress counter -- by BNN_OPT_WAIT_LIMIT_US.
 * A CTA whose wait runs out stops, frees its tensor memory, returns normally and sets a status
 * word on its device: 0 = no kernel gave up, 1 = one did (the results of that launch are
 * invalid; the context stays usable).
 *   bnn_device_status : SYNCHRONISES the current device, stores the word in *status (HOST
 *                       pointer) and returns BNN_ERR_TIMEOUT when it is set, BNN_OK otherwise.
 *   bnn_query_status  : the same read in stream order and without a synchronisation: enqueues
 *                       a 4-byte copy of the word into `dst` (DEVICE or pinned HOST memory) on
 *                       `stream`; the caller reads it once the stream has got there.
 *   bnn_reset_status  : enqueues the reset of the word to 0 on `stream`.
 *   bnn_wait_probe    : enqueues a one-warp launch that waits on a barrier on which nothing
 *                       arrives, so that its wait runs out after the limit and the word is set:
 *                       lets a caller (or a test) exercise the path above without a fault. */
BNN_API int bnn_device_status(int* status);
BNN_API int bnn_query_status(int* dst, void* stream);
BNN_API int bnn_reset_status(void* stream);
BNN_API int bnn_wait_probe(void* stream);

/* Micro-benchmarks of the pipes that bound the kernels above (measurement support; the paper
 * has no counterpart: its Section 3 reports accuracy only).  bnn_pipe_rate enqueues ONE launch
 * on `stream` that executes a fixed number of operations of the chosen kind on every SM and
 * stores that number in *work (host pointer, written before the call returns): bit
 * operations for POPC (32 x 2 per instruction, the convention of the XNOR layer: 1 bit-MAC =
 * 2 bop), thread-level instructions for LOP3 / IADD / FADD, flops for FFMA (2 per
 * instruction), bop for the 4-bit MMAs and flop for the fp16 MMA (2 per MAC), bytes for
 * L2_READ.  The caller times the launch with CUDA events on `stream`; rate = *work / time.
 *   POPC, LOP3, IADD, FADD, FFMA : 8 independent dependency chains per thread, 2048 threads/SM
 *   MMA_MXF4_N256 / _N192        : tcgen05.mma kind::mxf4, 128 x N x 64, operands in shared memory
 *   MMA_MXF4_N192_ATMEM          : the same with the A operand in tensor memory
 *   MMA_F16_N256                 : tcgen05.mma kind::f16, 128 x 256 x 16
 *   L2_READ                      : every SM reads the same 32 MB of `scratch`
 * repeat (1 .. 2^20) scales the work linearly (loop trips; groups of 64 MMAs; passes over
 * the 32 MB).  scratch: DEVICE buffer owned by the caller, 16-byte aligned, at least
 * bnn_pipe_rate_scratch_bytes(which) bytes; its contents are overwritten (L2_READ only reads
 * the first 32 MB).  Errors: BNN_ERR_NULL, BNN_ERR_SHAPE (repeat), BNN_ERR_WORKSPACE,
 * BNN_ERR_ALIGN, BNN_ERR_UNSUPPORTED (unknown kind), BNN_ERR_CUDA.  The MMA kinds use bounded
 * waits like every tensor kernel here; a wait that runs out shows in bnn_device_status. */
typedef enum {
    BNN_RATE_POPC = 0, BNN_RATE_LOP3 = 1, BNN_RATE_IADD = 2, BNN_RATE_FADD = 3, BNN_RATE_FFMA = 4,
    BNN_RATE_MMA_MXF4_N256 = 5, BNN_RATE_MMA_MXF4_N192 = 6, BNN_RATE_MMA_MXF4_N192_ATMEM = 7,
    BNN_RATE_MMA_F16_N256 = 8, BNN_RATE_L2_READ = 9
} bnn_rate_kind;
BNN_API size_t bnn_pipe_rate_scratch_bytes(int which);
BNN_API int bnn_pipe_rate(int which, int repeat, void* scratch, size_t scratch_bytes, double* work, void* stream);

/* Smallest legal packed pitch (in words) for rows of K bits: ceil(K/32) rounded up to 4. */
BNN_API int bnn_packed_pitch(int K);

BNN_API const char* bnn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* BNN_H_ */
