// extern "C" boundary: argument validation and kernel sequencing.  No allocation, no sync.
#include <stdint.h>

#include "bnn_common.cuh"

using namespace bnn;

namespace {

constexpr int kMaxK = 1 << 24;
int g_xnor_path = BNN_PATH_AUTO;
int g_real_path = BNN_PATH_AUTO;
int g_xnor_prepared = BNN_PREPARED_AUTO;
int g_small_batch = 1;  // batches of up to kSmallBatchMax frames take the matrix-vector kernels
int g_signw_terms = 2;  // |dot| <= K stays exact in every accumulator type used
int g_xnor_stack = 1;   // runs of equal binary hidden layers go out as one launch
int g_softmax_follow = 1;   // bnn_forward's log-softmax follows the top layer's kernel tile by tile

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

int check_packed(const void* p, int ld, int k) {
    if (!p) return BNN_ERR_NULL;
    if (ld < words_for(k)) return BNN_ERR_SHAPE;
    if (ld % 4 != 0 || !aligned16(p)) return BNN_ERR_ALIGN;
    return BNN_OK;
}

int check_dims(int a, int b, int c) {
    if (a < 1 || b < 1 || c < 1) return BNN_ERR_SHAPE;
    return BNN_OK;
}

int sign_pack_checked(const float* X, int R, int K, int ldx, uint32_t* P, int ldp, int mode,
                      void* stream) {
    if (!X || !P) return BNN_ERR_NULL;
    if (R < 1 || K < 1 || ldx < K) return BNN_ERR_SHAPE;
    if (mode != BNN_SIGN_ZERO_POS && mode != BNN_SIGN_ZERO_NEG) return BNN_ERR_UNSUPPORTED;
    int rc = check_packed(P, ldp, K);
    if (rc) return rc;
    return launch_sign_pack(X, R, K, ldx, P, ldp, mode, (cudaStream_t)stream);
}

// Bytes of one hidden layer's output for M frames.
size_t layer_out_bytes(const bnn_layer& L, int M) {
    if (L.act == BNN_ACT_SIGN_PACK) return (size_t)M * bnn_packed_pitch(L.N) * sizeof(uint32_t);
    return (size_t)M * L.N * sizeof(float);
}

int validate_model(const bnn_model* model) {
    if (!model || !model->layers) return BNN_ERR_NULL;
    const int L = model->n_layers;
    if (L < 1) return BNN_ERR_SHAPE;
    if (model->sign_mode != BNN_SIGN_ZERO_POS && model->sign_mode != BNN_SIGN_ZERO_NEG)
        return BNN_ERR_UNSUPPORTED;
    if (model->act_values != BNN_VALUES_PM1 && model->act_values != BNN_VALUES_01) return BNN_ERR_UNSUPPORTED;
    int prev_act = BNN_ACT_NONE;  // real-valued input h_0
    int prev_n = -1;
    for (int l = 0; l < L; ++l) {
        const bnn_layer& y = model->layers[l];
        if (y.K < 1 || y.N < 1 || y.K > kMaxK) return BNN_ERR_SHAPE;
        if (prev_n >= 0 && y.K != prev_n) return BNN_ERR_SHAPE;
        const bool in_bits = prev_act == BNN_ACT_SIGN_PACK;
        switch (y.kind) {
            case BNN_LAYER_SIGNW:
                if (in_bits || l == L - 1) return BNN_ERR_UNSUPPORTED;
                if (y.act != BNN_ACT_SIGN_PACK && y.act != BNN_ACT_HARDTANH && y.act != BNN_ACT_SIGMOID)
                    return BNN_ERR_UNSUPPORTED;
                if (int rc = check_packed(y.Wp, y.ldwp, y.K)) return rc;
                break;
            case BNN_LAYER_XNOR:
                if (!in_bits || l == L - 1) return BNN_ERR_UNSUPPORTED;
                if (y.act == BNN_ACT_SIGN_PACK) {
                    if (!y.thr || !y.flip) return BNN_ERR_NULL;
                } else if (y.act != BNN_ACT_SIGMOID) {
                    return BNN_ERR_UNSUPPORTED;
                }
                if (int rc = check_packed(y.Wp, y.ldwp, y.K)) return rc;
                break;
            case BNN_LAYER_REAL:
                if (in_bits || l == L - 1) return BNN_ERR_UNSUPPORTED;
                if (y.act != BNN_ACT_SIGMOID && y.act != BNN_ACT_HARDTANH) return BNN_ERR_UNSUPPORTED;
                if (!y.W) return BNN_ERR_NULL;
                if (y.ldw < y.K) return BNN_ERR_SHAPE;
                if (y.scale) return BNN_ERR_UNSUPPORTED;   // Eq. 1 as printed: weights and a bias
                break;
            case BNN_LAYER_REAL_OUT:
                if (l != L - 1) return BNN_ERR_UNSUPPORTED;
                if (!y.W) return BNN_ERR_NULL;
                if (y.ldw < y.K) return BNN_ERR_SHAPE;
                break;
            default:
                return BNN_ERR_UNSUPPORTED;
        }
        prev_act = y.act;
        prev_n = y.N;
    }
    if (model->layers[L - 1].kind != BNN_LAYER_REAL_OUT) return BNN_ERR_UNSUPPORTED;
    return BNN_OK;
}

// Whether hidden layer l can be part of a run launched as one kernel: a fused Sign layer on packed
// input with prepared weights, of a shape the resident-weights kernel takes (fan-in up to 3072).  As
// ONE launch of several layers that kernel also wins on its narrow tiles (fan-in above 2048: AMI-scale
// hidden layers 1.70 ms for five against 5 x 0.39 for the kernel that widens both operands on the fly);
// a single such layer is left to bnn_xnor_gemm_prepared's own choice.
bool stackable(const bnn_model* model, int l) {
    const bnn_layer& y = model->layers[l];
    if (y.kind != BNN_LAYER_XNOR || y.act != BNN_ACT_SIGN_PACK || !y.W_prepared) return false;
    if (g_xnor_path == BNN_PATH_CUDA_CORE || g_xnor_prepared == BNN_PREPARED_STREAM || y.K > kMaxKTensor) return false;
    if (reinterpret_cast<uintptr_t>(y.W_prepared) & 255u) return false;
    if (!xnor_res_applicable(y.N, y.K)) return false;
    return true;
}

}  // namespace

extern "C" {

int bnn_packed_pitch(int K) { return (words_for(K) + 3) & ~3; }

size_t bnn_pipe_rate_scratch_bytes(int which) { return pipe_rate_scratch_bytes(which); }

int bnn_pipe_rate(int which, int repeat, void* scratch, size_t scratch_bytes, double* work, void* stream) {
    return launch_pipe_rate(which, repeat, scratch, scratch_bytes, work, static_cast<cudaStream_t>(stream));
}

int bnn_set_option(int option, int value) {
    int* slot = nullptr;
    switch (option) {
        case BNN_OPT_XNOR_PATH: slot = &g_xnor_path; break;
        case BNN_OPT_REAL_PATH: slot = &g_real_path; break;
        case BNN_OPT_SIGNW_TERMS: slot = &g_signw_terms; break;
        case BNN_OPT_XNOR_PREPARED: slot = &g_xnor_prepared; break;
        case BNN_OPT_SMALL_BATCH: slot = &g_small_batch; break;
        case BNN_OPT_XNOR_STACK: slot = &g_xnor_stack; break;
        case BNN_OPT_SOFTMAX_FOLLOW: slot = &g_softmax_follow; break;
        case BNN_OPT_WAIT_LIMIT_US: {
            // microseconds -> SM clocks at a nominal 2 GHz
            if (value < 1) return -1;
            const long long prev = set_wait_limit_clocks((long long)value * 2000);
            return (int)(prev / 2000 > 0x7FFFFFFF ? 0x7FFFFFFF : prev / 2000);
        }
        default: return -1;
    }
    if (option == BNN_OPT_SIGNW_TERMS) {
        if (value != 2 && value != 3) return -1;
    } else if (option == BNN_OPT_SMALL_BATCH || option == BNN_OPT_XNOR_STACK || option == BNN_OPT_SOFTMAX_FOLLOW) {
        if (value != 0 && value != 1) return -1;
    } else if (option == BNN_OPT_XNOR_PREPARED) {
        if (value != BNN_PREPARED_AUTO && value != BNN_PREPARED_STREAM && value != BNN_PREPARED_RESIDENT) return -1;
    } else if (value != BNN_PATH_AUTO && value != BNN_PATH_CUDA_CORE && value != BNN_PATH_TENSOR) {
        return -1;
    }
    const int prev = *slot;
    *slot = value;
    return prev;
}

int bnn_device_status(int* status) {
    if (!status) return BNN_ERR_NULL;
    if (int rc = read_tc_status(status)) return rc;
    return *status ? BNN_ERR_TIMEOUT : BNN_OK;
}

int bnn_query_status(int* dst, void* stream) {
    if (!dst) return BNN_ERR_NULL;
    return copy_tc_status_async(dst, (cudaStream_t)stream);
}

int bnn_reset_status(void* stream) { return reset_tc_status_async((cudaStream_t)stream); }

int bnn_wait_probe(void* stream) { return launch_wait_probe((cudaStream_t)stream); }

const char* bnn_status_string(int status) {
    switch (status) {
        case BNN_OK: return "ok";
        case BNN_ERR_NULL: return "a required pointer is NULL";
        case BNN_ERR_SHAPE: return "bad size or pitch";
        case BNN_ERR_ALIGN: return "pointer or pitch breaks the 16-byte alignment rule";
        case BNN_ERR_UNSUPPORTED: return "unsupported combination of options";
        case BNN_ERR_WORKSPACE: return "workspace missing or too small";
        case BNN_ERR_CUDA: return "CUDA runtime error at launch";
        case BNN_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out (device status word set)";
        default: return "unknown status";
    }
}

int bnn_pack_weights(const float* W, int N, int K, int ldw, uint32_t* Wp, int ldwp,
                     int sign_mode, void* stream) {
    return sign_pack_checked(W, N, K, ldw, Wp, ldwp, sign_mode, stream);
}

int bnn_binarize_pack(const float* X, int M, int K, int ldx, uint32_t* Ap, int ldap,
                      int sign_mode, void* stream) {
    return sign_pack_checked(X, M, K, ldx, Ap, ldap, sign_mode, stream);
}

int bnn_fold_thresholds(const float* scale, const float* shift, int N, int K, int sign_mode,
                        int32_t* thr, uint32_t* flip, void* stream) {
    if (!thr || !flip) return BNN_ERR_NULL;
    if (N < 1 || K < 1 || K > kMaxK) return BNN_ERR_SHAPE;
    if (sign_mode != BNN_SIGN_ZERO_POS && sign_mode != BNN_SIGN_ZERO_NEG) return BNN_ERR_UNSUPPORTED;
    return launch_fold_thresholds(scale, shift, N, K, sign_mode, thr, flip, (cudaStream_t)stream);
}

// Shared by bnn_xnor_gemm (image == nullptr), bnn_xnor_gemm_prepared (Wp == nullptr) and
// bnn_forward (both, when the layer has an image).
static int xnor_gemm_impl(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, const void* image,
                          int M, int N, int K, int32_t* C, int ldc,
                          const bnn_epilogue* epi, int zo, void* stream) {
    if (int rc = check_dims(M, N, K)) return rc;
    if (K > kMaxK) return BNN_ERR_SHAPE;
    if (int rc = check_packed(Ap, ldap, K)) return rc;
    if (image) {
        if (K > kMaxKTensor) return BNN_ERR_UNSUPPORTED;
        if (reinterpret_cast<uintptr_t>(image) & 255u) return BNN_ERR_ALIGN;
    }
    if (Wp || !image)
        if (int rc = check_packed(Wp, ldwp, K)) return rc;
    if (C && ldc < N) return BNN_ERR_SHAPE;
    const int32_t* thr = nullptr;
    const uint32_t* flip = nullptr;
    uint32_t* ob = nullptr;
    int ldob = 0;
    if (epi && epi->act != BNN_ACT_NONE) {
        if (epi->act != BNN_ACT_SIGN_PACK) return BNN_ERR_UNSUPPORTED;
        if (!epi->thr || !epi->flip) return BNN_ERR_NULL;
        if (int rc = check_packed(epi->out_bits, epi->ldob, N)) return rc;
        thr = epi->thr; flip = epi->flip; ob = epi->out_bits; ldob = epi->ldob;
    }
    if (!C && !ob) return BNN_ERR_NULL;
    if (image) {
        // Fused Sign layer: the kernel that keeps a unit tile's weights in shared memory where
        // measurement favours it (K <= 2048, tiles of 192 units; with K <= 3072 its tiles shrink
        // to 128 units and the kernel that widens packed weights on the fly is faster, so that
        // one runs when the packed weights are at hand).  int32 output and the remaining shapes:
        // the kernel that streams the image.
        const bool fused = !C && g_xnor_prepared != BNN_PREPARED_STREAM && xnor_res_applicable(N, K);
        const bool wide_tiles = K <= 2048;
        if (fused && (wide_tiles || !Wp || g_xnor_prepared == BNN_PREPARED_RESIDENT))
            return launch_xnor_res(Ap, ldap, image, M, N, K, thr, flip, ob, ldob, zo, (cudaStream_t)stream);
        if (!Wp || g_xnor_prepared == BNN_PREPARED_STREAM)
            return launch_xnor_img(Ap, ldap, image, M, N, K, C, ldc, thr, flip, ob, ldob, zo, (cudaStream_t)stream);
    }
    const bool tensor = g_xnor_path != BNN_PATH_CUDA_CORE && K <= kMaxKTensor;
    return (tensor ? launch_xnor_tc : launch_xnor_popc)(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip,
                                                        ob, ldob, zo, (cudaStream_t)stream);
}

int bnn_xnor_gemm(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp,
                  int M, int N, int K, int32_t* C, int ldc,
                  const bnn_epilogue* epi, void* stream) {
    if (!Wp) return BNN_ERR_NULL;
    return xnor_gemm_impl(Ap, ldap, Wp, ldwp, nullptr, M, N, K, C, ldc, epi, 0, stream);
}

int bnn_gemm01(const uint32_t* Hp, int ldhp, const uint32_t* Wp, int ldwp, const void* prepared,
               int M, int N, int K, int32_t* C, int ldc, const bnn_epilogue* epi, void* stream) {
    if (!Wp && !prepared) return BNN_ERR_NULL;
    return xnor_gemm_impl(Hp, ldhp, Wp, ldwp, prepared, M, N, K, C, ldc, epi, 1, stream);
}

size_t bnn_xnor_prepared_bytes(int N, int K) {
    if (N < 1 || K < 1 || K > kMaxKTensor) return 0;
    return xnor_image_bytes(N, K);
}

int bnn_xnor_prepare(const uint32_t* Wp, int ldwp, int N, int K,
                     void* prepared, size_t prepared_bytes, void* stream) {
    if (!prepared) return BNN_ERR_NULL;
    if (N < 1 || K < 1) return BNN_ERR_SHAPE;
    if (K > kMaxKTensor) return BNN_ERR_UNSUPPORTED;
    if (int rc = check_packed(Wp, ldwp, K)) return rc;
    if (prepared_bytes < xnor_image_bytes(N, K)) return BNN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(prepared) & 255u) return BNN_ERR_ALIGN;
    return launch_xnor_prepare(Wp, ldwp, N, K, prepared, (cudaStream_t)stream);
}

int bnn_xnor_gemm_prepared(const uint32_t* Ap, int ldap, const void* prepared,
                           int M, int N, int K, int32_t* C, int ldc,
                           const bnn_epilogue* epi, void* stream) {
    if (!prepared) return BNN_ERR_NULL;
    return xnor_gemm_impl(Ap, ldap, nullptr, 0, prepared, M, N, K, C, ldc, epi, 0, stream);
}

size_t bnn_signw_workspace_bytes(int M, int K) {
    if (M < 1 || K < 1) return 0;
    return signw_image_bytes(M, K, g_signw_terms);
}

int bnn_signw_gemm(const float* X, int ldx, const uint32_t* Wp, int ldwp,
                   int M, int N, int K, float* Y, int ldy,
                   const bnn_epilogue* epi, void* stream) {
    return bnn_signw_gemm_ws(X, ldx, Wp, ldwp, M, N, K, Y, ldy, epi, nullptr, 0, stream);
}

// splice_dim > 0: X is [M][ldx] with splice_dim features per frame and row m of the product's
// input is the concatenation of frames m - splice_left .. (K / splice_dim frames), clamped to
// the batch; only the path that splits the activations into a scratch image forms it.
static int signw_impl(const float* X, int ldx, const uint32_t* Wp, int ldwp,
                      int M, int N, int K, float* Y, int ldy,
                      const bnn_epilogue* epi, void* workspace, size_t workspace_bytes,
                      int splice_dim, int splice_left, void* stream,
                      bool image_ready = false, void* out_image = nullptr, int out_kind = 0,
                      int* clear = nullptr, int clear_words = 0, bool* cleared = nullptr) {
    if (cleared) *cleared = false;
    if (int rc = check_dims(M, N, K)) return rc;
    if (!X && !image_ready) return BNN_ERR_NULL;
    if (ldx < (splice_dim > 0 ? splice_dim : K)) return BNN_ERR_SHAPE;
    if (int rc = check_packed(Wp, ldwp, K)) return rc;
    if (Y && ldy < N) return BNN_ERR_SHAPE;
    RealGemmArgs a{};
    a.Af = X; a.lda = ldx; a.Bb = Wp; a.ldb = ldwp;
    a.splice_dim = splice_dim; a.splice_left = splice_left;
    a.M = M; a.N = N; a.K = K;
    a.Y = Y; a.ldy = ldy;
    a.act = BNN_ACT_NONE; a.sign_mode = BNN_SIGN_ZERO_POS;
    if (epi) {
        if (epi->act != BNN_ACT_NONE && epi->act != BNN_ACT_SIGN_PACK && epi->act != BNN_ACT_HARDTANH &&
            epi->act != BNN_ACT_SIGMOID)
            return BNN_ERR_UNSUPPORTED;
        if (epi->sign_mode != BNN_SIGN_ZERO_POS && epi->sign_mode != BNN_SIGN_ZERO_NEG)
            return BNN_ERR_UNSUPPORTED;
        a.scale = epi->scale; a.shift = epi->shift; a.act = epi->act; a.sign_mode = epi->sign_mode;
        if (epi->act == BNN_ACT_SIGN_PACK) {
            if (int rc = check_packed(epi->out_bits, epi->ldob, N)) return rc;
            a.out_bits = epi->out_bits; a.ldob = epi->ldob;
        }
    }
    if (!a.Y && !a.out_bits && !out_image) return BNN_ERR_NULL;
    if (g_real_path != BNN_PATH_CUDA_CORE) {
        if (workspace && !(reinterpret_cast<uintptr_t>(workspace) & 255u) &&
            workspace_bytes >= signw_image_bytes(M, K, g_signw_terms)) {
            // the kernel that splits the activations can clear the caller's counters on its way
            const bool clears = clear && clear_words > 0 && !image_ready;
            if (cleared) *cleared = clears;
            return launch_signw_img(a, g_signw_terms, workspace, image_ready, out_image, out_kind,
                                    clears ? clear : nullptr, clears ? clear_words : 0, (cudaStream_t)stream);
        }
        if (splice_dim > 0 || image_ready || out_image) return BNN_ERR_WORKSPACE;
        return launch_signw_tc(a, g_signw_terms, (cudaStream_t)stream);
    }
    if (splice_dim > 0) return BNN_ERR_UNSUPPORTED;
    return launch_real_gemm(a, (cudaStream_t)stream);
}

int bnn_signw_gemm_ws(const float* X, int ldx, const uint32_t* Wp, int ldwp,
                      int M, int N, int K, float* Y, int ldy,
                      const bnn_epilogue* epi, void* workspace, size_t workspace_bytes,
                      void* stream) {
    return signw_impl(X, ldx, Wp, ldwp, M, N, K, Y, ldy, epi, workspace, workspace_bytes, 0, 0, stream);
}

size_t bnn_output_prepared_bytes(int C, int H) {
    if (C < 1 || H < 1) return 0;
    return out_prepared_bytes(C, H);
}

int bnn_output_prepare(const float* Wout, int ldw, int C, int H,
                       void* prepared, size_t prepared_bytes, void* stream) {
    if (!Wout || !prepared) return BNN_ERR_NULL;
    if (C < 1 || H < 1 || ldw < H) return BNN_ERR_SHAPE;
    if (prepared_bytes < out_prepared_bytes(C, H)) return BNN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(prepared) & 255u) return BNN_ERR_ALIGN;
    return launch_out_prepare(Wout, ldw, C, H, prepared, (cudaStream_t)stream);
}

static int output_layer_impl(const uint32_t* Hp, int ldhp, const float* Hf, int ldhf,
                             const float* Wout, int ldw, const float* b, const void* prepared,
                             int M, int C, int H, float* logp, int ldo, int log_softmax,
                             int zo, void* workspace, size_t workspace_bytes, const float* log_prior,
                             int act, void* mid_event, void* stream, bool image_ready = false,
                             int* done = nullptr) {
    if (int rc = check_dims(M, C, H)) return rc;
    if (act != BNN_ACT_NONE && (Hp || log_softmax || (act != BNN_ACT_SIGMOID && act != BNN_ACT_HARDTANH)))
        return BNN_ERR_UNSUPPORTED;
    if (!Wout || !logp) return BNN_ERR_NULL;
    if ((Hp == nullptr) == (Hf == nullptr)) return Hp ? BNN_ERR_UNSUPPORTED : BNN_ERR_NULL;
    if (ldw < H || ldo < C) return BNN_ERR_SHAPE;
    RealGemmArgs a{};
    if (Hp) {
        if (int rc = check_packed(Hp, ldhp, H)) return rc;
        a.Ab = Hp; a.lda = ldhp; a.a_zero_one = zo;
    } else {
        if (ldhf < H) return BNN_ERR_SHAPE;
        a.Af = Hf; a.lda = ldhf;
    }
    a.Bf = Wout; a.ldb = ldw;
    a.M = M; a.N = C; a.K = H;
    a.shift = b;
    a.act = act;
    a.Y = logp; a.ldy = ldo;
    if (prepared && (reinterpret_cast<uintptr_t>(prepared) & 255u)) return BNN_ERR_ALIGN;
    int rc;
    // `done` (zeroed counters in the caller's workspace): the log-softmax kernel is launched right behind
    // the tensor-core kernel and takes each group of frames as soon as all its logits are stored
    const bool follow = done && Hp && prepared && g_real_path != BNN_PATH_CUDA_CORE && log_softmax && !mid_event &&
                        g_softmax_follow && log_softmax_can_follow(logp, ldo, C, log_prior) &&
                        out_tc_more_than_one_wave(M, C);
    if (Hp && prepared && g_real_path != BNN_PATH_CUDA_CORE)
        rc = launch_out_tc(Hp, ldhp, prepared, b, M, C, H, logp, ldo, zo, follow ? done : nullptr, (cudaStream_t)stream);
    else if (Hf && prepared && g_real_path != BNN_PATH_CUDA_CORE && workspace &&
             !(reinterpret_cast<uintptr_t>(workspace) & 255u) && workspace_bytes >= outf_image_bytes(M, H))
        rc = launch_outf_tc(Hf, ldhf, prepared, b, M, C, H, logp, ldo, act, workspace, image_ready, (cudaStream_t)stream);
    else if (image_ready)
        return BNN_ERR_WORKSPACE;
    else
        rc = launch_real_gemm(a, (cudaStream_t)stream);
    if (rc) return rc;
    if (mid_event && cudaEventRecord((cudaEvent_t)mid_event, (cudaStream_t)stream) != cudaSuccess)
        return BNN_ERR_CUDA;
    if (follow)
        return launch_log_softmax_rows_follow(logp, ldo, M, C, log_prior, done, out_tc_group_arrivals(C),
                                              out_tc_group_rows(), (cudaStream_t)stream);
    if (log_softmax) return launch_log_softmax_rows(logp, ldo, M, C, log_prior, (cudaStream_t)stream);
    return BNN_OK;
}

int bnn_output_layer(const uint32_t* Hp, int ldhp, const float* Hf, int ldhf,
                     const float* Wout, int ldw, const float* b, const void* prepared,
                     int M, int C, int H, float* logp, int ldo, int log_softmax,
                     void* stream) {
    return output_layer_impl(Hp, ldhp, Hf, ldhf, Wout, ldw, b, prepared, M, C, H, logp, ldo,
                             log_softmax, 0, nullptr, 0, nullptr, BNN_ACT_NONE, nullptr, stream);
}

int bnn_real_layer(const float* Hf, int ldhf, const float* W, int ldw, const float* bias,
                   const void* prepared, int M, int N, int K, float* Y, int ldy, int act,
                   void* workspace, size_t workspace_bytes, void* stream) {
    if (!Hf) return BNN_ERR_NULL;
    return output_layer_impl(nullptr, 0, Hf, ldhf, W, ldw, bias, prepared, M, N, K, Y, ldy, 0, 0,
                             workspace, workspace_bytes, nullptr, act, nullptr, stream);
}

int bnn_affine_sigmoid_i32(const int32_t* D, int ldd, const float* scale, const float* shift,
                           int M, int N, float* Y, int ldy, void* stream) {
    if (!D || !Y) return BNN_ERR_NULL;
    if (M < 1 || N < 1 || ldd < N || ldy < N) return BNN_ERR_SHAPE;
    if (static_cast<const void*>(D) == static_cast<const void*>(Y) && ldd != ldy) return BNN_ERR_SHAPE;
    return launch_affine_sigmoid_i32(D, ldd, scale, shift, M, N, Y, ldy, (cudaStream_t)stream);
}

size_t bnn_output_workspace_bytes(int M, int H) {
    if (M < 1 || H < 1) return 0;
    return outf_image_bytes(M, H);
}

int bnn_output_layer_ws(const float* Hf, int ldhf, const float* Wout, int ldw, const float* b,
                        const void* prepared, int M, int C, int H, float* logp, int ldo,
                        int log_softmax, void* workspace, size_t workspace_bytes, void* stream) {
    if (!Hf) return BNN_ERR_NULL;
    return output_layer_impl(nullptr, 0, Hf, ldhf, Wout, ldw, b, prepared, M, C, H, logp, ldo,
                             log_softmax, 0, workspace, workspace_bytes, nullptr, BNN_ACT_NONE, nullptr, stream);
}

int bnn_output_layer01(const uint32_t* Hp, int ldhp, const float* Wout, int ldw, const float* b,
                       const void* prepared, int M, int C, int H, float* logp, int ldo,
                       int log_softmax, void* stream) {
    if (!Hp) return BNN_ERR_NULL;
    return output_layer_impl(Hp, ldhp, nullptr, 0, Wout, ldw, b, prepared, M, C, H, logp, ldo,
                             log_softmax, 1, nullptr, 0, nullptr, BNN_ACT_NONE, nullptr, stream);
}

// Layout of the forward workspace: two activation buffers of `half` bytes each, then `sync` bytes of
// counters (the arrival counters of the stacked binary layers, `stack_sync` bytes, then the top
// layer's completed-frame-group counters), then whatever the caller gave beyond that
// (split-activation images).
struct WorkspaceLayout {
    size_t half, stack_sync, sync;
    size_t need() const { return 2 * half + sync; }
};
static WorkspaceLayout workspace_layout(const bnn_model* model, int M) {
    size_t mx = 0;
    int xnor_layers = 0;
    for (int l = 0; l + 1 < model->n_layers; ++l) {
        size_t b = layer_out_bytes(model->layers[l], M);
        if (b > mx) mx = b;
        if (model->layers[l].kind == BNN_LAYER_XNOR) ++xnor_layers;
    }
    const size_t stack = round256(xnor_stack_sync_bytes(M, xnor_layers));
    const bool top = model->layers[model->n_layers - 1].kind == BNN_LAYER_REAL_OUT && model->n_layers > 1;
    return WorkspaceLayout{round256(mx), stack, stack + (top ? round256(out_tc_done_bytes(M)) : 0)};
}

size_t bnn_forward_min_workspace_bytes(const bnn_model* model, int M) {
    if (validate_model(model) != BNN_OK || M < 1) return 0;
    return workspace_layout(model, M).need();
}

size_t bnn_forward_workspace_bytes(const bnn_model* model, int M) {
    const size_t base = bnn_forward_min_workspace_bytes(model, M);
    if (base == 0) return 0;
    size_t img = 0;
    for (int l = 0; l < model->n_layers; ++l) {
        const bnn_layer& y = model->layers[l];
        size_t b = 0;
        if (y.kind == BNN_LAYER_SIGNW) {
            b = signw_image_bytes(M, y.K, 3);  // room for either term count
            // a layer of this kind that feeds another one writes that layer's image while it reads its own
            if (y.act != BNN_ACT_SIGN_PACK && l + 1 < model->n_layers && model->layers[l + 1].kind != BNN_LAYER_XNOR)
                b = 2 * round256(signw_image_bytes(M, y.N > y.K ? y.N : y.K, 3));
        } else if (y.kind == BNN_LAYER_REAL ||
                   (y.kind == BNN_LAYER_REAL_OUT && l > 0 && model->layers[l - 1].act != BNN_ACT_SIGN_PACK)) {
            b = outf_image_bytes(M, y.K);      // fp32 activations into a real-valued layer
        }
        if (b > img) img = b;
    }
    return base + round256(img);
}

int bnn_forward(const bnn_model* model, const float* X, int ldx, int M,
                float* logp, int ldo, void* workspace, size_t workspace_bytes,
                void* const* layer_out, void* stream) {
    return bnn_forward_events(model, X, ldx, M, logp, ldo, workspace, workspace_bytes, layer_out,
                              nullptr, stream);
}

int bnn_forward_events(const bnn_model* model, const float* X, int ldx, int M,
                       float* logp, int ldo, void* workspace, size_t workspace_bytes,
                       void* const* layer_out, void* const* events, void* stream) {
    if (int rc = validate_model(model)) return rc;
    if (!X || !logp) return BNN_ERR_NULL;
    // context window formed inside the first layer: X holds K / (left + right + 1) features per frame
    const int ctx = model->splice_left + model->splice_right + 1;
    if (model->splice_left < 0 || model->splice_right < 0) return BNN_ERR_SHAPE;
    if (ctx > 1 && (model->layers[0].K % ctx != 0 || model->layers[0].kind != BNN_LAYER_SIGNW)) return BNN_ERR_SHAPE;
    const int splice_dim = ctx > 1 ? model->layers[0].K / ctx : 0;
    if (M < 1 || ldx < (ctx > 1 ? splice_dim : model->layers[0].K)) return BNN_ERR_SHAPE;
    const int L = model->n_layers;
    if (ldo < model->layers[L - 1].N) return BNN_ERR_SHAPE;
    const WorkspaceLayout lay = workspace_layout(model, M);
    const size_t need = lay.need();
    if (L > 1) {
        if (!workspace || workspace_bytes < need) return BNN_ERR_WORKSPACE;
        if (reinterpret_cast<uintptr_t>(workspace) & 255u) return BNN_ERR_ALIGN;
    }
    // everything that can be refused is checked before the first launch
    for (int l = 0; l + 1 < L; ++l)
        if (layer_out && layer_out[l] && model->layers[l].act == BNN_ACT_SIGN_PACK && !aligned16(layer_out[l]))
            return BNN_ERR_ALIGN;
    char* buf[2] = {static_cast<char*>(workspace), static_cast<char*>(workspace) + lay.half};
    int* sync = reinterpret_cast<int*>(static_cast<char*>(workspace) + 2 * lay.half);
    // whatever lies beyond the two activation buffers and the counters serves the split-activation images
    char* img = static_cast<char*>(workspace) + need;
    const size_t img_bytes = workspace_bytes > need ? workspace_bytes - need : 0;
    const void* in = X;
    int in_ld = ldx;
    bool in_bits = false;
    // A handful of frames: the layers made of packed bits take the matrix-vector kernels, which
    // spread the weights over all SMs instead of tiling the frames (small_batch.cu).
    const bool small = g_small_batch && M <= kSmallBatchMax;
    const int zo01 = model->act_values == BNN_VALUES_01;
    // The arrival counters of stacked binary layers are cleared before the first layer's kernels, not
    // in front of the stacked launch itself: a memset between the first layer's kernel and that launch
    // would take away its programmatic overlap with the first layer's tail.
    // The same goes for the counters on which the log-softmax follows the top layer's kernel.
    int* top_done = nullptr;
    bool clear_pending = false, clear_by_first = false;
    if (!small && lay.sync > 0) {
        bool any = false;
        for (int l = 0; g_xnor_stack && l + 1 < L && !any; ++l)
            any = stackable(model, l) && stackable(model, l + 1) && model->layers[l].N == model->layers[l].K &&
                  model->layers[l + 1].N == model->layers[l].N && model->layers[l + 1].K == model->layers[l].K;
        const bnn_layer& top = model->layers[L - 1];
        if (g_softmax_follow && !events && lay.sync > lay.stack_sync && top.kind == BNN_LAYER_REAL_OUT && top.W_prepared &&
            L > 1 && model->layers[L - 2].act == BNN_ACT_SIGN_PACK && out_tc_more_than_one_wave(M, top.N))
            top_done = sync + lay.stack_sync / sizeof(int);
        clear_pending = any || top_done;
        // When the first layer splits its input into an image, that kernel clears them on its way (a memset
        // node of its own costs about 4 us per step in a replayed graph); otherwise a memset does.
        clear_by_first = clear_pending && model->layers[0].kind == BNN_LAYER_SIGNW && g_real_path != BNN_PATH_CUDA_CORE;
        if (clear_pending && !clear_by_first) {
            if (cudaMemsetAsync(sync, 0, lay.sync, (cudaStream_t)stream) != cudaSuccess) return BNN_ERR_CUDA;
            clear_pending = false;
        }
    }
    bool chain_in = false;   // the layer before wrote this layer's split-activation image (slot chain_slot)
    int chain_slot = 0;
    size_t img_half = 0;     // bytes of one of the two alternating images: the largest any sign-weight layer reads
    for (int l = 0; l < L; ++l)
        if (model->layers[l].kind == BNN_LAYER_SIGNW) {
            size_t b = round256(signw_image_bytes(M, model->layers[l].K, g_signw_terms));
            if (b > img_half) img_half = b;
            // the real-valued layer it may feed reads an image of its own format
            if (l + 1 < L && (model->layers[l + 1].kind == BNN_LAYER_REAL_OUT || model->layers[l + 1].kind == BNN_LAYER_REAL)) {
                b = round256(outf_image_bytes(M, model->layers[l].N));
                if (b > img_half) img_half = b;
            }
        }
    int sync_used = 0;   // counters handed to earlier runs of this call
    for (int l = 0; l < L; ++l) {
        const bnn_layer& y = model->layers[l];
        if (events && events[l] &&
            cudaEventRecord((cudaEvent_t)events[l], (cudaStream_t)stream) != cudaSuccess)
            return BNN_ERR_CUDA;
        if (y.kind == BNN_LAYER_REAL_OUT && small && in_bits && small_fits_out(y.K)) {
            if (int rc = check_packed(in, in_ld, y.K)) return rc;
            if (int rc = launch_small_out(static_cast<const uint32_t*>(in), in_ld, y.W, y.ldw, y.shift, M, y.N, y.K,
                                          logp, ldo, zo01, (cudaStream_t)stream)) return rc;
            if (events && events[L + 1] &&
                cudaEventRecord((cudaEvent_t)events[L + 1], (cudaStream_t)stream) != cudaSuccess)
                return BNN_ERR_CUDA;
            if (int rc = launch_log_softmax_rows(logp, ldo, M, y.N, model->log_prior, (cudaStream_t)stream)) return rc;
            if (events && events[L] &&
                cudaEventRecord((cudaEvent_t)events[L], (cudaStream_t)stream) != cudaSuccess)
                return BNN_ERR_CUDA;
            return BNN_OK;
        }
        if (y.kind == BNN_LAYER_REAL_OUT) {
            int rc = output_layer_impl(in_bits ? static_cast<const uint32_t*>(in) : nullptr, in_ld,
                                       in_bits ? nullptr : static_cast<const float*>(in), in_ld,
                                       y.W, y.ldw, y.shift, y.W_prepared, M, y.N, y.K, logp, ldo, 1,
                                       in_bits && model->act_values == BNN_VALUES_01,
                                       chain_in ? img + (size_t)chain_slot * img_half : img, chain_in ? img_half : img_bytes,
                                       model->log_prior, BNN_ACT_NONE, events ? events[L + 1] : nullptr, stream, chain_in,
                                       in_bits ? top_done : nullptr);
            if (rc) return rc;
            if (events && events[L] &&
                cudaEventRecord((cudaEvent_t)events[L], (cudaStream_t)stream) != cudaSuccess)
                return BNN_ERR_CUDA;
            return BNN_OK;
        }
        // A run of binary hidden layers of one shape whose weights are prepared goes out as ONE launch
        // of the kernel that keeps a unit tile's weights in shared memory (xnor_gemm_res.cu).
        if (g_xnor_stack && !small && stackable(model, l)) {
            int n = 1;
            while (n < kXnorStackMax && l + n < L && stackable(model, l + n) && model->layers[l + n].N == y.N &&
                   model->layers[l + n].K == y.K && y.N == y.K)
                ++n;
            if (n > 1) {
                XnorStackLayer sl[kXnorStackMax];
                for (int i = 0; i < n; ++i) {
                    const bnn_layer& z = model->layers[l + i];
                    void* o = (layer_out && layer_out[l + i]) ? layer_out[l + i] : buf[(l + i) & 1];
                    sl[i] = XnorStackLayer{z.W_prepared, z.thr, z.flip, static_cast<uint32_t*>(o)};
                    if (i > 0 && events && events[l + i] &&
                        cudaEventRecord((cudaEvent_t)events[l + i], (cudaStream_t)stream) != cudaSuccess)
                        return BNN_ERR_CUDA;
                }
                if (int rc = check_packed(in, in_ld, y.K)) return rc;
                const int ldob = bnn_packed_pitch(y.N);
                if (int rc = launch_xnor_stack(static_cast<const uint32_t*>(in), in_ld, sl, n, M, y.N, y.K, ldob, zo01,
                                               sync + sync_used, true, (cudaStream_t)stream))
                    return rc;
                sync_used += (int)(xnor_stack_sync_bytes(M, n) / sizeof(int));
                in = sl[n - 1].out_bits;
                in_ld = ldob;
                in_bits = true;
                l += n - 1;
                continue;
            }
        }
        void* out = (layer_out && layer_out[l]) ? layer_out[l] : buf[l & 1];
        bnn_epilogue e{};
        e.act = y.act;
        e.sign_mode = model->sign_mode;
        int rc;
        if (small && y.act == BNN_ACT_SIGN_PACK && y.kind == BNN_LAYER_SIGNW && !(l == 0 && splice_dim > 0) &&
            small_fits_real(y.K)) {
            const int ldob = bnn_packed_pitch(y.N);
            rc = launch_small_signw(static_cast<const float*>(in), in_ld, y.Wp, y.ldwp, M, y.N, y.K, y.scale, y.shift,
                                    model->sign_mode, static_cast<uint32_t*>(out), ldob, (cudaStream_t)stream);
            in_ld = ldob;
        } else if (small && y.act == BNN_ACT_SIGN_PACK && y.kind == BNN_LAYER_XNOR && small_fits_bits(y.K)) {
            const int ldob = bnn_packed_pitch(y.N);
            rc = launch_small_xnor(static_cast<const uint32_t*>(in), in_ld, y.Wp, y.ldwp, M, y.N, y.K, y.thr, y.flip,
                                   static_cast<uint32_t*>(out), ldob, zo01, (cudaStream_t)stream);
            in_ld = ldob;
        } else if (y.kind == BNN_LAYER_SIGNW) {
            e.scale = y.scale; e.shift = y.shift;
            float* yf = nullptr;
            int out_ld;
            // A layer of this kind that feeds another one writes its outputs straight into that layer's
            // split-activation image (two images alternate in the scratch beyond the activation buffers),
            // and as fp32 only where the caller asked to see them.
            const bnn_layer* nx = l + 1 < L ? &model->layers[l + 1] : nullptr;
            const bool to_signw = nx && nx->kind == BNN_LAYER_SIGNW && !(small && nx->act == BNN_ACT_SIGN_PACK);
            const bool to_real = nx && (nx->kind == BNN_LAYER_REAL_OUT || nx->kind == BNN_LAYER_REAL) && nx->W_prepared;
            const bool chain_out = y.act != BNN_ACT_SIGN_PACK && (to_signw || to_real) &&
                                   g_real_path != BNN_PATH_CUDA_CORE && img_bytes >= 2 * img_half;
            char* img_in = img + (chain_in ? (size_t)chain_slot * img_half : 0);
            char* img_out = chain_out ? img + (size_t)((chain_in ? chain_slot : 0) ^ 1) * img_half : nullptr;
            if (y.act == BNN_ACT_SIGN_PACK) {
                e.out_bits = static_cast<uint32_t*>(out); e.ldob = bnn_packed_pitch(y.N);
                out_ld = e.ldob;
            } else {
                if (!chain_out || (layer_out && layer_out[l])) yf = static_cast<float*>(out);
                out_ld = y.N;
            }
            bool cleared = false;
            rc = signw_impl(static_cast<const float*>(in), in_ld, y.Wp, y.ldwp, M, y.N, y.K,
                            yf, y.N, &e, img_in, chain_in ? img_half : (chain_out ? img_half : img_bytes),
                            l == 0 ? splice_dim : 0, model->splice_left, stream, chain_in, img_out, to_real ? 1 : 0,
                            (l == 0 && clear_by_first) ? sync : nullptr, (int)(lay.sync / sizeof(int)), &cleared);
            if (l == 0 && clear_pending) {
                // the layer took another kernel than the one that clears the counters: clear them now
                if (rc == BNN_OK && !cleared && cudaMemsetAsync(sync, 0, lay.sync, (cudaStream_t)stream) != cudaSuccess)
                    return BNN_ERR_CUDA;
                clear_pending = false;
            }
            in_ld = out_ld;
            if (chain_out) chain_slot = (chain_in ? chain_slot : 0) ^ 1;
            chain_in = chain_out;
        } else if (y.kind == BNN_LAYER_REAL) {
            if (l == 0 && splice_dim > 0) return BNN_ERR_UNSUPPORTED;
            rc = output_layer_impl(nullptr, 0, static_cast<const float*>(in), in_ld, y.W, y.ldw, y.shift,
                                   y.W_prepared, M, y.N, y.K, static_cast<float*>(out), y.N, 0, 0,
                                   chain_in ? img + (size_t)chain_slot * img_half : img, chain_in ? img_half : img_bytes,
                                   nullptr, y.act, nullptr, stream, chain_in);
            in_ld = y.N;
            chain_in = false;
        } else if (y.act == BNN_ACT_SIGMOID) {
            // binary layer with Sigmoid units: the integer dot products go to the output buffer
            // and are turned into fp32 activations in place
            const bool image = y.W_prepared && g_xnor_path != BNN_PATH_CUDA_CORE && y.K <= kMaxKTensor;
            rc = xnor_gemm_impl(static_cast<const uint32_t*>(in), in_ld, y.Wp, y.ldwp,
                                image ? y.W_prepared : nullptr, M, y.N, y.K, static_cast<int32_t*>(out), y.N,
                                nullptr, model->act_values == BNN_VALUES_01, stream);
            // The real-valued layer that consumes these units reads its activations as an image of fp16
            // terms: when there is room for it the Sigmoid goes straight into that image, else into fp32.
            const bnn_layer* nx = l + 1 < L ? &model->layers[l + 1] : nullptr;
            const size_t need_img = round256(outf_image_bytes(M, y.N));
            const bool to_image = nx && (nx->kind == BNN_LAYER_REAL_OUT || nx->kind == BNN_LAYER_REAL) && nx->W_prepared &&
                                  g_real_path != BNN_PATH_CUDA_CORE && img_bytes >= need_img && !(layer_out && layer_out[l]);
            if (!rc && to_image) {
                rc = launch_outf_image_from_i32(static_cast<const int32_t*>(out), y.N, y.scale, y.shift, M, y.N, img,
                                                (cudaStream_t)stream);
                chain_in = true; chain_slot = 0;
                if (img_half < need_img) img_half = need_img;
            } else if (!rc) {
                rc = launch_affine_sigmoid_i32(static_cast<const int32_t*>(out), y.N, y.scale, y.shift, M, y.N,
                                               static_cast<float*>(out), y.N, (cudaStream_t)stream);
            }
            in_ld = y.N;
        } else {
            e.thr = y.thr; e.flip = y.flip;
            e.out_bits = static_cast<uint32_t*>(out); e.ldob = bnn_packed_pitch(y.N);
            const bool image = y.W_prepared && g_xnor_path != BNN_PATH_CUDA_CORE && y.K <= kMaxKTensor;
            rc = xnor_gemm_impl(static_cast<const uint32_t*>(in), in_ld, y.Wp, y.ldwp,
                                image ? y.W_prepared : nullptr, M, y.N, y.K, nullptr, 0, &e,
                                model->act_values == BNN_VALUES_01, stream);
            in_ld = e.ldob;
        }
        if (rc) return rc;
        in = out;
        in_bits = y.act == BNN_ACT_SIGN_PACK;
    }
    return BNN_OK;
}

}  // extern "C"
