// Shared device/host helpers of the sm_100a binarised-DNN forward library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "bnn.h"

namespace bnn {

constexpr int kSignZeroPos = BNN_SIGN_ZERO_POS;
constexpr int kSignZeroNeg = BNN_SIGN_ZERO_NEG;

// Eq. 3: +1 iff x > 0 (ZERO_NEG, as printed) or x >= 0 (ZERO_POS).  NaN -> false.
__device__ __forceinline__ bool sign_is_pos(float x, int mode) {
    return mode == kSignZeroNeg ? (x > 0.0f) : (x >= 0.0f);
}

__host__ __device__ __forceinline__ int words_for(int k) { return (k + 31) >> 5; }
__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Mask that keeps the valid bits of the last word of a K-bit row.
__host__ __device__ __forceinline__ uint32_t tail_mask(int k) {
    int t = k & 31;
    return t ? ((1u << t) - 1u) : 0xFFFFFFFFu;
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, bool valid) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    int bytes = valid ? 16 : 0;  // src-size 0 => the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// 16-byte read-only global load issued exactly where it is written (a volatile asm keeps its place
// among the other volatile statements: barrier waits, shared-memory stores).  Producer warps use it
// to fetch operands for later pipeline stages while they work on the current one.
__device__ __forceinline__ uint4 ldg_nc_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Programmatic dependent launch, used by the kernel of the binary hidden layers: it starts with
// pdl_trigger() (the kernel after it in the stream may be scheduled as soon as all CTAs of this
// one have got that far and SM resources free up), does what does not depend on the kernel
// before it (set-up, the copy of its weight slice) and calls pdl_wait() before it reads that
// kernel's output: the wait returns once the kernel before it has completed and its writes are
// visible.  A kernel of this kind cannot finish before its wait returns, so completion of one
// implies completion of everything before it in the stream.  (Measured on B200: giving the
// other kernels of the forward the same treatment, with the wait right after their set-up,
// made the step 1 % slower instead of faster, so they are launched the ordinary way.)
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with programmatic stream serialisation allowed (see above).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? BNN_OK : BNN_ERR_CUDA; }

// ---- launchers implemented in the .cu files (host side, arguments already validated) ----
int launch_sign_pack(const float* X, int M, int K, int ldx, uint32_t* P, int ldp, int mode,
                     cudaStream_t st);
int launch_fold_thresholds(const float* scale, const float* shift, int N, int K, int mode,
                           int32_t* thr, uint32_t* flip, cudaStream_t st);
// `zo` != 0 in the binary GEMMs below: the bits of the frame operand stand for (0,1) instead of
// (-1,+1), so the result is sum_k h*w with h in {0,1} and w in {-1,+1}.
int launch_xnor_popc(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                     int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                     uint32_t* out_bits, int ldob, int zo, cudaStream_t st);

// Tensor-core (tcgen05) XNOR GEMM; same contract as launch_xnor_popc.  K <= kMaxKTensor.
constexpr int kMaxKTensor = 1 << 22;
int launch_xnor_tc(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                   int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                   uint32_t* out_bits, int ldob, int zo, cudaStream_t st);
// The same product with the unit operand given as the image launch_xnor_prepare built from the
// packed weights (xnor_gemm_img.cu): xnor_image_bytes(N, K) bytes, 256-byte aligned.
size_t xnor_image_bytes(int N, int K);
// Units per chunk of the image: N rounded up to a multiple of 384 (tiles of 192 or 128 units).
__host__ __device__ __forceinline__ int xnor_image_npad(int N) { return ceil_div(N, 384) * 384; }
// Fused Sign layer with the weights of a unit tile resident in shared memory (xnor_gemm_res.cu);
// xnor_res_applicable says whether a layer of this shape fits that kernel.
bool xnor_res_applicable(int N, int K);
int launch_xnor_res(const uint32_t* Ap, int ldap, const void* image, int M, int N, int K,
                    const int32_t* thr, const uint32_t* flip, uint32_t* out_bits, int ldob, int zo, cudaStream_t st);
// A run of consecutive fused Sign layers of one shape (N == K beyond the first) in ONE launch of that
// kernel: layer l reads the bits layer l - 1 wrote (pitch ldob), layer 0 reads Ap.  `progress` points
// to xnor_stack_sync_bytes(M, n_layers) bytes of ZEROED device memory (per frame tile and layer
// boundary a counter of the unit tiles that have stored their bits).  `chained`: the launch is part of a
// forward pass (programmatic dependent launch on the layer kernel before it).
constexpr int kXnorStackMax = 8;
struct XnorStackLayer {
    const void* image;
    const int32_t* thr;
    const uint32_t* flip;
    uint32_t* out_bits;
};
size_t xnor_stack_sync_bytes(int M, int n_layers);
int launch_xnor_stack(const uint32_t* Ap, int ldap, const XnorStackLayer* layers, int n_layers, int M, int N, int K,
                      int ldob, int zo, int* progress, bool chained, cudaStream_t st);
int launch_xnor_prepare(const uint32_t* Wp, int ldwp, int N, int K, void* image, cudaStream_t st);
int launch_xnor_img(const uint32_t* Ap, int ldap, const void* image, int M, int N, int K,
                    int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                    uint32_t* out_bits, int ldob, int zo, cudaStream_t st);
// Small batches (small_batch.cu): plain kernels that spread a layer's weights over all SMs, one
// warp per output unit, for M <= kSmallBatchMax frames.
constexpr int kSmallBatchMax = 16;
// Whether a layer of fan-in K fits those kernels: they stage the batch's operand in dynamic shared
// memory (16 x K floats for real input, 16 x K bits for packed input) next to up to 1 KB of static
// arrays, and the two together must stay within the 48 KB a kernel gets without opting in.
constexpr size_t kSmallSmemMax = 47 * 1024;
inline bool small_fits_real(int K) { return (size_t)kSmallBatchMax * K * sizeof(float) <= kSmallSmemMax; }
inline bool small_fits_bits(int K) { return (size_t)kSmallBatchMax * words_for(K) * sizeof(uint32_t) <= kSmallSmemMax; }
inline bool small_fits_out(int H) { return (size_t)words_for(H) * 32 * sizeof(uint16_t) <= kSmallSmemMax; }
int launch_small_signw(const float* X, int ldx, const uint32_t* Wp, int ldwp, int M, int N, int K,
                       const float* scale, const float* shift, int sign_mode,
                       uint32_t* out_bits, int ldob, cudaStream_t st);
int launch_small_xnor(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N, int K,
                      const int32_t* thr, const uint32_t* flip, uint32_t* out_bits, int ldob, int zo,
                      cudaStream_t st);
int launch_small_out(const uint32_t* Hp, int ldhp, const float* W, int ldw, const float* bias,
                     int M, int C, int H, float* Z, int ldz, int zo, cudaStream_t st);
// Pipe micro-benchmarks (pipe_rates.cu).
size_t pipe_rate_scratch_bytes(int which);
int launch_pipe_rate(int which, int repeat, void* scratch, size_t scratch_bytes, double* work, cudaStream_t st);
// Tensor map of a packed operand [rows][ceil(K/32) words] of pitch `ld` words: boxes of 16 words x
// box_rows rows, 64-byte swizzle, zero fill outside the tensor.  False when the encoder fails.
bool encode_packed_map(CUtensorMap* map, const uint32_t* base, int ld, int rows, int K, int box_rows);
// Reads (synchronously) the word that a tensor-core kernel sets when a bounded wait ran out.
int read_tc_status(int* out);
// The same as a copy enqueued on `st` (dst: device or pinned host memory), and the reset of the word.
int copy_tc_status_async(int* dst, cudaStream_t st);
int reset_tc_status_async(cudaStream_t st);
// Limit of every bounded wait in SM clocks; returns the previous value.
long long set_wait_limit_clocks(long long clocks);
// A one-warp launch whose wait runs out (see tc_support.cu).
int launch_wait_probe(cudaStream_t st);
// Per-device bookkeeping of the launchers: SM count of the current device (0 on failure), and
// cudaFuncAttributeMaxDynamicSharedMemorySize raised once per device and kernel.
int device_sm_count();
bool ensure_dynamic_smem(const void* kernel, int bytes);

// Real-valued GEMM on the FP32 pipe: D[m][n] = sum_k A[m][k]*B[n][k], where each operand is
// either fp32 or packed +-1 bits.
struct RealGemmArgs {
    const float* Af;      // fp32 A [M][lda] or nullptr
    int splice_dim;       // > 0: row m of A is the concatenation of rows clamp(m - splice_left + t)
    int splice_left;      //      (t = 0 .. K/splice_dim - 1) of an fp32 matrix [M][lda] of splice_dim columns
    const uint32_t* Ab;   // packed A [M][lda] or nullptr
    int a_zero_one;       // packed A stands for (0,1) instead of (-1,+1)
    int lda;
    const float* Bf;      // fp32 B [N][ldb] or nullptr
    const uint32_t* Bb;   // packed B [N][ldb] or nullptr
    int ldb;
    int M, N, K;
    const float* scale;   // [N] or nullptr
    const float* shift;   // [N] or nullptr
    int act;              // bnn_act
    int sign_mode;
    float* Y;             // fp32 out [M][ldy] or nullptr
    int ldy;
    uint32_t* out_bits;   // packed out [M][ldob] or nullptr
    int ldob;
};
int launch_real_gemm(const RealGemmArgs& a, cudaStream_t st);
// Tensor-core versions: +-1 weights x real input (A fp32, B bits; `terms` bf16 terms), and
// the top layer on packed activations with prepared fp16 weight terms.
int launch_signw_tc(const RealGemmArgs& a, int terms, cudaStream_t st);
// Same product with the activations split once into a scratch image (see signw_img_tc.cu):
// `workspace` must hold signw_image_bytes(M, K, terms) bytes, 256-byte aligned.
size_t signw_image_bytes(int M, int K, int terms);
// image_ready: `workspace` already holds the image of a.Af's values (a.Af is not read then);
// out_image (256-byte aligned, signw_image_bytes(M, N, terms) bytes) or nullptr: the outputs are also
// written as the image of a following layer of this kind with fan-in N.
// out_kind 0: that layer's own image (bf16 terms, blocks of 128 frames); 1: the image the real-valued
// layer on fp32 activations reads (two fp16 terms, blocks of 256 frames, outf_image_bytes(M, N) bytes).
// clear / clear_words (optional, only with image_ready == false): words the splitting kernel sets to zero on
// its way -- bnn_forward's counters, which would otherwise need a memset of their own in front of it.
int launch_signw_img(const RealGemmArgs& a, int terms, void* workspace, bool image_ready, void* out_image, int out_kind,
                     int* clear, int clear_words, cudaStream_t st);
size_t out_prepared_bytes(int C, int H);
int launch_out_prepare(const float* W, int ldw, int C, int H, void* prepared, cudaStream_t st);
// `done` (optional, out_tc_done_bytes(M) zeroed bytes): one counter per out_tc_group_rows() frames, then
// the row counter of the kernel that follows; every epilogue warp adds 1 to a group's counter once its
// share of a tile of that group is stored; out_tc_group_arrivals(C) arrivals complete a group.
// launch_log_softmax_rows_follow, launched right behind, consumes the groups in order.
int out_tc_group_rows();
int out_tc_group_arrivals(int C);
size_t out_tc_done_bytes(int M);
bool out_tc_more_than_one_wave(int M, int C);
int launch_out_tc(const uint32_t* Hp, int ldhp, const void* prepared, const float* bias,
                  int M, int C, int H, float* Z, int ldz, int zo, int* done, cudaStream_t st);
bool log_softmax_can_follow(const float* Z, int ldz, int C, const float* prior);
int launch_log_softmax_rows_follow(float* Z, int ldz, int M, int C, const float* prior, int* done, int need,
                                   int group_rows, cudaStream_t st);
// The top layer on fp32 activations (finite, |a| < 65504) with both operands split into fp16
// terms (out_gemm_f32_tc.cu): `workspace` holds outf_image_bytes(M, H) bytes, 256-byte aligned.
size_t outf_image_bytes(int M, int H);
// `act`: bnn_act applied after the bias (NONE, SIGMOID, HARDTANH).  image_ready: `workspace` already
// holds the fp16 image of the activations (written by launch_signw_img with out_kind 1); Hf is not read.
int launch_outf_tc(const float* Hf, int ldhf, const void* prepared, const float* bias,
                   int M, int C, int H, float* Z, int ldz, int act, void* workspace, bool image_ready, cudaStream_t st);
// The image launch_outf_tc reads (image_ready), made from integer dot products D [M][ldd]: the activations
// are Sigmoid(fma(scale[h], d, shift[h])).  image: outf_image_bytes(M, H) bytes, 256-byte aligned.
int launch_outf_image_from_i32(const int32_t* D, int ldd, const float* scale, const float* shift, int M, int H,
                               void* image, cudaStream_t st);
// Y = Sigmoid(fma(scale, D, shift)) element by element (Y may alias D when the pitches agree).
int launch_affine_sigmoid_i32(const int32_t* D, int ldd, const float* scale, const float* shift,
                              int M, int N, float* Y, int ldy, cudaStream_t st);
// Z <- log softmax of each row, minus prior[c] when `prior` (device, [C]) is given.
int launch_log_softmax_rows(float* Z, int ldz, int M, int C, const float* prior, cudaStream_t st);

}  // namespace bnn
