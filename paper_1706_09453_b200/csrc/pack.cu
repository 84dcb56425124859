// Binarisation (Eq. 3) of fp32 matrices into packed sign bits, and folding of the per-unit
// affine + Sign of a binary hidden layer into integer thresholds.
#include "bnn_common.cuh"

namespace bnn {

// One warp turns 128 consecutive elements of a row into four 32-bit words per step.
// HBM-bound: 4 bytes read per element, 1/8 byte written.
template <bool VEC4>
__global__ void __launch_bounds__(256)
sign_pack_kernel(const float* __restrict__ X, int M, int K, int ldx,
                 uint32_t* __restrict__ P, int ldp, int mode) {
    const int lane = threadIdx.x & 31;
    const int groups = (K + 127) >> 7;          // 128-element groups per row
    const int kw = words_for(K);
    const long long tasks = (long long)M * groups;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long t = warp0; t < tasks; t += nwarps) {
        const int row = (int)(t / groups);
        const int g = (int)(t % groups);
        const int k0 = (g << 7) + (lane << 2);
        const float* src = X + (size_t)row * ldx + k0;
        float v[4];
        if (VEC4 && k0 + 3 < K) {
            float4 q = __ldg(reinterpret_cast<const float4*>(src));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) v[c] = (k0 + c < K) ? __ldg(src + c) : -1.0f;
        }
        uint32_t nib = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            nib |= (uint32_t)((k0 + c < K) && sign_is_pos(v[c], mode)) << c;
        uint32_t w = nib << ((lane & 7) << 2);
        w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1);
        w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2);
        w |= __shfl_xor_sync(0xFFFFFFFFu, w, 4);
        // lanes 8j..8j+7 now all hold word 4g+j
        uint32_t w1 = __shfl_sync(0xFFFFFFFFu, w, 8);
        uint32_t w2 = __shfl_sync(0xFFFFFFFFu, w, 16);
        uint32_t w3 = __shfl_sync(0xFFFFFFFFu, w, 24);
        if (lane == 0) {
            uint32_t* dst = P + (size_t)row * ldp + (g << 2);
            if ((g << 2) + 3 < kw) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(w, w1, w2, w3);
            } else {
                uint32_t ws[4] = {w, w1, w2, w3};
                for (int j = 0; j < 4; ++j)
                    if ((g << 2) + j < kw) dst[j] = ws[j];
            }
        }
    }
}

int launch_sign_pack(const float* X, int M, int K, int ldx, uint32_t* P, int ldp, int mode,
                     cudaStream_t st) {
    const long long tasks = (long long)M * ((K + 127) >> 7);
    long long blocks = (tasks + 7) / 8;
    const long long cap = 148LL * 16;  // persistent-style grid: 16 CTAs of 256 threads per SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const bool vec = (ldx % 4 == 0) && aligned16(X);
    if (vec)
        sign_pack_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(X, M, K, ldx, P, ldp, mode);
    else
        sign_pack_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(X, M, K, ldx, P, ldp, mode);
    return launch_status();
}

// Sign(fma(s, d, b)) is monotone in the integer d, so it equals (d >= thr) XOR flip for a
// threshold found by bisection over d in [-K, K] with the very same fma.  thr = K+1 means
// "never", thr = -K means "always".
__global__ void fold_thresholds_kernel(const float* __restrict__ scale,
                                       const float* __restrict__ shift, int N, int K, int mode,
                                       int32_t* __restrict__ thr, uint32_t* __restrict__ flip) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    bool fl = false;
    if (n < N) {
        const float s = scale ? scale[n] : 1.0f;
        const float b = shift ? shift[n] : 0.0f;
        fl = s < 0.0f;
        // first d in [-K, K] with (Sign(fma(s,d,b)) == +1) != fl ; K+1 if there is none
        int lo = -K, hi = K + 1;
        while (lo < hi) {
            const int mid = lo + ((hi - lo) >> 1);
            const bool pred = sign_is_pos(fmaf(s, (float)mid, b), mode) != fl;
            if (pred) hi = mid; else lo = mid + 1;
        }
        thr[n] = lo;
    }
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, fl);
    if ((threadIdx.x & 31) == 0 && n < N) flip[n >> 5] = word;
}

int launch_fold_thresholds(const float* scale, const float* shift, int N, int K, int mode,
                           int32_t* thr, uint32_t* flip, cudaStream_t st) {
    fold_thresholds_kernel<<<ceil_div(N, 128), 128, 0, st>>>(scale, shift, N, K, mode, thr, flip);
    return launch_status();
}

// Binary layer with Sigmoid units: y = Sigmoid(fma(scale[n], d, shift[n])) for the integer dot
// products d; Y may alias D (same pitch): every element is read and written by one thread.
__global__ void affine_sigmoid_i32_kernel(const int32_t* D, int ldd, const float* __restrict__ scale,
                                          const float* __restrict__ shift, int M, int N, float* Y, int ldy) {
    const long long total = (long long)M * N;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int m = (int)(i / N), n = (int)(i % N);
        const float v = fmaf(scale ? scale[n] : 1.0f, (float)D[(size_t)m * ldd + n], shift ? shift[n] : 0.0f);
        Y[(size_t)m * ldy + n] = 1.0f / (1.0f + expf(-v));
    }
}

int launch_affine_sigmoid_i32(const int32_t* D, int ldd, const float* scale, const float* shift,
                              int M, int N, float* Y, int ldy, cudaStream_t st) {
    const long long total = (long long)M * N;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    affine_sigmoid_i32_kernel<<<(int)blocks, 256, 0, st>>>(D, ldd, scale, shift, M, N, Y, ldy);
    return launch_status();
}

}  // namespace bnn
