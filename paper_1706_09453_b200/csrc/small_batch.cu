// Small batches (1 .. 16 frames): the matrix-vector regime the paper has in mind for embedded
// recognisers.  With so few frames the tiled tensor-core kernels leave almost the whole GPU idle
// and pay their set-up (tensor memory, barriers, a 192 KB weight slice per CTA) for one nearly
// empty tile; what matters here is to spread each layer's WEIGHTS over all SMs and to read them
// once.  Three plain kernels on the integer / FP32 pipes, one warp per output unit:
//
//   small_signw_kernel   y[m][n] = sum_k w[n][k] x[m][k], w = +-1 from packed bits, then the
//                        per-unit affine, Sign and packing (first layer)
//   small_xnor_kernel    d[m][n] = K - 2 popc(a[m] xor w[n])  (or 2 popc(a and w) - popc(a) for
//                        (0,1) frames), threshold, packing (binary hidden layers)
//   small_out_kernel     z[m][c] = sum_n Wout[c][n] h[m][n] + b[c] on packed h (top layer, fp32)
//
// A block of 32 warps owns 32 consecutive units, so that one ballot per frame yields a whole
// packed word of the next layer's input.  Lane l of a warp takes the positions k = l, l + 32, ...
// of the unit's row; the per-frame partial sums are reduced with shuffles.  Integer results are
// exact; the fp32 sums differ from the oracle only by the order of fp32 additions.
#include "bnn_common.cuh"

namespace bnn {

namespace {

constexpr int MAXM = kSmallBatchMax;   // frames per launch

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// The kernels are instantiated for MT = 1, 4 and 16 frames (the smallest that holds the batch is
// launched), so that a single frame does not pay for sixteen.
// Warp 0 turns the block's 32 x M decisions (dec[unit][frame]) into one packed word per frame.
__device__ __forceinline__ void pack_block(const unsigned char (*dec)[MAXM], int M, int n0, int N,
                                           uint32_t* __restrict__ out_bits, int ldob, int lane) {
    for (int m = 0; m < M; ++m) {
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, (n0 + lane < N) && dec[lane][m]);
        if (lane == 0) out_bits[(size_t)m * ldob + (n0 >> 5)] = word;
    }
}

template <int MT>
__global__ void __launch_bounds__(1024)
small_signw_kernel(const float* __restrict__ X, int ldx, const uint32_t* __restrict__ Wp, int ldwp,
                   int M, int N, int K, const float* __restrict__ scale, const float* __restrict__ shift,
                   int sign_mode, uint32_t* __restrict__ out_bits, int ldob) {
    __shared__ unsigned char dec[32][MAXM];
    extern __shared__ float xs[];   // the batch's input, [MT][K]; rows >= M are zero
    __shared__ float xsum[MT];      // sum_k x[m][k], the same for every unit
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * 32, n = n0 + warp;
    for (int i = threadIdx.x; i < MT * K; i += blockDim.x) {
        const int m = i / K, k = i - m * K;
        xs[i] = m < M ? __ldg(X + (size_t)m * ldx + k) : 0.f;
    }
    __syncthreads();
    if (warp < MT) {   // warp m adds up row m
        float t = 0.f;
        for (int k = lane; k < K; k += 32) t += xs[warp * K + k];
        t = warp_sum(t);
        if (lane == 0) xsum[warp] = t;
    }
    __syncthreads();
    // sum_k w x = 2 * (sum of x where the weight bit is set) - sum_k x: one predicated add per
    // position and frame
    float acc[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[m] = 0.f;
    if (n < N) {
        const uint32_t* w = Wp + (size_t)n * ldwp;
        for (int k0 = 0; k0 < K; k0 += 32) {
            const int k = k0 + lane;
            const bool plus = (__ldg(w + (k0 >> 5)) >> lane) & 1u;
            if (k < K && plus) {
#pragma unroll
                for (int m = 0; m < MT; ++m) acc[m] += xs[m * K + k];
            }
        }
    }
    const float sc = (scale && n < N) ? scale[n] : 1.0f, sh = (shift && n < N) ? shift[n] : 0.0f;
#pragma unroll
    for (int m = 0; m < MT; ++m)
        if (m < M) {
            const float y = fmaf(sc, 2.0f * warp_sum(acc[m]) - xsum[m], sh);
            if (lane == 0) dec[warp][m] = sign_is_pos(y, sign_mode);
        }
    __syncthreads();
    if (warp == 0) pack_block(dec, M, n0, N, out_bits, ldob, lane);
}

template <bool ZO, int MT>
__global__ void __launch_bounds__(1024)
small_xnor_kernel(const uint32_t* __restrict__ Ap, int ldap, const uint32_t* __restrict__ Wp, int ldwp,
                  int M, int N, int K, const int32_t* __restrict__ thr, const uint32_t* __restrict__ flip,
                  uint32_t* __restrict__ out_bits, int ldob) {
    __shared__ unsigned char dec[32][MAXM];
    extern __shared__ uint32_t as[];   // the batch's packed frames, [MT][kw]; rows >= M are zero
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * 32, n = n0 + warp;
    const int kw = words_for(K);
    const uint32_t tmask = tail_mask(K);
    for (int i = threadIdx.x; i < MT * kw; i += blockDim.x) {
        const int m = i / kw, g = i - m * kw;
        as[i] = m < M ? __ldg(Ap + (size_t)m * ldap + g) : 0u;
    }
    __syncthreads();
    int acc[MT], ones[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) { acc[m] = 0; ones[m] = 0; }
    if (n < N) {
        const uint32_t* w = Wp + (size_t)n * ldwp;
        for (int g = lane; g < kw; g += 32) {
            const uint32_t valid = g == kw - 1 ? tmask : 0xFFFFFFFFu;   // bits >= K hold anything
            const uint32_t wv = __ldg(w + g);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint32_t a = as[m * kw + g];
                if (ZO) { acc[m] += __popc(a & wv & valid); ones[m] += __popc(a & valid); }
                else acc[m] += __popc((a ^ wv) & valid);
            }
        }
    }
    const int t = n < N ? thr[n] : 0;
    const bool f = n < N ? ((flip[n >> 5] >> (n & 31)) & 1u) : false;
#pragma unroll
    for (int m = 0; m < MT; ++m)
        if (m < M) {
            const int p = warp_sum(acc[m]);
            const int d = ZO ? 2 * p - warp_sum(ones[m]) : K - 2 * p;
            if (lane == 0) dec[warp][m] = (d >= t) != f;
        }
    __syncthreads();
    if (warp == 0) pack_block(dec, M, n0, N, out_bits, ldob, lane);
}

// One warp per class; 8 classes per block.
template <bool ZO, int MT>
__global__ void __launch_bounds__(256)
small_out_kernel(const uint32_t* __restrict__ Hp, int ldhp, const float* __restrict__ W, int ldw,
                 const float* __restrict__ bias, int M, int C, int H, float* __restrict__ Z, int ldz) {
    // fm[g][lane]: bit m set <=> frame m has a one at position 32 g + lane (frames >= M: clear).
    // Built once per block; the inner loop then needs one shared-memory load per weight.
    extern __shared__ uint16_t fm[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hw = words_for(H);
    for (int i = threadIdx.x; i < hw * 32; i += blockDim.x) {
        const int g = i >> 5, l = i & 31;
        uint32_t t = 0u;
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < M) t |= ((__ldg(Hp + (size_t)m * ldhp + g) >> l) & 1u) << m;
        fm[i] = (uint16_t)t;
    }
    __syncthreads();
    const int c = blockIdx.x * 8 + warp;
    if (c >= C) return;
    const float* w = W + (size_t)c * ldw;
    // acc[m] = sum of the weights at the positions where frame m's bit is set (one predicated add
    // per weight and frame); with +-1 activations z = 2 acc - (sum of all weights of the class).
    float acc[MT], tot = 0.f;
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[m] = 0.f;
    // eight independent loads of the class's weights in flight per lane: this kernel is bound by
    // how fast the 4 bytes per weight arrive
    for (int g0 = 0; g0 < hw; g0 += 8) {
        float wv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int n = (g0 + u) * 32 + lane;
            wv[u] = n < H ? __ldg(w + n) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (g0 + u < hw) {
                tot += wv[u];
                const uint32_t t = fm[(g0 + u) * 32 + lane];
#pragma unroll
                for (int m = 0; m < MT; ++m)
                    if (t & (1u << m)) acc[m] += wv[u];
            }
        }
    }
    const float b = bias ? bias[c] : 0.f;
    tot = warp_sum(tot);
#pragma unroll
    for (int m = 0; m < MT; ++m)
        if (m < M) {
            const float s1 = warp_sum(acc[m]);
            const float z = (ZO ? s1 : 2.0f * s1 - tot) + b;
            if (lane == 0) Z[(size_t)m * ldz + c] = z;
        }
}

}  // namespace

#define BNN_SMALL_DISPATCH(M, CALL) \
    do { if ((M) <= 1) { constexpr int MT = 1; CALL; } else if ((M) <= 4) { constexpr int MT = 4; CALL; } \
         else { constexpr int MT = 16; CALL; } } while (0)
static int frames_bound(int M) { return M <= 1 ? 1 : (M <= 4 ? 4 : 16); }

int launch_small_signw(const float* X, int ldx, const uint32_t* Wp, int ldwp, int M, int N, int K,
                       const float* scale, const float* shift, int sign_mode,
                       uint32_t* out_bits, int ldob, cudaStream_t st) {
    const size_t smem = (size_t)frames_bound(M) * K * sizeof(float);
    if (M > MAXM || smem > kSmallSmemMax) return BNN_ERR_UNSUPPORTED;
    BNN_SMALL_DISPATCH(M, (small_signw_kernel<MT><<<ceil_div(N, 32), 1024, smem, st>>>(X, ldx, Wp, ldwp, M, N, K, scale, shift,
                                                                                      sign_mode, out_bits, ldob)));
    return launch_status();
}

int launch_small_xnor(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N, int K,
                      const int32_t* thr, const uint32_t* flip, uint32_t* out_bits, int ldob, int zo,
                      cudaStream_t st) {
    const size_t smem = (size_t)frames_bound(M) * words_for(K) * sizeof(uint32_t);
    if (M > MAXM || smem > kSmallSmemMax) return BNN_ERR_UNSUPPORTED;
    if (zo)
        BNN_SMALL_DISPATCH(M, (small_xnor_kernel<true, MT><<<ceil_div(N, 32), 1024, smem, st>>>(Ap, ldap, Wp, ldwp, M, N, K, thr, flip,
                                                                                               out_bits, ldob)));
    else
        BNN_SMALL_DISPATCH(M, (small_xnor_kernel<false, MT><<<ceil_div(N, 32), 1024, smem, st>>>(Ap, ldap, Wp, ldwp, M, N, K, thr, flip,
                                                                                                out_bits, ldob)));
    return launch_status();
}

int launch_small_out(const uint32_t* Hp, int ldhp, const float* W, int ldw, const float* bias,
                     int M, int C, int H, float* Z, int ldz, int zo, cudaStream_t st) {
    const size_t smem = (size_t)words_for(H) * 32 * sizeof(uint16_t);
    if (M > MAXM || smem > kSmallSmemMax) return BNN_ERR_UNSUPPORTED;
    if (zo)
        BNN_SMALL_DISPATCH(M, (small_out_kernel<true, MT><<<ceil_div(C, 8), 256, smem, st>>>(Hp, ldhp, W, ldw, bias, M, C, H, Z, ldz)));
    else
        BNN_SMALL_DISPATCH(M, (small_out_kernel<false, MT><<<ceil_div(C, 8), 256, smem, st>>>(Hp, ldhp, W, ldw, bias, M, C, H, Z, ldz)));
    return launch_status();
}

}  // namespace bnn
