// Real-valued GEMM on the FP32 pipe where one operand may be packed +-1 bits:
//   D[m][n] = sum_k A[m][k] * B[n][k]
//   - +-1 weights x real activations (additions/subtractions of Section 2.1): A fp32, B bits
//   - real top-layer weights x +-1 activations:                                A bits, B fp32
//   - real top-layer weights x real activations (binary-weights-only nets):    A fp32, B fp32
// followed by the per-unit affine (one fp32 fma) and Sign+pack / hardtanh / identity.
// Also the row-wise log-softmax that finishes the top layer.
//
// CTA tile 128x128, K step 32, 256 threads, 8x8 accumulators per thread.  A bit operand is
// expanded to +-1.0f while it is stored to shared memory, so the inner loop is plain FFMA.
#include <float.h>

#include "bnn_common.cuh"

namespace bnn {

namespace {

constexpr int TM = 128, TN = 128, TK = 32, THREADS = 256;
constexpr int PADW = TM + 4;  // row pitch of the k-major tiles (keeps float4 reads aligned)

struct Operand {
    const float* f;
    const uint32_t* b;
    int ld;
    int rows;
};

// Global -> registers for one K step of a 128-row operand tile.
struct Fetch {
    float4 v[4];
    uint32_t word;
};

template <bool BITS>
__device__ __forceinline__ void fetch(Fetch& r, const Operand& op, int row0, int kbase, int K,
                                      bool vec_ok) {
    const int t = threadIdx.x;
    if (BITS) {
        r.word = 0u;
        if (t < TM) {
            const int row = row0 + t;
            const int wi = kbase >> 5;
            if (row < op.rows && wi < words_for(K)) {
                uint32_t w = __ldg(op.b + (size_t)row * op.ld + wi);
                if (wi == words_for(K) - 1) w &= tail_mask(K);
                r.word = w;
            }
        }
    } else {
        const int kq = t & 7;
        const int k = kbase + kq * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = row0 + (t >> 3) + 32 * i;
            float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
            if (row < op.rows) {
                const float* src = op.f + (size_t)row * op.ld + k;
                if (vec_ok && k + 3 < K) {
                    q = __ldg(reinterpret_cast<const float4*>(src));
                } else {
                    if (k + 0 < K) q.x = __ldg(src + 0);
                    if (k + 1 < K) q.y = __ldg(src + 1);
                    if (k + 2 < K) q.z = __ldg(src + 2);
                    if (k + 3 < K) q.w = __ldg(src + 3);
                }
            }
            r.v[i] = q;
        }
    }
}

// Registers -> shared tile S[k][row] (k-major).  Bits become +1.0f / `low` (-1.0f, or 0.0f for
// activations that stand for (0,1)); positions k >= K of a bit operand become `low`, which is
// harmless because the fp32 operand is zero there.
template <bool BITS>
__device__ __forceinline__ void stash(const Fetch& r, float (*S)[PADW], float low = -1.0f) {
    const int t = threadIdx.x;
    if (BITS) {
        if (t < TM) {
#pragma unroll
            for (int k = 0; k < TK; ++k) S[k][t] = ((r.word >> k) & 1u) ? 1.0f : low;
        }
    } else {
        const int kq = t & 7;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = (t >> 3) + 32 * i;
            S[kq * 4 + 0][row] = r.v[i].x;
            S[kq * 4 + 1][row] = r.v[i].y;
            S[kq * 4 + 2][row] = r.v[i].z;
            S[kq * 4 + 3][row] = r.v[i].w;
        }
    }
}

template <bool A_BITS, bool B_BITS>
__global__ void __launch_bounds__(THREADS, 2)
real_gemm_kernel(RealGemmArgs g) {
    __shared__ __align__(16) float As[TK][PADW];
    __shared__ __align__(16) float Bs[TK][PADW];
    const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
    Operand opa{g.Af, g.Ab, g.lda, g.M}, opb{g.Bf, g.Bb, g.ldb, g.N};
    const bool va = !A_BITS && (g.lda % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.Af) & 15) == 0);
    const bool vb = !B_BITS && (g.ldb % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.Bf) & 15) == 0);

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    Fetch fa, fb;
    fetch<A_BITS>(fa, opa, m0, 0, g.K, va);
    fetch<B_BITS>(fb, opb, n0, 0, g.K, vb);
    for (int kb = 0; kb < g.K; kb += TK) {
        stash<A_BITS>(fa, As, g.a_zero_one ? 0.0f : -1.0f);
        stash<B_BITS>(fb, Bs);
        __syncthreads();
        if (kb + TK < g.K) {
            fetch<A_BITS>(fa, opa, m0, kb + TK, g.K, va);
            fetch<B_BITS>(fb, opb, n0, kb + TK, g.K, vb);
        }
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

    // ---- epilogue: affine (one fma), activation, store ----
    uint8_t (*sb)[TN] = reinterpret_cast<uint8_t (*)[TN]>(&As[0][0]);  // 16 KB <= sizeof(As)
    const bool pack = g.act == BNN_ACT_SIGN_PACK;
    const bool vy = g.Y && (g.ldy % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.Y) & 15) == 0);
#pragma unroll
    for (int jh = 0; jh < 2; ++jh) {
        const int nl = jh * 64 + tx * 4;
        const int n = n0 + nl;
        float sc[4], sh[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            sc[j] = (g.scale && n + j < g.N) ? g.scale[n + j] : 1.0f;
            sh[j] = (g.shift && n + j < g.N) ? g.shift[n + j] : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int ml = (i >> 2) * 64 + ty * 4 + (i & 3);
            const int m = m0 + ml;
            float y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                y[j] = fmaf(sc[j], acc[i][jh * 4 + j], sh[j]);
                if (g.act == BNN_ACT_HARDTANH) y[j] = fminf(fmaxf(y[j], -1.0f), 1.0f);
                if (g.act == BNN_ACT_SIGMOID) y[j] = 1.0f / (1.0f + expf(-y[j]));
            }
            if (pack) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    sb[ml][nl + j] = (n + j < g.N) && sign_is_pos(y[j], g.sign_mode);
            }
            if (g.Y && m < g.M) {
                float* dst = g.Y + (size_t)m * g.ldy + n;
                if (vy && n + 3 < g.N) {
                    *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (n + j < g.N) dst[j] = y[j];
                }
            }
        }
    }
    if (pack) {
        __syncthreads();
        const int lane = t & 31, wy = t >> 5;
        const int nw = words_for(g.N);
        const int w0 = n0 >> 5;
        for (int r = 0; r < 16; ++r) {
            const int ml = wy * 16 + r;
            uint32_t mine = 0u;
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {
                const uint32_t word = __ballot_sync(0xFFFFFFFFu, sb[ml][wd * 32 + lane] != 0);
                if (lane == wd) mine = word;
            }
            const int m = m0 + ml;
            if (lane < 4 && m < g.M && w0 + lane < nw)
                g.out_bits[(size_t)m * g.ldob + w0 + lane] = mine;
        }
    }
}

// Block-wide (max, sum of exp) combination used by both log-softmax kernels.
__device__ __forceinline__ float block_logsumexp(float mx, float s, float* sm, float* ss) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xFFFFFFFFu, mx, o);
        const float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, o);
        const float mn = fmaxf(mx, m2);
        s = s * expf(mx - mn) + s2 * expf(m2 - mn);
        mx = mn;
    }
    if (lane == 0) { sm[w] = mx; ss[w] = s; }
    __syncthreads();
    float gm = sm[0], gs = ss[0];
    for (int i = 1; i < 8; ++i) {
        const float mn = fmaxf(gm, sm[i]);
        gs = gs * expf(gm - mn) + ss[i] * expf(sm[i] - mn);
        gm = mn;
    }
    __syncthreads();
    return gm + logf(gs);
}

// One CTA per row, any C: online (max, sum exp) in one sweep, then z - logsumexp in a second.
__global__ void __launch_bounds__(256)
log_softmax_rows_kernel(float* __restrict__ Z, int ldz, int M, int C, const float* __restrict__ prior) {
    __shared__ float sm[8], ss[8];
    for (int row = blockIdx.x; row < M; row += gridDim.x) {
        float* z = Z + (size_t)row * ldz;
        float mx = -FLT_MAX, s = 0.f;
        for (int c = threadIdx.x; c < C; c += blockDim.x) {
            const float v = z[c];
            if (v > mx) { s *= expf(mx - v); mx = v; }
            s += expf(v - mx);
        }
        const float lse = block_logsumexp(mx, s, sm, ss);
        for (int c = threadIdx.x; c < C; c += blockDim.x) z[c] = z[c] - lse - (prior ? prior[c] : 0.f);
    }
}

// 2^x on the special-function unit (relative error ~2^-22; the arguments here are <= 0).
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Same result with the whole row held in registers (C <= 256*4*V, 16-byte aligned rows):
// every logit is read from memory once and written once.  The maximum is reduced first (warp
// shuffles, then 8 values through shared memory), so each element costs a subtract, a
// multiply, one ex2 and one add; the sum is reduced the same way.
template <int V>
__global__ void __launch_bounds__(256)
log_softmax_rows_reg_kernel(float* __restrict__ Z, int ldz, int M, int C, const float* __restrict__ prior) {
    __shared__ float sm[2][8], ss[2][8];
    const int c4 = C >> 2;  // C % 4 == 0
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    int par = 0;   // the two halves of the scratch alternate, which saves a barrier per row
    // Rows are taken from the last one down: the kernel that wrote the logits just before this one
    // produced the last frames last, and those are the rows the L2 cache still holds.
    for (int r = blockIdx.x; r < M; r += gridDim.x, par ^= 1) {
        const int row = M - 1 - r;
        float4* z = reinterpret_cast<float4*>(Z + (size_t)row * ldz);
        float4 v[V];
        float mx = -FLT_MAX;
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int c = threadIdx.x + i * 256;
            v[i] = c < c4 ? z[c] : make_float4(-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX);
            mx = fmaxf(fmaxf(mx, fmaxf(v[i].x, v[i].y)), fmaxf(v[i].z, v[i].w));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        if (lane == 0) sm[par][w] = mx;
        __syncthreads();
        mx = sm[par][0];
#pragma unroll
        for (int i = 1; i < 8; ++i) mx = fmaxf(mx, sm[par][i]);
        // sum of exp(z - max) = sum of 2^((z - max) log2 e); the difference is taken first, so the
        // rounding error scales with the distance from the maximum, not with the logit itself;
        // padding (-FLT_MAX) contributes 0
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i)
            s += (ex2_approx((v[i].x - mx) * kLog2e) + ex2_approx((v[i].y - mx) * kLog2e)) +
                 (ex2_approx((v[i].z - mx) * kLog2e) + ex2_approx((v[i].w - mx) * kLog2e));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0) ss[par][w] = s;
        __syncthreads();
        s = ss[par][0];
#pragma unroll
        for (int i = 1; i < 8; ++i) s += ss[par][i];
        const float lse = mx + kLn2 * log2f(s);
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int c = threadIdx.x + i * 256;
            if (c < c4) {
                // optional log-prior of each class (16-byte aligned, C % 4 == 0): a hybrid decoder
                // wants log p(state | frame) - log p(state)
                const float4 pr = prior ? __ldg(reinterpret_cast<const float4*>(prior) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
                z[c] = make_float4(v[i].x - lse - pr.x, v[i].y - lse - pr.y, v[i].z - lse - pr.z, v[i].w - lse - pr.w);
            }
        }
    }
}

}  // namespace

int launch_real_gemm(const RealGemmArgs& a, cudaStream_t st) {
    dim3 grid(ceil_div(a.M, TM), ceil_div(a.N, TN));
    if (a.Ab && a.Bf)
        real_gemm_kernel<true, false><<<grid, THREADS, 0, st>>>(a);
    else if (a.Af && a.Bb)
        real_gemm_kernel<false, true><<<grid, THREADS, 0, st>>>(a);
    else if (a.Af && a.Bf)
        real_gemm_kernel<false, false><<<grid, THREADS, 0, st>>>(a);
    else
        return BNN_ERR_UNSUPPORTED;
    return launch_status();
}

int launch_log_softmax_rows(float* Z, int ldz, int M, int C, const float* prior, cudaStream_t st) {
    const int blocks = M < 148 * 8 ? M : 148 * 8;
    const bool reg = (C % 4 == 0) && (ldz % 4 == 0) && aligned16(Z) && C <= 256 * 4 * 4 && (!prior || aligned16(prior));
    if (reg && C <= 256 * 4 * 2)
        log_softmax_rows_reg_kernel<2><<<blocks, 256, 0, st>>>(Z, ldz, M, C, prior);
    else if (reg)
        log_softmax_rows_reg_kernel<4><<<blocks, 256, 0, st>>>(Z, ldz, M, C, prior);
    else
        log_softmax_rows_kernel<<<blocks, 256, 0, st>>>(Z, ldz, M, C, prior);
    return launch_status();
}

}  // namespace bnn
