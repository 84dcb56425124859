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
#include "tcgen05.cuh"

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

// One row held in registers by the 256 threads of a CTA (C <= 256*4*V, 16-byte aligned rows): every
// logit is read from memory once and written once.  The maximum is reduced first (warp shuffles, then
// 8 values through shared memory), so each element costs a subtract, a multiply, one ex2 and one add;
// the sum is reduced the same way.  sm/ss: 8 floats of shared scratch each; the caller alternates two
// sets from row to row, which saves a barrier per row.
template <int V>
__device__ __forceinline__ void log_softmax_row_reg(float4* __restrict__ z, int c4, const float* __restrict__ prior,
                                                    float* sm, float* ss) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
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
    if (lane == 0) sm[w] = mx;
    __syncthreads();
    mx = sm[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, sm[i]);
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
    if (lane == 0) ss[w] = s;
    __syncthreads();
    s = ss[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) s += ss[i];
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

// R rows at once by a CTA of NT threads (z0, z0 + ldz4, ...; rows at or beyond `rows` are left alone):
// the loads of all of them are in flight together and the reductions share their barriers.
// sm/ss: R x (NT / 32) floats each.
template <int V, int R, int NT>
__device__ __forceinline__ void log_softmax_rows_reg(float4* __restrict__ z0, size_t ldz4, int rows, int c4,
                                                     const float* __restrict__ prior, float (*sm)[NT / 32],
                                                     float (*ss)[NT / 32]) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
    float4 v[R][V];
    float mx[R], s[R];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int c = threadIdx.x + i * NT;
            v[r][i] = (c < c4 && r < rows) ? __ldcs(z0 + r * ldz4 + c) : make_float4(-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX);
        }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        mx[r] = -FLT_MAX;
#pragma unroll
        for (int i = 0; i < V; ++i)
            mx[r] = fmaxf(fmaxf(mx[r], fmaxf(v[r][i].x, v[r][i].y)), fmaxf(v[r][i].z, v[r][i].w));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], o));
        if (lane == 0) sm[r][w] = mx[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
        mx[r] = sm[r][0];
#pragma unroll
        for (int i = 1; i < NT / 32; ++i) mx[r] = fmaxf(mx[r], sm[r][i]);
        // sum of 2^((z - max) log2 e), as in log_softmax_row_reg; padding (-FLT_MAX) contributes 0
        s[r] = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i)
            s[r] += (ex2_approx((v[r][i].x - mx[r]) * kLog2e) + ex2_approx((v[r][i].y - mx[r]) * kLog2e)) +
                    (ex2_approx((v[r][i].z - mx[r]) * kLog2e) + ex2_approx((v[r][i].w - mx[r]) * kLog2e));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s[r] += __shfl_xor_sync(0xFFFFFFFFu, s[r], o);
        if (lane == 0) ss[r][w] = s[r];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float t = ss[r][0];
#pragma unroll
        for (int i = 1; i < NT / 32; ++i) t += ss[r][i];
        const float lse = mx[r] + kLn2 * log2f(t);
#pragma unroll
        for (int i = 0; i < V; ++i) {
            const int c = threadIdx.x + i * NT;
            if (c < c4 && r < rows) {
                const float4 pr = prior ? __ldg(reinterpret_cast<const float4*>(prior) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
                __stcs(z0 + r * ldz4 + c, make_float4(v[r][i].x - lse - pr.x, v[r][i].y - lse - pr.y, v[r][i].z - lse - pr.z, v[r][i].w - lse - pr.w));
            }
        }
    }
}

// Same result as log_softmax_rows_kernel, one CTA per row at a time.
template <int V>
__global__ void __launch_bounds__(256)
log_softmax_rows_reg_kernel(float* __restrict__ Z, int ldz, int M, int C, const float* __restrict__ prior) {
    __shared__ float sm[2][8], ss[2][8];
    const int c4 = C >> 2;  // C % 4 == 0
    int par = 0;
    // Rows are taken from the last one down: the kernel that wrote the logits just before this one
    // produced the last frames last, and those are the rows the L2 cache still holds.
    for (int r = blockIdx.x; r < M; r += gridDim.x, par ^= 1)
        log_softmax_row_reg<V>(reinterpret_cast<float4*>(Z + (size_t)(M - 1 - r) * ldz), c4, prior, sm[par], ss[par]);
}

// The same rows, taken while the kernel that writes the logits is still running.  That kernel counts, per
// group of `group_rows` consecutive frames, the arrivals of the warps that have stored their share of the
// group (release at GPU scope); a group is complete at `need` arrivals.  This kernel is launched behind it
// with programmatic stream serialisation: its first CTAs move onto the SMs as soon as every CTA of the
// producer is resident, share them with it (the producer is bound by the tensor pipe, this one by memory)
// and follow it group by group, reading the logits from the L2 cache that has just received them; the
// rest of the grid moves in when the producer's CTAs leave and helps with the last groups.  Rows are
// claimed kFollowRows at a time, in order, from one counter (done[groups], zero at launch), so a CTA that starts
// late goes straight to the rows that are left.  Every wait is bounded: after status.limit clocks the
// CTA sets the status word and returns.
// The CTA is small -- four warps, one per scheduler of an SM -- because that is what fits beside the 17 warps
// of 72 registers of the kernel it follows: the busiest scheduler's register file has room for one more
// warp of up to 152 registers.
constexpr int kFollowRows = 2, kFollowThreads = 128;
template <int V>
__global__ void __launch_bounds__(kFollowThreads)
log_softmax_rows_follow_kernel(float* __restrict__ Z, int ldz, int M, int C, const float* __restrict__ prior,
                               int* __restrict__ done, int need, int group_rows, tc::TcStatus status) {
    constexpr int R = kFollowRows, NT = kFollowThreads;
    __shared__ float sm[2][R][NT / 32], ss[2][R][NT / 32];
    __shared__ int claim;
    const int c4 = C >> 2;
    int* next_row = done + ceil_div(M, group_rows);
    int pending = 0, ready_group = -1;   // thread 0: the claim in flight; the last group seen complete
    int par = 0;
    if (threadIdx.x == 0) pending = atomicAdd(next_row, R);
    while (true) {
        if (threadIdx.x == 0) {
            int r = pending;
            const int gi = r / group_rows;           // group_rows is a multiple of R: the rows lie in one group
            if (r < M && gi > ready_group) {
                const long long t0 = clock64();
#pragma unroll 1
                while (true) {
                    int v;
                    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(done + gi) : "memory");
                    if (v >= need) { ready_group = gi; break; }
                    if (clock64() - t0 > status.limit) { r = -1; break; }
                    __nanosleep(200);
                }
            }
            claim = r;
        }
        __syncthreads();
        const int r = claim;
        if (r < 0 || r >= M) {
            if (threadIdx.x == 0 && r < 0) atomicExch(status.word, 1);
            break;
        }
        if (threadIdx.x == 0) pending = atomicAdd(next_row, R);   // in flight while these rows are worked on
        log_softmax_rows_reg<V, R, NT>(reinterpret_cast<float4*>(Z + (size_t)r * ldz), (size_t)(ldz >> 2), M - r, c4, prior,
                                   sm[par], ss[par]);
        par ^= 1;   // the scratch alternates; `claim` is rewritten only after the two barriers inside
    }
    // completion of this kernel implies completion of the one it followed
    if (threadIdx.x == 0) pdl_wait();
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

bool log_softmax_can_follow(const float* Z, int ldz, int C, const float* prior) {
    return (C % 4 == 0) && (ldz % 4 == 0) && aligned16(Z) && C <= 128 * 4 * 8 && (!prior || aligned16(prior));
}

int launch_log_softmax_rows_follow(float* Z, int ldz, int M, int C, const float* prior, int* done, int need,
                                   int group_rows, cudaStream_t st) {
    const int sms = device_sm_count();
    const tc::TcStatus status = tc_status();
    if (sms <= 0 || !status.word || !log_softmax_can_follow(Z, ldz, C, prior)) return BNN_ERR_CUDA;
    if (group_rows % kFollowRows != 0) return BNN_ERR_UNSUPPORTED;
    const int blocks = M < sms * 5 * kFollowRows ? ceil_div(M, kFollowRows) : sms * 5;
    const cudaError_t e = C <= kFollowThreads * 4 * 4
        ? launch_pdl(log_softmax_rows_follow_kernel<4>, dim3(blocks), dim3(kFollowThreads), 0, st, Z, ldz, M, C, prior, done, need, group_rows, status)
        : launch_pdl(log_softmax_rows_follow_kernel<8>, dim3(blocks), dim3(kFollowThreads), 0, st, Z, ldz, M, C, prior, done, need, group_rows, status);
    return e == cudaSuccess ? launch_status() : BNN_ERR_CUDA;
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
