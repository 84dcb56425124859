// XNOR-popcount GEMM on the integer pipes: d[m][n] = K - 2*popc(a[m] xor w[n]); with the frame
// bits standing for (0,1) instead of (-1,+1): d[m][n] = 2*popc(a[m] and w[n]) - popc(a[m]).
//
// CTA tile 128 (frames) x 128 (units), 256 threads.  Warp y owns 16 frames; lane x owns the
// four units x, x+32, x+64, x+96, so that one ballot over the warp yields a whole packed
// word of the next layer's input.  Packed rows are staged through shared memory with 16-byte
// cp.async copies, double buffered, 16 words (512 bits) of K per stage.
#include "bnn_common.cuh"

namespace bnn {

namespace {

constexpr int BM = 128, BN = 128, KT = 16;  // KT words of K per stage
constexpr int THREADS = 256;

struct __align__(16) Stage {
    uint32_t a[BM][KT];         // a[m][k]: a warp reads one address (broadcast)
    uint32_t w[KT / 4][BN][4];  // w[k/4][n][k%4]: lanes read consecutive 16-byte chunks
};

// Copy one K-stage of both tiles.  Rows beyond M/N and 16-byte chunks that start at or
// beyond word kw are zero-filled, so they add nothing to the popcount of the XOR.
__device__ __forceinline__ void load_stage(Stage& s, const uint32_t* __restrict__ Ap, int ldap,
                                           const uint32_t* __restrict__ Wp, int ldwp,
                                           int m0, int n0, int M, int N, int kw, int kbase) {
    // 128 rows x 4 chunks per operand = 512 chunks each; 256 threads -> 2 + 2 per thread
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int c = threadIdx.x + it * THREADS;  // 0..511
        const int row = c >> 2, q = c & 3;
        const int k = kbase + q * 4;
        const bool kin = k < kw;
        {
            const int gm = m0 + row;
            const bool ok = kin && gm < M;
            const uint32_t* src = ok ? Ap + (size_t)gm * ldap + k : Ap;
            cp_async16(&s.a[row][q * 4], src, ok);
        }
        {
            const int gn = n0 + row;
            const bool ok = kin && gn < N;
            const uint32_t* src = ok ? Wp + (size_t)gn * ldwp + k : Wp;
            cp_async16(&s.w[q][row][0], src, ok);
        }
    }
}

// After the copies of the stage holding word kw-1 have landed: clear, in the chunk that
// this thread itself copied, the bits at positions >= K (pad bits of the last word and
// pitch words after it), so the result does not depend on what the caller left there.
__device__ __forceinline__ void mask_tail(Stage& s, int kw, int kbase, uint32_t tmask) {
    const int last = kw - 1 - kbase;  // index of the last valid word inside this stage
    if (last < 0 || last >= KT) return;
    const int lq = last >> 2, lw = last & 3;
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int c = threadIdx.x + it * THREADS;
        const int row = c >> 2, q = c & 3;
        if (q != lq) continue;
        s.a[row][q * 4 + lw] &= tmask;
        s.w[q][row][lw] &= tmask;
        for (int j = lw + 1; j < 4; ++j) {
            s.a[row][q * 4 + j] = 0u;
            s.w[q][row][j] = 0u;
        }
    }
}

template <bool STORE_C, bool SIGN_PACK, bool ZO>
__global__ void __launch_bounds__(THREADS, 2)
xnor_popc_kernel(const uint32_t* __restrict__ Ap, int ldap, const uint32_t* __restrict__ Wp,
                 int ldwp, int M, int N, int K, int32_t* __restrict__ C, int ldc,
                 const int32_t* __restrict__ thr, const uint32_t* __restrict__ flip,
                 uint32_t* __restrict__ out_bits, int ldob) {
    __shared__ Stage st[2];
    const int lane = threadIdx.x & 31, wy = threadIdx.x >> 5;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int kw = words_for(K);
    const uint32_t tmask = tail_mask(K);
    const int nstages = ceil_div(kw, KT);

    int acc[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0;
    int ones[16];   // (0,1) frames: number of ones in the row
#pragma unroll
    for (int i = 0; i < 16; ++i) ones[i] = 0;

    load_stage(st[0], Ap, ldap, Wp, ldwp, m0, n0, M, N, kw, 0);
    cp_async_commit();
    for (int s = 0; s < nstages; ++s) {
        if (s + 1 < nstages)
            load_stage(st[(s + 1) & 1], Ap, ldap, Wp, ldwp, m0, n0, M, N, kw, (s + 1) * KT);
        cp_async_commit();
        cp_async_wait<1>();
        Stage& cur = st[s & 1];
        mask_tail(cur, kw, s * KT, tmask);
        __syncthreads();
#pragma unroll
        for (int q = 0; q < KT / 4; ++q) {
            uint4 w4[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                w4[j] = *reinterpret_cast<const uint4*>(&cur.w[q][lane + 32 * j][0]);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const uint4 a4 = *reinterpret_cast<const uint4*>(&cur.a[wy * 16 + i][q * 4]);
                if (ZO) ones[i] += __popc(a4.x) + __popc(a4.y) + __popc(a4.z) + __popc(a4.w);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (ZO)
                        acc[i][j] += __popc(a4.x & w4[j].x) + __popc(a4.y & w4[j].y) +
                                     __popc(a4.z & w4[j].z) + __popc(a4.w & w4[j].w);
                    else
                        acc[i][j] += __popc(a4.x ^ w4[j].x) + __popc(a4.y ^ w4[j].y) +
                                     __popc(a4.z ^ w4[j].z) + __popc(a4.w ^ w4[j].w);
                }
            }
        }
        __syncthreads();
    }

    // ---- epilogue ----
    int tj[4];
    bool fj[4];
    if (SIGN_PACK) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + lane + 32 * j;
            tj[j] = n < N ? thr[n] : 0x7FFFFFFF;
            fj[j] = n < N ? ((flip[n >> 5] >> (n & 31)) & 1u) : false;
        }
    }
    uint32_t keep[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int m = m0 + wy * 16 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + lane + 32 * j;
            const int d = ZO ? 2 * acc[i][j] - ones[i] : K - 2 * acc[i][j];
            if (STORE_C) {
                if (m < M && n < N) C[(size_t)m * ldc + n] = d;
            }
            if (SIGN_PACK) {
                const bool bit = (n < N) && ((d >= tj[j]) != fj[j]);
                const uint32_t word = __ballot_sync(0xFFFFFFFFu, bit);
                if (lane == i) keep[j] = word;
            }
        }
    }
    if (SIGN_PACK && lane < 16) {
        const int m = m0 + wy * 16 + lane;
        if (m < M) {
            const int nw = words_for(N);
            const int w0 = n0 >> 5;
            uint32_t* dst = out_bits + (size_t)m * ldob + w0;
            if (w0 + 3 < nw) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(keep[0], keep[1], keep[2], keep[3]);
            } else {
                for (int j = 0; j < 4; ++j)
                    if (w0 + j < nw) dst[j] = keep[j];
            }
        }
    }
}

}  // namespace

template <bool ZO>
static void launch_zo(dim3 grid, const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                      int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                      uint32_t* out_bits, int ldob, cudaStream_t st) {
    const bool sp = out_bits != nullptr;
    if (C && sp)
        xnor_popc_kernel<true, true, ZO><<<grid, THREADS, 0, st>>>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob);
    else if (C)
        xnor_popc_kernel<true, false, ZO><<<grid, THREADS, 0, st>>>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob);
    else
        xnor_popc_kernel<false, true, ZO><<<grid, THREADS, 0, st>>>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob);
}

int launch_xnor_popc(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                     int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                     uint32_t* out_bits, int ldob, int zo, cudaStream_t st) {
    dim3 grid(ceil_div(M, BM), ceil_div(N, BN));
    if (zo) launch_zo<true>(grid, Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, st);
    else launch_zo<false>(grid, Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, st);
    return launch_status();
}

}  // namespace bnn
