// Binary weights x real-valued activations on the tensor cores (tcgen05 kind::f16, bf16
// operands, fp32 accumulators in TMEM):  y[m][n] = sum_k w[n][k] * x[m][k],  w in {-1,+1}.
//
// +-1 is exact in bf16.  The real operand is split on chip into bf16 terms
//     x = x_hi + x_lo (+ x_lo2),   |x - x_hi - x_lo| <= 2^-17 |x|   (3 terms: exact),
// and one MMA per term accumulates into the same fp32 accumulator, so the result differs from
// the exact sum by at most 2^-17 * sum_k |x[m][k]| plus fp32 accumulation rounding.
//
// The contraction index is permuted inside each group of 32 (identically for both operands):
// 32-bit word t of a K step holds logical k = t and k = t + 16, so one shift and one
// AND/OR turn a packed weight word into two bf16 values.
//
// CTA tile 128 frames x 256 units, 32 k per stage.  Warps 0-3 epilogue (affine, Sign+pack or
// hardtanh), warp 4 MMA issue, warps 5-12 producers.
#include <cuda_bf16.h>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 32;
constexpr int A_PLANE = BM * BK * 2;  // 8 KB: one bf16 term of the activation tile
constexpr int B_BYTES = BN * BK * 2;  // 16 KB
constexpr int MMA_WARP = 4, PROD_WARP0 = 5, PROD_WARPS = 8, EPI_WARPS = 4;
constexpr int THREADS = (PROD_WARP0 + PROD_WARPS) * 32;  // 416
constexpr uint32_t TMEM_COLS = 512;

template <int NT> struct Cfg {
    static constexpr int STAGE_BYTES = NT * A_PLANE + B_BYTES;
    static constexpr int STAGES = NT == 2 ? 6 : 5;
};

struct Control {
    float sc[BN], sh[BN];
    uint64_t full[8], empty[8], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    WaitState wait;
};


__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo_as_float(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi_as_float(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

struct Args {
    const float* X; int ldx;
    const uint32_t* Wp; int ldwp;
    int M, N, K;
    const float* scale; const float* shift;
    int act, sign_mode;
    float* Y; int ldy;
    uint32_t* out_bits; int ldob;
    TcStatus status;
};

template <int NT>
__global__ void __launch_bounds__(THREADS, 1) signw_tc_kernel(Args g) {
    using C = Cfg<NT>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    Control* ctl = reinterpret_cast<Control*>(smem + C::STAGES * C::STAGE_BYTES);
    volatile int* abort_flag = &ctl->wait.abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = g.M, N = g.N, K = g.K;
    const int kw = words_for(K);
    const int nks = ceil_div(K, BK);
    const int m_tiles = ceil_div(M, BM), n_tiles = ceil_div(N, BN);
    const int tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), PROD_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), EPI_WARPS);
        }
        wait_state_init(&ctl->wait, g.status);
        mbar_init_fence();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(smem_u32(&ctl->tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;

    if (warp >= PROD_WARP0) {
        // ---------------- producers: thread p converts half a K step of activation row p/2
        // (16 floats -> NT x 8 bf16x2 words) and widens packed weight row p (32 bits -> 16 words)
        const int p = threadIdx.x - PROD_WARP0 * 32;  // 0..255
        const int ra = p >> 1, h = p & 1;
        const bool vec = (g.ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.X) & 15) == 0);
        const int my_tiles = (tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
        const int total = my_tiles * nks;

        struct Raw { float x[16]; uint32_t w; };
        int pf_i = 0, pf_ks = 0, pf_tile = blockIdx.x;
        auto fetch = [&](Raw& o) {
#pragma unroll
            for (int j = 0; j < 16; ++j) o.x[j] = 0.f;
            o.w = 0u;
            if (pf_i >= total) return;
            const int m = (pf_tile % m_tiles) * BM + ra;
            const int n = (pf_tile / m_tiles) * BN + p;
            const int kb = pf_ks * BK;
            if (m < M) {
                const float* src = g.X + (size_t)m * g.ldx + kb + 8 * h;
#pragma unroll
                for (int part = 0; part < 2; ++part) {       // floats [8h, 8h+8) and [16+8h, 16+8h+8)
                    const int k0 = kb + 8 * h + 16 * part;
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int k = k0 + 4 * q;
                        float* d = &o.x[part * 8 + q * 4];
                        if (vec && k + 3 < K) {
                            const float4 v = __ldg(reinterpret_cast<const float4*>(src + 16 * part + 4 * q));
                            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (k + e < K) d[e] = __ldg(src + 16 * part + 4 * q + e);
                        }
                    }
                }
            }
            if (n < N && pf_ks < kw) o.w = __ldg(g.Wp + (size_t)n * g.ldwp + pf_ks);
            ++pf_i;
            if (++pf_ks == nks) { pf_ks = 0; pf_tile += gridDim.x; }
        };

        Raw cur, nxt;
        fetch(cur);
        for (int it = 0; it < total; ++it) {
            fetch(nxt);
            const int s = it % C::STAGES;
            const uint32_t ph = (uint32_t)((it / C::STAGES) & 1);
            // activation terms: word t pairs x[t] (low half) with x[t+8] (high half), t = 0..7
            uint32_t term[NT][8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                float a = cur.x[t], b = cur.x[8 + t];
#pragma unroll
                for (int q = 0; q < NT; ++q) {
                    const uint32_t w = pack_bf16x2(a, b);
                    term[q][t] = w;
                    if (q + 1 < NT) { a -= bf16_lo_as_float(w); b -= bf16_hi_as_float(w); }
                }
            }
            // weight bits -> +-1 in bf16: word t holds bit t (low half) and bit t+16 (high half)
            uint32_t wv[16];
            const uint32_t nw = ~cur.w;
#pragma unroll
            for (int t = 0; t < 16; ++t) wv[t] = ((nw << (15 - t)) & 0x80008000u) | 0x3F803F80u;

            if (!warp_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag, lane)) break;
            const uint32_t st = smem_u32(smem) + s * C::STAGE_BYTES;
#pragma unroll
            for (int q = 0; q < NT; ++q)
#pragma unroll
                for (int c = 0; c < 2; ++c)
                    sts128(st + q * A_PLANE + ((h * 2 + c) * BM + ra) * 16,
                           term[q][4 * c], term[q][4 * c + 1], term[q][4 * c + 2], term[q][4 * c + 3]);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                sts128(st + NT * A_PLANE + (c * BN + p) * 16, wv[4 * c], wv[4 * c + 1], wv[4 * c + 2], wv[4 * c + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
            cur = nxt;
        }
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kAccF32, kFmtBF16, kFmtBF16, BM, BN);
            int it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
                const int b = tl & 1;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), (uint32_t)(((tl >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d = tmem + (uint32_t)(b * BN);
                for (int ks = 0; ks < nks; ++ks, ++it) {
                    const int s = it % C::STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)((it / C::STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a0 = smem_u32(smem + s * C::STAGE_BYTES);
                    const uint32_t b0 = a0 + NT * A_PLANE;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {   // two K steps of 16 per stage
                        const uint64_t db = smem_desc_kmajor(b0 + 2 * j * (BN * 16), BN * 16, 128);
#pragma unroll
                        for (int q = 0; q < NT; ++q) {
                            const uint64_t da = smem_desc_kmajor(a0 + q * A_PLANE + 2 * j * (BM * 16), BM * 16, 128);
                            mma_f16(d, da, db, idesc, (ks | j | q) != 0);
                        }
                    }
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) mma_commit(smem_u32(&ctl->acc_full[b]));
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: thread = one frame
        const int row_in_tile = warp * 32 + lane;
        const bool pack = g.act == BNN_ACT_SIGN_PACK;
        const bool vy = g.Y && (g.ldy % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.Y) & 15) == 0);
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
            const int m = m0 + row_in_tile;
            epi_bar_sync();
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int nl = row_in_tile + hh * 128, n = n0 + nl;
                ctl->sc[nl] = (g.scale && n < N) ? g.scale[n] : 1.0f;
                ctl->sh[nl] = (g.shift && n < N) ? g.shift[n] : 0.0f;
            }
            epi_bar_sync();
            const int b = tl & 1;
            ok = epi_all(warp_wait(smem_u32(&ctl->acc_full[b]), (uint32_t)((tl >> 1) & 1), abort_flag, lane));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * BN);
            uint32_t words[BN / 32];
#pragma unroll
            for (int gi = 0; gi < BN / 32; ++gi) {
                uint32_t acc[32];
                tmem_ld32(taddr + gi * 32, acc);
                tmem_ld_wait();
                const int nb = n0 + gi * 32;
                float y[32];
                uint32_t wd = 0u;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float v = fmaf(ctl->sc[gi * 32 + j], __uint_as_float(acc[j]), ctl->sh[gi * 32 + j]);
                    if (g.act == BNN_ACT_HARDTANH) v = fminf(fmaxf(v, -1.0f), 1.0f);
                    if (g.act == BNN_ACT_SIGMOID) v = 1.0f / (1.0f + expf(-v));
                    y[j] = v;
                    wd |= (uint32_t)(nb + j < N && sign_is_pos(v, g.sign_mode)) << j;
                }
                words[gi] = wd;
                if (g.Y && m < M) {
                    float* dst = g.Y + (size_t)m * g.ldy + nb;
                    if (vy && nb + 31 < N) {
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            reinterpret_cast<float4*>(dst)[q] = make_float4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < N) dst[j] = y[j];
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
            if (pack && m < M) {
                const int nw = words_for(N), w0 = n0 >> 5;
                uint32_t* dst = g.out_bits + (size_t)m * g.ldob + w0;
                if (w0 + BN / 32 <= nw) {
                    reinterpret_cast<uint4*>(dst)[0] = make_uint4(words[0], words[1], words[2], words[3]);
                    reinterpret_cast<uint4*>(dst)[1] = make_uint4(words[4], words[5], words[6], words[7]);
                } else {
#pragma unroll
                    for (int gi = 0; gi < BN / 32; ++gi)
                        if (w0 + gi < nw) dst[gi] = words[gi];
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
    if (threadIdx.x == 0 && ctl->wait.abort) atomicExch(g.status.word, 1);
}

template <int NT>
int launch_nt(const Args& a, cudaStream_t st) {
    using C = Cfg<NT>;
    constexpr int SMEM = C::STAGES * C::STAGE_BYTES + (int)sizeof(Control) + 128;
    const int sms = device_sm_count();
    if (sms <= 0 || !ensure_dynamic_smem(reinterpret_cast<const void*>(signw_tc_kernel<NT>), SMEM)) return BNN_ERR_CUDA;
    const int tiles = ceil_div(a.M, BM) * ceil_div(a.N, BN);
    signw_tc_kernel<NT><<<tiles < sms ? tiles : sms, THREADS, SMEM, st>>>(a);
    return launch_status();
}

}  // namespace

int launch_signw_tc(const RealGemmArgs& r, int terms, cudaStream_t st) {
    Args a{r.Af, r.lda, r.Bb, r.ldb, r.M, r.N, r.K, r.scale, r.shift, r.act, r.sign_mode,
           r.Y, r.ldy, r.out_bits, r.ldob, tc_status()};
    if (!a.status.word) return BNN_ERR_CUDA;
    return terms == 3 ? launch_nt<3>(a, st) : launch_nt<2>(a, st);
}

}  // namespace bnn
