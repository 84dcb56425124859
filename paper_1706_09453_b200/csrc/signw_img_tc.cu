// Binary weights x real-valued activations on the tensor cores, with the activations split
// ONCE per call into bf16 terms (instead of once per tile of units):
//
//   1. x_split_kernel writes x = x_hi + x_lo (+ x_lo2) as bf16 planes into a scratch "image"
//      that is stored in exactly the order the MMA reads shared memory (a memory-bound pass:
//      every fp32 input is read once);
//   2. signw_img_kernel runs the GEMM: a pipeline stage of activations is ONE bulk asynchronous
//      copy of the image (no tensor map, no multicast), the packed +-1 weights are widened to
//      bf16 on chip, one MMA per term accumulates in fp32 in tensor memory.
//
// Frames are on the M side (TMEM lane = frame), units on the N side.  A CTA tile is 128 frames
// x 512 units (two 256-column accumulators fed by the same activation stage).  The epilogue
// thread owns a frame: per-unit affine (one fma), then Sign + pack (16 words per row and
// tile) and/or fp32 stores of 128 contiguous bytes.  When the layer that consumes the outputs is
// again of this kind (a network with binary weights and real activations, Algorithm 1), the
// epilogue can also write them as that layer's image (step 1 above), which saves the split pass
// and one round trip of the fp32 activations.
//
// |result - exact| <= 2^-17 * sum_k |x[m][k]| with 2 terms (products exact with 3), plus fp32
// accumulation rounding.  The contraction index is permuted inside each group of 32 exactly
// as in the other sign-weight kernel: word t of a K step holds k = t and k = t + 16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BM = 128;           // frames per tile
constexpr int UN = 512;           // units per tile (2 x 256)
constexpr int BK = 32;            // k per stage
constexpr int A_PLANE = BM * BK * 2;        // 8 KB per bf16 term
constexpr int B_BYTES = UN * BK * 2;        // 32 KB
constexpr int MMA_WARP = 4, PROD_WARP0 = 5, PROD_WARPS = 8, EPI_WARPS = 4;
constexpr int THREADS = (PROD_WARP0 + PROD_WARPS) * 32;
constexpr uint32_t TMEM_COLS = 512;

template <int NT> struct Cfg {
    static constexpr int A_BYTES = NT * A_PLANE;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = NT == 2 ? 4 : 3;
};

struct Control {
    float sc[UN], sh[UN];
    uint64_t full[4], empty[4], acc_full, acc_empty[2];
    uint32_t tmem_base;
    WaitState wait;
};

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo_as_float(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi_as_float(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ---- split: one CTA per (frame tile, stage): 128 rows x 32 floats -> NT planes of 8 KB ------
template <int NT>
__global__ void __launch_bounds__(256)
x_split_kernel(const float* __restrict__ X, int ldx, int M, int K, int nks, uint8_t* __restrict__ img,
               int sdim, int sleft, int* __restrict__ clear, int clear_words) {
    __shared__ float raw[BM][BK + 1];
    pdl_trigger();   // the GEMM may be scheduled as SMs free up; it waits before it reads the image
    // As the first kernel of a forward pass this one also clears the pass's counters (a few hundred
    // words): a memset node of its own in front of it costs about 4 us per step.
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < clear_words; i += gridDim.x * blockDim.x) clear[i] = 0;
    const int mt = blockIdx.x / nks, ks = blockIdx.x % nks;
    const int t = threadIdx.x;
    // coalesced read: 8 consecutive threads fetch the 32 floats of one row segment.  With splicing
    // (sdim > 0, a multiple of 4 on the vector path) position k of row m is feature k % sdim of
    // input row m - sleft + k / sdim, clamped to the rows that exist: the context window of the
    // feature front end, formed here instead of being materialised in memory.
    const bool vec = (ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15) == 0) && (sdim % 4 == 0);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = (t >> 3) + 32 * i, m = mt * BM + row;
        const int c4 = (t & 7) * 4, k = ks * BK + c4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m < M) {
            const float* src = X + (size_t)m * ldx + k;
            if (sdim > 0) {
                int r = m - sleft + k / sdim;
                r = r < 0 ? 0 : (r >= M ? M - 1 : r);
                src = X + (size_t)r * ldx + k % sdim;
            }
            if (vec && k + 3 < K) {
                v = __ldg(reinterpret_cast<const float4*>(src));
            } else {
                if (sdim > 0) {   // the four positions may straddle two input rows
                    float e[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (k + q < K) {
                            int r = m - sleft + (k + q) / sdim;
                            r = r < 0 ? 0 : (r >= M ? M - 1 : r);
                            e[q] = __ldg(X + (size_t)r * ldx + (k + q) % sdim);
                        }
                    v = make_float4(e[0], e[1], e[2], e[3]);
                } else {
                    if (k + 0 < K) v.x = __ldg(src + 0);
                    if (k + 1 < K) v.y = __ldg(src + 1);
                    if (k + 2 < K) v.z = __ldg(src + 2);
                    if (k + 3 < K) v.w = __ldg(src + 3);
                }
            }
        }
        raw[row][c4 + 0] = v.x; raw[row][c4 + 1] = v.y; raw[row][c4 + 2] = v.z; raw[row][c4 + 3] = v.w;
    }
    __syncthreads();
    // coalesced write: consecutive threads write consecutive 16-byte chunks (consecutive rows)
    uint8_t* blk = img + ((size_t)mt * nks + ks) * (NT * A_PLANE);
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int chunk = t + 256 * i;          // 0..511 = (K step j, half-step cc, row)
        const int row = chunk & (BM - 1), jc = chunk >> 7;   // jc = 2j + cc
        uint32_t w[NT][4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {           // word e pairs k = 4jc + e with k + 16
            float a = raw[row][4 * jc + e], b = raw[row][4 * jc + e + 16];
#pragma unroll
            for (int q = 0; q < NT; ++q) {
                const uint32_t p = pack_bf16x2(a, b);
                w[q][e] = p;
                if (q + 1 < NT) { a -= bf16_lo_as_float(p); b -= bf16_hi_as_float(p); }
            }
        }
#pragma unroll
        for (int q = 0; q < NT; ++q)
            *reinterpret_cast<uint4*>(blk + q * A_PLANE + (size_t)chunk * 16) = make_uint4(w[q][0], w[q][1], w[q][2], w[q][3]);
    }
}


// TMEM -> registers: lane i of the warp reads 16 columns of TMEM lane (base lane + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

// Sign of 16 affine outputs: bit j = (Sign(fma(sc[j], acc[j], sh[j])) is +1).
// sc / sh: 16-byte aligned shared memory.
template <bool ZERO_NEG>
__device__ __forceinline__ uint32_t sign_bits16(const uint32_t (&acc)[16], const float* sc, const float* sh) {
    const float4* s4 = reinterpret_cast<const float4*>(sc);
    const float4* h4 = reinterpret_cast<const float4*>(sh);
    uint32_t wd = 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 s = s4[q], h = h4[q];
        const float v0 = fmaf(s.x, __uint_as_float(acc[4 * q + 0]), h.x);
        const float v1 = fmaf(s.y, __uint_as_float(acc[4 * q + 1]), h.y);
        const float v2 = fmaf(s.z, __uint_as_float(acc[4 * q + 2]), h.z);
        const float v3 = fmaf(s.w, __uint_as_float(acc[4 * q + 3]), h.w);
        wd |= (uint32_t)(ZERO_NEG ? v0 > 0.0f : v0 >= 0.0f) << (4 * q + 0);
        wd |= (uint32_t)(ZERO_NEG ? v1 > 0.0f : v1 >= 0.0f) << (4 * q + 1);
        wd |= (uint32_t)(ZERO_NEG ? v2 > 0.0f : v2 >= 0.0f) << (4 * q + 2);
        wd |= (uint32_t)(ZERO_NEG ? v3 > 0.0f : v3 >= 0.0f) << (4 * q + 3);
    }
    return wd;
}

template <int ACT>
__device__ __forceinline__ float activate(float v) {
    if (ACT == BNN_ACT_HARDTANH) return fminf(fmaxf(v, -1.0f), 1.0f);
    if (ACT == BNN_ACT_SIGMOID) return 1.0f / (1.0f + expf(-v));
    return v;
}

// Epilogue of one 256-column accumulator for a layer that hands on nothing but bits.
template <bool ZERO_NEG>
__device__ __forceinline__ void epilogue_bits(uint32_t taddr, const float* sc, const float* sh, int cols_left,
                                              uint32_t* dst, int words_left, bool row_ok) {
    // (loads of columns beyond the layer's last unit stay inside the accumulator; their bits are
    // masked to zero and never stored)
    uint32_t a0[16], a1[16];
    tmem_ld16(taddr, a0);
#pragma unroll 1
    for (int q4 = 0; q4 < 2; ++q4) {              // 128 columns = four words = one 16-byte store
        if (q4 * 128 >= cols_left) break;         // uniform over the CTA
        uint32_t words[4];
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
            const int c = q4 * 128 + gq * 32;
            tmem_ld_wait();
            tmem_ld16(taddr + c + 16, a1);
            uint32_t wd = sign_bits16<ZERO_NEG>(a0, sc + c, sh + c);
            tmem_ld_wait();
            if (c + 32 < 256) tmem_ld16(taddr + c + 32, a0);
            wd |= sign_bits16<ZERO_NEG>(a1, sc + c + 16, sh + c + 16) << 16;
            const int valid = cols_left - c;
            words[gq] = valid >= 32 ? wd : (valid > 0 ? (wd & ((1u << valid) - 1u)) : 0u);
        }
        if (row_ok) {
            if (q4 * 4 + 4 <= words_left) {
                *reinterpret_cast<uint4*>(dst + q4 * 4) = make_uint4(words[0], words[1], words[2], words[3]);
            } else {
#pragma unroll
                for (int gq = 0; gq < 4; ++gq)
                    if (q4 * 4 + gq < words_left) dst[q4 * 4 + gq] = words[gq];
            }
        }
    }
    tmem_ld_wait();
}

// Epilogue of one 256-column accumulator with real-valued outputs: fp32 rows in `y`, packed bits as
// well when the activation is Sign, and / or the outputs as the split-activation image of the layer
// that consumes them (`img`: the block of this frame tile and of the first K stage these columns
// belong to; 32 columns are one stage of the consumer, stored exactly as x_split_kernel stores them).
// Where an epilogue thread writes its row of a consumer's image: address of its 16 bytes in chunk 0 of
// term 0 of the first stage, and the distances between stages, terms and chunks.
struct ImageOut {
    uint8_t* base;
    uint32_t stage_stride, plane_stride, chunk_stride;
    bool fp16;
};

template <int ACT, int NT>
__device__ __forceinline__ void epilogue_real(uint32_t taddr, const float* sc, const float* sh, int cols_left,
                                              float* y, bool vec, uint32_t* bits, int words_left, bool row_ok,
                                              int sign_mode, const ImageOut& img) {
    uint32_t a0[16], a1[16];
    tmem_ld16(taddr, a0);
    auto emit = [&](uint32_t (&a)[16], int c) -> uint32_t {   // columns c .. c+15 of the accumulator
        uint32_t wd = 0u;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float v = activate<ACT>(fmaf(sc[c + j], __uint_as_float(a[j]), sh[c + j]));
            a[j] = __float_as_uint(v);
            if (ACT == BNN_ACT_SIGN_PACK) wd |= (uint32_t)sign_is_pos(v, sign_mode) << j;
        }
        if (y && row_ok && c < cols_left) {
            if (vec && c + 16 <= cols_left) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    reinterpret_cast<float4*>(y + c)[q] = make_float4(__uint_as_float(a[4 * q]), __uint_as_float(a[4 * q + 1]),
                                                                      __uint_as_float(a[4 * q + 2]), __uint_as_float(a[4 * q + 3]));
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (c + j < cols_left) y[c + j] = __uint_as_float(a[j]);
            }
        }
        return wd;
    };
#pragma unroll 1
    for (int gi = 0; gi < 8; ++gi) {              // one packed word / one K stage of the consumer per iteration
        const int c = gi * 32;
        if (c >= cols_left) break;                // uniform over the CTA
        tmem_ld_wait();
        tmem_ld16(taddr + c + 16, a1);
        uint32_t wd = emit(a0, c);
        tmem_ld_wait();
        wd |= emit(a1, c + 16) << 16;
        if (ACT == BNN_ACT_SIGN_PACK && bits && row_ok && gi < words_left) {
            const int valid = cols_left - c;
            bits[gi] = valid >= 32 ? wd : (wd & ((1u << valid) - 1u));
        }
        if (img.base) {
            // word e of 16-byte chunk jc pairs column 4 jc + e (low half) with column 4 jc + e + 16;
            // columns beyond the layer's last unit and rows beyond the batch are stored as zeros
            uint8_t* blk = img.base + (size_t)gi * img.stage_stride;
#pragma unroll
            for (int jc = 0; jc < 4; ++jc) {
                uint32_t w[3][4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = 4 * jc + e;
                    float lo = (row_ok && c + i < cols_left) ? __uint_as_float(a0[i]) : 0.f;
                    float hi = (row_ok && c + 16 + i < cols_left) ? __uint_as_float(a1[i]) : 0.f;
                    if (img.fp16) {     // two fp16 terms
                        const __half l1 = __float2half_rn(lo), h1 = __float2half_rn(hi);
                        const __half l2 = __float2half_rn(lo - __half2float(l1)), h2 = __float2half_rn(hi - __half2float(h1));
                        w[0][e] = (uint32_t)__half_as_ushort(l1) | ((uint32_t)__half_as_ushort(h1) << 16);
                        w[1][e] = (uint32_t)__half_as_ushort(l2) | ((uint32_t)__half_as_ushort(h2) << 16);
                    } else {            // NT bf16 terms
#pragma unroll
                        for (int q = 0; q < NT; ++q) {
                            const uint32_t pk = pack_bf16x2(lo, hi);
                            w[q][e] = pk;
                            if (q + 1 < NT) { lo -= bf16_lo_as_float(pk); hi -= bf16_hi_as_float(pk); }
                        }
                    }
                }
                const int planes = img.fp16 ? 2 : NT;
#pragma unroll
                for (int q = 0; q < 3; ++q)
                    if (q < planes)
                        *reinterpret_cast<uint4*>(blk + q * img.plane_stride + jc * img.chunk_stride) = make_uint4(w[q][0], w[q][1], w[q][2], w[q][3]);
            }
        }
        if (c + 32 < 256) tmem_ld16(taddr + c + 32, a0);
    }
    tmem_ld_wait();
}

struct Args {
    uint8_t* img_out;        // split-activation image of the layer that consumes this one's outputs, or nullptr
    int nks_out;             //   its K stages per block of frames
    int img_out_kind;        //   0: bf16 terms, blocks of 128 frames (this kernel's own input format);
                             //   1: two fp16 terms, blocks of 256 frames (the real-valued layer on fp32 activations)
    const uint8_t* img;
    const uint32_t* Wp; int ldwp;
    int M, N, K;
    const float* scale; const float* shift;
    int act, sign_mode;
    float* Y; int ldy;
    uint32_t* out_bits; int ldob;
    TcStatus status;
};

template <int NT>
__global__ void __launch_bounds__(THREADS, 1) signw_img_kernel(Args g) {
    using C = Cfg<NT>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    Control* ctl = reinterpret_cast<Control*>(smem + C::STAGES * C::STAGE_BYTES);
    volatile int* abort_flag = &ctl->wait.abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = g.M, N = g.N;
    const int nks = ceil_div(g.K, BK);
    const int m_tiles = ceil_div(M, BM), n_tiles = ceil_div(N, UN);
    const int tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), PROD_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->acc_full), 1);
        mbar_init(smem_u32(&ctl->acc_empty[0]), EPI_WARPS);
        mbar_init(smem_u32(&ctl->acc_empty[1]), EPI_WARPS);
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
        // ---------------- producers: thread p widens packed weight rows p and p+256 of the unit
        // tile; the first producer thread also starts the bulk copy of the activation stage.
        const int p = threadIdx.x - PROD_WARP0 * 32;  // 0..255
        const int my_tiles = (tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
        const int total = my_tiles * nks;
        // Packed rows are read 16 bytes (4 stages) at a time, one group ahead of use.  Bits at
        // positions >= K may hold anything: the activation image is zero there.
        const int ngroups = ceil_div(nks, 4);
        int pf_g = 0, pf_tile = blockIdx.x, pf_left = my_tiles;
        auto fetch = [&](uint4 (&o)[2]) {
            o[0] = make_uint4(0u, 0u, 0u, 0u);
            o[1] = o[0];
            if (pf_left == 0) return;
            const int n0 = (pf_tile / m_tiles) * UN;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int n = n0 + p + 256 * q;
                if (n < N) o[q] = ldg_nc_u4(reinterpret_cast<const uint4*>(g.Wp + (size_t)n * g.ldwp) + pf_g);
            }
            if (++pf_g == ngroups) { pf_g = 0; pf_tile += gridDim.x; --pf_left; }
        };
        uint4 grp[2], nxt[2];
        fetch(grp);
        fetch(nxt);
        int ks = 0, tile = blockIdx.x, s = 0;
        uint32_t ph = 1;  // parity to wait for on `empty`: a fresh barrier passes parity 1
        for (int it = 0; it < total; ++it) {
            const int sub = ks & 3;
            uint32_t cur[2];
#pragma unroll
            for (int q = 0; q < 2; ++q)
                cur[q] = sub == 0 ? grp[q].x : sub == 1 ? grp[q].y : sub == 2 ? grp[q].z : grp[q].w;
            if (!warp_wait(smem_u32(&ctl->empty[s]), ph, abort_flag, lane)) break;
            const uint32_t st = smem_u32(smem) + s * C::STAGE_BYTES;
            if (p == 0) {
                // the image is the output of the kernel before this one in the stream: wait until that
                // kernel has completed and its writes are visible (the weights do not depend on it)
                if (it == 0) pdl_wait();
                const int mt = tile % m_tiles;
                mbar_expect_tx(smem_u32(&ctl->full[s]), C::A_BYTES);
                bulk_g2s(st, g.img + ((size_t)mt * nks + ks) * C::A_BYTES, C::A_BYTES, smem_u32(&ctl->full[s]));
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint32_t nw = ~cur[q];
                uint32_t wv[16];
#pragma unroll
                for (int t = 0; t < 16; ++t) wv[t] = ((nw << (15 - t)) & 0x80008000u) | 0x3F803F80u;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    sts128(st + C::A_BYTES + (c * UN + p + 256 * q) * 16, wv[4 * c], wv[4 * c + 1], wv[4 * c + 2], wv[4 * c + 3]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
            if (++s == C::STAGES) { s = 0; ph ^= 1u; }
            ++ks;
            if ((ks & 3) == 0 || ks == nks) {   // group used up: take the prefetched one
                grp[0] = nxt[0]; grp[1] = nxt[1];
                fetch(nxt);
            }
            if (ks == nks) { ks = 0; tile += gridDim.x; }
        }
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kAccF32, kFmtBF16, kFmtBF16, BM, 256);
            // MMAs of one stage into accumulator `sub` (units [256 sub, 256 sub + 256) of the tile)
            auto issue = [&](int s, int sub, int ks) {
                const uint32_t a0 = smem_u32(smem + s * C::STAGE_BYTES);
                const uint32_t b0 = a0 + C::A_BYTES;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint64_t db = smem_desc_kmajor(b0 + 2 * j * (UN * 16) + sub * 256 * 16, UN * 16, 128);
#pragma unroll
                    for (int q = 0; q < NT; ++q) {
                        const uint64_t da = smem_desc_kmajor(a0 + q * A_PLANE + 2 * j * (BM * 16), BM * 16, 128);
                        mma_f16(tmem + sub * 256, da, db, idesc, (ks | j | q) != 0);
                    }
                }
            };
            int it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
                const uint32_t par = (uint32_t)((tl & 1) ^ 1);
                // The epilogue hands accumulator 0 back first.  The first stages go into it alone
                // (their slots stay occupied) until accumulator 1 is free as well; then accumulator 1
                // catches up and the stages are released.
                ok = mbar_wait(smem_u32(&ctl->acc_empty[0]), par, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const int lead = nks < C::STAGES ? nks : C::STAGES;
                for (int ks = 0; ks < lead && ok; ++ks) {
                    const int s = (it + ks) % C::STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)(((it + ks) / C::STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue(s, 0, ks);
                }
                if (!ok) break;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[1]), par, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                for (int ks = 0; ks < lead; ++ks) {
                    const int s = (it + ks) % C::STAGES;
                    issue(s, 1, ks);
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                it += lead;
                for (int ks = lead; ks < nks; ++ks, ++it) {
                    const int s = it % C::STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)((it / C::STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue(s, 0, ks);
                    issue(s, 1, ks);
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) mma_commit(smem_u32(&ctl->acc_full));
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: thread = one frame (TMEM lane), columns = units
        const int row_in_tile = warp * 32 + lane;
        const bool pack = g.act == BNN_ACT_SIGN_PACK;
        const bool vy = g.Y && (g.ldy % 4 == 0) && ((reinterpret_cast<uintptr_t>(g.Y) & 15) == 0);
        const int nw = words_for(N);
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * UN;
            const int m = m0 + row_in_tile;
            epi_bar_sync();   // previous tile's readers of sc/sh are done
#pragma unroll
            for (int hh = 0; hh < UN / 128; ++hh) {
                const int nl = row_in_tile + hh * 128, n = n0 + nl;
                ctl->sc[nl] = (g.scale && n < N) ? g.scale[n] : 1.0f;
                ctl->sh[nl] = (g.shift && n < N) ? g.shift[n] : 0.0f;
            }
            epi_bar_sync();
            ok = epi_all(warp_wait(smem_u32(&ctl->acc_full), (uint32_t)(tl & 1), abort_flag, lane));
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll 1
            for (int sub = 0; sub < 2; ++sub) {
                const int c0 = sub * 256, left = N - (n0 + c0);        // columns of this accumulator that exist
                if (left > 0) {                                        // uniform over the CTA
                    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0;
                    const int w0 = (n0 + c0) >> 5;
                    uint32_t* bits = g.out_bits ? g.out_bits + (size_t)(m < M ? m : 0) * g.ldob + w0 : nullptr;
                    float* y = g.Y ? g.Y + (size_t)(m < M ? m : 0) * g.ldy + n0 + c0 : nullptr;
                    const float* sc = &ctl->sc[c0];
                    const float* sh = &ctl->sh[c0];
                    ImageOut io{nullptr, 0u, 0u, 0u, false};
                    if (g.img_out) {
                        const int ks0 = (n0 + c0) >> 5;   // first K stage of the consumer these columns belong to
                        if (g.img_out_kind == 1) {
                            const int mrow = m0 + row_in_tile;   // blocks of 256 frames, 32 KB per stage: [term][chunk][row][16 B]
                            io = ImageOut{g.img_out + ((size_t)(mrow >> 8) * g.nks_out + ks0) * 32768u + (size_t)(mrow & 255) * 16,
                                          32768u, 16384u, 4096u, true};
                        } else {
                            io = ImageOut{g.img_out + ((size_t)(m0 / BM) * g.nks_out + ks0) * (NT * A_PLANE) + (size_t)row_in_tile * 16,
                                          (uint32_t)(NT * A_PLANE), (uint32_t)A_PLANE, (uint32_t)(BM * 16), false};
                        }
                    }
                    if (pack && !g.Y) {
                        if (g.sign_mode == kSignZeroNeg) epilogue_bits<true>(taddr, sc, sh, left, bits, nw - w0, m < M);
                        else epilogue_bits<false>(taddr, sc, sh, left, bits, nw - w0, m < M);
                    } else if (pack) {
                        epilogue_real<BNN_ACT_SIGN_PACK, NT>(taddr, sc, sh, left, y, vy, bits, nw - w0, m < M, g.sign_mode, ImageOut{nullptr, 0u, 0u, 0u, false});
                    } else if (g.act == BNN_ACT_HARDTANH) {
                        epilogue_real<BNN_ACT_HARDTANH, NT>(taddr, sc, sh, left, y, vy, nullptr, 0, m < M, g.sign_mode, io);
                    } else if (g.act == BNN_ACT_SIGMOID) {
                        epilogue_real<BNN_ACT_SIGMOID, NT>(taddr, sc, sh, left, y, vy, nullptr, 0, m < M, g.sign_mode, io);
                    } else {
                        epilogue_real<BNN_ACT_NONE, NT>(taddr, sc, sh, left, y, vy, nullptr, 0, m < M, g.sign_mode, io);
                    }
                }
                // accumulator `sub` is free again: the MMA thread starts the next tile on accumulator 0
                // while accumulator 1 is still being read
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[sub]));
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
int launch_nt(const RealGemmArgs& r, void* workspace, bool image_ready, void* out_image, int out_kind, int* clear,
              int clear_words, cudaStream_t st) {
    using C = Cfg<NT>;
    constexpr int SMEM = C::STAGES * C::STAGE_BYTES + (int)sizeof(Control) + 128;
    const int sms = device_sm_count();
    if (sms <= 0 || !ensure_dynamic_smem(reinterpret_cast<const void*>(signw_img_kernel<NT>), SMEM)) return BNN_ERR_CUDA;
    const int nks = ceil_div(r.K, BK), mt = ceil_div(r.M, BM);
    uint8_t* img = static_cast<uint8_t*>(workspace);
    // (when the kernel before this one in the stream already wrote the image -- the layer that produced
    // these activations -- there is nothing to split)
    if (!image_ready)
        x_split_kernel<NT><<<mt * nks, 256, 0, st>>>(r.Af, r.lda, r.M, r.K, nks, img, r.splice_dim, r.splice_left, clear,
                                                     clear ? clear_words : 0);
    Args a{static_cast<uint8_t*>(out_image), ceil_div(r.N, BK), out_kind, img, r.Bb, r.ldb, r.M, r.N, r.K, r.scale, r.shift, r.act, r.sign_mode, r.Y, r.ldy, r.out_bits, r.ldob,
           tc_status()};
    if (!a.status.word) return BNN_ERR_CUDA;
    const int tiles = mt * ceil_div(r.N, UN);
    if (launch_pdl(signw_img_kernel<NT>, dim3(tiles < sms ? tiles : sms), dim3(THREADS), SMEM, st, a) != cudaSuccess)
        return BNN_ERR_CUDA;
    return launch_status();
}

}  // namespace

size_t signw_image_bytes(int M, int K, int terms) {
    return (size_t)ceil_div(M, BM) * ceil_div(K, BK) * (terms == 3 ? 3 : 2) * A_PLANE;
}

int launch_signw_img(const RealGemmArgs& r, int terms, void* workspace, bool image_ready, void* out_image, int out_kind,
                     int* clear, int clear_words, cudaStream_t st) {
    if (clear && image_ready) return BNN_ERR_UNSUPPORTED;   // no split kernel runs: nobody to clear the words
    return terms == 3 ? launch_nt<3>(r, workspace, image_ready, out_image, out_kind, clear, clear_words, st)
                      : launch_nt<2>(r, workspace, image_ready, out_image, out_kind, clear, clear_words, st);
}

}  // namespace bnn
