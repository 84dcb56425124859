// Real-valued layer on real-valued activations, on the tensor cores: the top layer of the
// binary-weights-only networks of Algorithm 1 (whose last hidden layer hands on fp32 values) and
// the real-valued hidden layers of the paper's mixed networks (Table 2), with an optional
// activation f (Sigmoid, clamp):
//   z[m][c] = f( sum_h Wout[c][h] * a[m][h] + b[c] ).
//
// Both operands are split into two fp16 terms.  The weights use the image bnn_output_prepare
// builds (per-row power-of-two scaling, w * 2^e = w1 + w2, about 22 significant bits).  The
// activations are split once per call into a scratch image, a = a1 + a2 with
// |a - a1 - a2| <= max(2^-22 |a|, 2^-25), in the order the MMA reads shared memory
// (h_split_kernel, a memory-bound pass).  Three MMAs per K step, a1 w1 + a1 w2 + a2 w1,
// accumulate in fp32 in tensor memory; the term a2 w2 (<= 2^-22 |a w|) is dropped, so
//   |z - exact| <= ~3 * 2^-22 * sum_h |a[m][h]| |Wout[c][h]|  + fp32 accumulation rounding.
// Activations must be finite fp16-range numbers (|a| < 65504; the outputs of hardtanh are
// within [-1, 1]).
//
// Orientation as in out_gemm_tc.cu: classes on the M side (TMEM lanes), frames on the N side;
// a CTA tile is 128 classes x 256 frames with two accumulators, so the epilogue of one tile
// overlaps the MMAs of the next.  A pipeline stage (32 positions of K) is two bulk copies:
// 16 KB of the weight image and 32 KB of the activation image; nothing is widened on chip.
//   warp 5       one thread issues the bulk copies
//   warp 4       one thread issues the MMAs (6 per stage) and the commits
//   warps 0-3    epilogue: z = acc * 2^-e + b, 32 consecutive classes of a frame per warp store
// Every wait is bounded; a wait that runs out sets the CTA's abort flag, all roles fall
// through to the common teardown and the device status word is set.
#include <cuda_fp16.h>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BC = 128;           // classes per tile (as the prepared weight image)
constexpr int FN = 256;           // frames per tile
constexpr int BK = 32;            // k per stage
constexpr int A_PLANE = BC * BK * 2;        // 8 KB per weight term
constexpr int A_BYTES = 2 * A_PLANE;
constexpr int B_PLANE = FN * BK * 2;        // 16 KB per activation term
constexpr int B_BYTES = 2 * B_PLANE;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;   // 48 KB
constexpr int STAGES = 4;
constexpr int EPI_WARPS = 4, MMA_WARP = 4, TMA_WARP = 5;
constexpr int THREADS = (TMA_WARP + 1) * 32;
constexpr uint32_t TMEM_COLS = 512;

struct Control {
    uint64_t full[STAGES], empty[STAGES], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    WaitState wait;
};
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + (int)sizeof(Control) + 128;
static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");

__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ---- split: one CTA per (tile of 256 frames, stage): thread = frame row ---------------------
// Block (ft, ks) of the image: [term 0..1][chunk c = 2 j + cc][row 0..255][16 bytes], where
// chunk (j, cc) holds, in element e, position k = 32 ks + 8 j + (pos >> 1) + 16 (pos & 1),
// pos = 8 cc + e: the order of the prepared weight image, so both operands agree on k.
// FROM_I32: the activations are Sigmoid(fma(scale[h], d, shift[h])) of integer dot products d (a binary
// layer with Sigmoid units, Section 3.2 / Table 2), evaluated here instead of in a pass of their own.
template <bool FROM_I32>
__global__ void __launch_bounds__(FN)
h_split_kernel(const void* __restrict__ src, int ldh, int M, int H, int nks, uint8_t* __restrict__ img,
               const float* __restrict__ scale, const float* __restrict__ shift) {
    const int ft = blockIdx.x / nks, ks = blockIdx.x % nks;
    const int row = threadIdx.x, m = ft * FN + row;
    float v[BK];
    const bool vec = (ldh % 4 == 0) && ((reinterpret_cast<uintptr_t>(src) & 15) == 0) && ks * BK + BK <= H;
    if (m < M && vec) {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint32_t*>(src) + (size_t)m * ldh + ks * BK);
#pragma unroll
        for (int q = 0; q < BK / 4; ++q) {
            const uint4 t = __ldg(p + q);
            v[4 * q] = __uint_as_float(t.x); v[4 * q + 1] = __uint_as_float(t.y);
            v[4 * q + 2] = __uint_as_float(t.z); v[4 * q + 3] = __uint_as_float(t.w);
        }
    } else {
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const int kk = ks * BK + k;
            v[k] = (m < M && kk < H) ? __uint_as_float(__ldg(static_cast<const uint32_t*>(src) + (size_t)m * ldh + kk)) : 0.f;
        }
    }
    if (FROM_I32) {
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const int kk = ks * BK + k;
            if (m < M && kk < H) {
                const float d = (float)__float_as_int(v[k]);
                const float y = fmaf(scale ? __ldg(scale + kk) : 1.0f, d, shift ? __ldg(shift + kk) : 0.0f);
                v[k] = 1.0f / (1.0f + expf(-y));
            } else {
                v[k] = 0.f;
            }
        }
    }
    uint8_t* blk = img + ((size_t)ft * nks + ks) * B_BYTES;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int j = c >> 1, cc = c & 1;
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int pos = cc * 8 + e;
            const float x = v[8 * j + (pos >> 1) + 16 * (pos & 1)];
            const __half h1 = __float2half_rn(x);
            const __half h2 = __float2half_rn(x - __half2float(h1));
            const uint32_t b1 = __half_as_ushort(h1), b2 = __half_as_ushort(h2);
            if (e & 1) { hi[e >> 1] |= b1 << 16; lo[e >> 1] |= b2 << 16; }
            else { hi[e >> 1] = b1; lo[e >> 1] = b2; }
        }
        *reinterpret_cast<uint4*>(blk + (size_t)(c * FN + row) * 16) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4*>(blk + B_PLANE + (size_t)(c * FN + row) * 16) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
}

// ---- the GEMM ---------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS, 1)
outf_tc_kernel(const uint8_t* __restrict__ himg, const uint8_t* __restrict__ wimg,
               const float* __restrict__ rs, const float* __restrict__ bias,
               int M, int C, int H, float* __restrict__ Z, int ldz, int act, TcStatus status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    Control* ctl = reinterpret_cast<Control*>(smem + STAGES * STAGE_BYTES);
    volatile int* abort_flag = &ctl->wait.abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nks = ceil_div(H, BK);
    const int c_tiles = ceil_div(C, BC), f_tiles = ceil_div(M, FN);
    const int tiles = c_tiles * f_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);    // the copying thread (+ bytes)
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), EPI_WARPS);
        }
        wait_state_init(&ctl->wait, status);
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

    if (warp == TMA_WARP) {
        // ---------------- one thread streams both images, class tiles varying fastest so that
        // consecutive CTAs share a tile of frames in L2
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const uint8_t* wsrc = wimg + (size_t)(tile % c_tiles) * nks * A_BYTES;
                const uint8_t* hsrc = himg + (size_t)(tile / c_tiles) * nks * B_BYTES;
                for (int ks = 0; ks < nks; ++ks, ++it) {
                    const int s = it % STAGES;
                    if (it >= STAGES) {
                        ok = mbar_wait(smem_u32(&ctl->empty[s]), (uint32_t)(((it / STAGES) - 1) & 1), abort_flag);
                        if (!ok) break;
                    }
                    const uint32_t bar = smem_u32(&ctl->full[s]);
                    const uint32_t st = smem_u32(smem) + s * STAGE_BYTES;
                    mbar_arrive_expect_tx(bar, STAGE_BYTES);
                    bulk_g2s(st, wsrc + (size_t)ks * A_BYTES, A_BYTES, bar);
                    bulk_g2s(st + A_BYTES, hsrc + (size_t)ks * B_BYTES, B_BYTES, bar);
                }
            }
        }
        __syncwarp();
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kAccF32, kFmtF16, kFmtF16, BC, FN);
            int it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
                const int b = tl & 1;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), (uint32_t)(((tl >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d = tmem + (uint32_t)(b * FN);
                for (int ks = 0; ks < nks; ++ks, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)((it / STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a0 = smem_u32(smem + s * STAGE_BYTES);
                    const uint32_t b0 = a0 + A_BYTES;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {   // K step of 16 = two 16-byte chunks
                        const uint64_t w1 = smem_desc_kmajor(a0 + 2 * j * (BC * 16), BC * 16, 128);
                        const uint64_t w2 = smem_desc_kmajor(a0 + A_PLANE + 2 * j * (BC * 16), BC * 16, 128);
                        const uint64_t h1 = smem_desc_kmajor(b0 + 2 * j * (FN * 16), FN * 16, 128);
                        const uint64_t h2 = smem_desc_kmajor(b0 + B_PLANE + 2 * j * (FN * 16), FN * 16, 128);
                        mma_f16(d, w1, h1, idesc, (ks | j) != 0);
                        mma_f16(d, w2, h1, idesc, 1u);
                        mma_f16(d, w1, h2, idesc, 1u);
                    }
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) mma_commit(smem_u32(&ctl->acc_full[b]));
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: thread = one class (TMEM lane), columns = frames
        const int row_in_tile = warp * 32 + lane;
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int c = (tile % c_tiles) * BC + row_in_tile;
            const int f0 = (tile / c_tiles) * FN;
            const float scl = rs[c];                       // rs is padded to whole tiles
            const float bia = (bias && c < C) ? bias[c] : 0.f;
            const int b = tl & 1;
            ok = epi_all(warp_wait_relaxed(smem_u32(&ctl->acc_full[b]), (uint32_t)((tl >> 1) & 1), abort_flag, lane));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * FN);
#pragma unroll 1
            for (int gi = 0; gi < FN / 32; ++gi) {
                if (f0 + gi * 32 >= M) break;              // uniform over the CTA
                uint32_t acc[32];
                tmem_ld32(taddr + gi * 32, acc);
                tmem_ld_wait();
                if (c < C) {
                    float* dst = Z + (size_t)(f0 + gi * 32) * ldz + c;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (f0 + gi * 32 + j < M) {
                            float v = fmaf(__uint_as_float(acc[j]), scl, bia);
                            if (act == BNN_ACT_SIGMOID) v = 1.0f / (1.0f + expf(-v));
                            else if (act == BNN_ACT_HARDTANH) v = fminf(fmaxf(v, -1.0f), 1.0f);
                            dst[(size_t)j * ldz] = v;
                        }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
    if (threadIdx.x == 0 && ctl->wait.abort) atomicExch(status.word, 1);
}

}  // namespace

size_t outf_image_bytes(int M, int H) {
    return (size_t)ceil_div(M, FN) * ceil_div(H, BK) * B_BYTES;
}

int launch_outf_tc(const float* Hf, int ldhf, const void* prepared, const float* bias,
                   int M, int C, int H, float* Z, int ldz, int act, void* workspace, bool image_ready, cudaStream_t st) {
    const int sms = device_sm_count();
    if (sms <= 0 || !ensure_dynamic_smem(reinterpret_cast<const void*>(outf_tc_kernel), SMEM_BYTES)) return BNN_ERR_CUDA;
    const int ct = ceil_div(C, BC), hs = ceil_div(H, BK), ft = ceil_div(M, FN);
    // the prepared weight image: ct * hs blocks of both terms, then the per-class factors 2^-e
    const uint8_t* wimg = static_cast<const uint8_t*>(prepared);
    const float* rs = reinterpret_cast<const float*>(wimg + (size_t)ct * hs * A_BYTES);
    uint8_t* himg = static_cast<uint8_t*>(workspace);
    const TcStatus status = tc_status();
    if (!status.word) return BNN_ERR_CUDA;
    if (!image_ready)   // (else the layer that produced the activations wrote the image itself)
        h_split_kernel<false><<<ft * hs, FN, 0, st>>>(Hf, ldhf, M, H, hs, himg, nullptr, nullptr);
    const int tiles = ct * ft;
    outf_tc_kernel<<<tiles < sms ? tiles : sms, THREADS, SMEM_BYTES, st>>>(himg, wimg, rs, bias, M, C, H, Z, ldz, act, status);
    return launch_status();
}


int launch_outf_image_from_i32(const int32_t* D, int ldd, const float* scale, const float* shift, int M, int H,
                               void* image, cudaStream_t st) {
    const int hs = ceil_div(H, BK), ft = ceil_div(M, FN);
    h_split_kernel<true><<<ft * hs, FN, 0, st>>>(D, ldd, M, H, hs, static_cast<uint8_t*>(image), scale, shift);
    return launch_status();
}

}  // namespace bnn
