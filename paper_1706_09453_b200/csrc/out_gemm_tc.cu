// Real-valued top layer on +-1 activations, on the tensor cores (tcgen05 kind::f16, fp16
// operands, fp32 accumulators in TMEM):  z[m][c] = sum_h Wout[c][h] * a[m][h] + b[c].
//
// The weights are static, so they are prepared once (bnn_output_prepare): every class row
// is scaled by a power of two that brings its largest magnitude into [2^13, 2^14) and split
// into two fp16 terms, w * 2^e = hi + lo, |w*2^e - hi - lo| <= max(2^-22 |w*2^e|, 2^-25):
// about 22 significant bits, against 24 for fp32.  +-1 is exact in fp16, so with one MMA per
// term the accumulator holds the scaled logit up to fp32 accumulation rounding; the epilogue
// multiplies by 2^-e (exact) and adds the bias.  The prepared image is stored in exactly the
// order the MMA reads shared memory, so a pipeline stage of weights is ONE 16 KB bulk
// asynchronous copy (no tensor map, no multicast).
//
// Orientation: classes on the M side (TMEM lanes), frames on the N side.  A CTA tile is 128
// classes x 512 frames (two 256-column accumulators fed by the same weight stage, which
// halves the weight traffic from L2).  A warp stores 32 consecutive classes of one frame at a
// time: 128 contiguous bytes of the row-major [frames][classes] output.
#include <cuda_fp16.h>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BC = 128;           // classes per tile
constexpr int FN = 512;           // frames per tile (2 x 256)
constexpr int BK = 32;            // k per stage
constexpr int A_PLANE = BC * BK * 2;        // 8 KB per term
constexpr int A_BYTES = 2 * A_PLANE;        // hi + lo
constexpr int B_BYTES = FN * BK * 2;        // 32 KB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int STAGES = 4;
constexpr int MMA_WARP = 4, PROD_WARP0 = 5, PROD_WARPS = 8;
// Epilogue: warps 0-3 and four more after the producers, two per tensor-memory lane quarter.  Of each
// 256-frame accumulator the first group stores frames [0, 128), the second frames [128, 256): an
// accumulator is read, and handed back to the MMA thread, in half the time.
constexpr int EPI2_WARP0 = PROD_WARP0 + PROD_WARPS, EPI_WARPS = 8;
constexpr int THREADS = (EPI2_WARP0 + 4) * 32;   // 544
constexpr uint32_t TMEM_COLS = 512;

struct Control {
    uint64_t full[STAGES], empty[STAGES], acc_full, acc_empty[2];
    uint32_t tmem_base;
    WaitState wait;
};
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + (int)sizeof(Control) + 128;

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// 1-D bulk asynchronous copy global -> shared; completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ---- one-time preparation of the weights -------------------------------------------------
// rs[c] = 2^-e with e chosen so that max_h |W[c][h]| * 2^e lies in [2^13, 2^14)
__global__ void out_rowscale_kernel(const float* __restrict__ W, int ldw, int C, int H, int Cpad,
                                    float* __restrict__ rs) {
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (c >= Cpad) return;
    float mx = 0.f;
    if (c < C)
        for (int h = lane; h < H; h += 32) mx = fmaxf(mx, fabsf(W[(size_t)c * ldw + h]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    if (lane == 0) {
        int e = 0;
        if (mx > 0.f && mx < 3.0e38f) e = 13 - ilogbf(mx);
        e = e > 120 ? 120 : (e < -120 ? -120 : e);
        rs[c] = scalbnf(1.0f, -e);
    }
}

// One thread writes one 16-byte chunk (8 consecutive positions of a K step) of both terms.
__global__ void out_split_kernel(const float* __restrict__ W, int ldw, int C, int H, int Hs,
                                 const float* __restrict__ rs, uint8_t* __restrict__ img, long long chunks) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= chunks) return;
    const int row = (int)(i % BC);
    long long r = i / BC;
    const int cc = (int)(r & 1); r >>= 1;
    const int j = (int)(r & 1); r >>= 1;
    const int hs = (int)(r % Hs);
    const int ct = (int)(r / Hs);
    const int c = ct * BC + row;
    const float up = c < C ? 1.0f / rs[c] : 0.f;  // power of two: exact
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int pos = cc * 8 + e;                           // position inside the K step
        const int k = hs * BK + 8 * j + (pos >> 1) + 16 * (pos & 1);
        float v = (c < C && k < H) ? W[(size_t)c * ldw + k] * up : 0.f;
        const __half h1 = __float2half_rn(v);
        const __half h2 = __float2half_rn(v - __half2float(h1));
        const uint32_t b1 = __half_as_ushort(h1), b2 = __half_as_ushort(h2);
        if (e & 1) { hi[e >> 1] |= b1 << 16; lo[e >> 1] |= b2 << 16; }
        else { hi[e >> 1] = b1; lo[e >> 1] = b2; }
    }
    const size_t blk = ((size_t)ct * Hs + hs) * A_BYTES;
    const size_t off = (size_t)((j * 2 + cc) * BC + row) * 16;
    *reinterpret_cast<uint4*>(img + blk + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(img + blk + A_PLANE + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

// ---- the GEMM ---------------------------------------------------------------------------
// ZO: the activation bits stand for (0,1) instead of (-1,+1).
template <bool ZO>
__global__ void __launch_bounds__(THREADS, 1)
out_tc_kernel(const uint32_t* __restrict__ Hp, int ldhp, const uint8_t* __restrict__ img,
              const float* __restrict__ rs, const float* __restrict__ bias,
              int M, int C, int H, float* __restrict__ Z, int ldz, int* __restrict__ done, TcStatus status) {
    extern __shared__ uint8_t smem_raw[];
    // A kernel launched behind this one with programmatic stream serialisation (the log-softmax that
    // follows the frame tiles as they complete) may move onto the SMs once every CTA has got this far.
    pdl_trigger();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    Control* ctl = reinterpret_cast<Control*>(smem + STAGES * STAGE_BYTES);
    volatile int* abort_flag = &ctl->wait.abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nks = ceil_div(H, BK);
    const int c_tiles = ceil_div(C, BC), f_tiles = ceil_div(M, FN);
    const int tiles = c_tiles * f_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), PROD_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl->acc_full), 1);
        mbar_init(smem_u32(&ctl->acc_empty[0]), EPI_WARPS);
        mbar_init(smem_u32(&ctl->acc_empty[1]), EPI_WARPS);
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

    if (warp >= PROD_WARP0 && warp < EPI2_WARP0) {
        // ---------------- producers: thread p widens the packed activation rows p and p+256;
        // the first producer thread also starts the bulk copy of the stage's weights.
        const int p = threadIdx.x - PROD_WARP0 * 32;  // 0..255
        const int my_tiles = (tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
        const int total = my_tiles * nks;
        // Packed rows are read 16 bytes (4 stages) at a time, one group ahead of use.  Words at
        // or beyond ceil(H/32) may hold anything: the weight image is zero there.
        const int ngroups = ceil_div(nks, 4);
        int pf_g = 0, pf_tile = blockIdx.x, pf_left = my_tiles;
        auto fetch = [&](uint4 (&o)[2]) {
            o[0] = make_uint4(0u, 0u, 0u, 0u);
            o[1] = o[0];
            if (pf_left == 0) return;
            const int f0 = (pf_tile / c_tiles) * FN;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int f = f0 + p + 256 * q;
                if (f < M) o[q] = ldg_nc_u4(reinterpret_cast<const uint4*>(Hp + (size_t)f * ldhp) + pf_g);
            }
            if (++pf_g == ngroups) { pf_g = 0; pf_tile += gridDim.x; --pf_left; }
        };
        uint4 grp[2], nxt[2];
        fetch(grp);
        fetch(nxt);
        int ks = 0, tile = blockIdx.x;
        for (int it = 0; it < total; ++it) {
            const int s = it % STAGES;
            const uint32_t ph = (uint32_t)((it / STAGES) & 1);
            const int sub = ks & 3;
            uint32_t cur[2];
#pragma unroll
            for (int q = 0; q < 2; ++q)
                cur[q] = sub == 0 ? grp[q].x : sub == 1 ? grp[q].y : sub == 2 ? grp[q].z : grp[q].w;
            if (!warp_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag, lane)) break;
            const uint32_t st = smem_u32(smem) + s * STAGE_BYTES;
            if (p == 0) {
                const int ct = tile % c_tiles;
                mbar_expect_tx(smem_u32(&ctl->full[s]), A_BYTES);
                bulk_g2s(st, img + ((size_t)ct * nks + ks) * A_BYTES, A_BYTES, smem_u32(&ctl->full[s]));
            }
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint32_t nw = ~cur[q];
                uint32_t wv[16];
                if (ZO) {   // (0,1) activations: 1.0 (0x3C00) where the bit is set, +0 elsewhere
#pragma unroll
                    for (int t = 0; t < 16; ++t) wv[t] = ((cur[q] >> t) & 0x00010001u) * 0x3C00u;
                } else {
#pragma unroll
                    for (int t = 0; t < 16; ++t) wv[t] = ((nw << (15 - t)) & 0x80008000u) | 0x3C003C00u;
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    sts128(st + A_BYTES + (c * FN + p + 256 * q) * 16, wv[4 * c], wv[4 * c + 1], wv[4 * c + 2], wv[4 * c + 3]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
            ++ks;
            if ((ks & 3) == 0 || ks == nks) {   // group used up: take the prefetched one
                grp[0] = nxt[0]; grp[1] = nxt[1];
                fetch(nxt);
            }
            if (ks == nks) { ks = 0; tile += gridDim.x; }
        }
    } else if (warp == MMA_WARP) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kAccF32, kFmtF16, kFmtF16, BC, 256);
            // MMAs of one stage into accumulator `sub` (frames [256 sub, 256 sub + 256) of the tile)
            auto issue = [&](int s, int sub, int ks) {
                const uint32_t a0 = smem_u32(smem + s * STAGE_BYTES);
                const uint32_t b0 = a0 + A_BYTES;
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint64_t db = smem_desc_kmajor(b0 + 2 * j * (FN * 16) + sub * 256 * 16, FN * 16, 128);
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const uint64_t da = smem_desc_kmajor(a0 + q * A_PLANE + 2 * j * (BC * 16), BC * 16, 128);
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
                const int lead = nks < STAGES ? nks : STAGES;
                for (int ks = 0; ks < lead && ok; ++ks) {
                    const int s = (it + ks) % STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)(((it + ks) / STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue(s, 0, ks);
                }
                if (!ok) break;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[1]), par, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                for (int ks = 0; ks < lead; ++ks) {
                    const int s = (it + ks) % STAGES;
                    issue(s, 1, ks);
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                it += lead;
                for (int ks = lead; ks < nks; ++ks, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)((it / STAGES) & 1), abort_flag);
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
        // ---------------- epilogue: thread = one class (TMEM lane), columns = frames
        const int row_in_tile = (warp & 3) * 32 + lane;   // a warp reads the lanes of its quarter: 32 (warp % 4) ..
        const int half = warp < 4 ? 0 : 1;                // which 128 frames of each accumulator
        uint64_t pol;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int c = (tile % c_tiles) * BC + row_in_tile;
            const int f0 = (tile / c_tiles) * FN;
            const float scl = rs[c];                       // rs is padded to whole tiles
            const float bia = (bias && c < C) ? bias[c] : 0.f;
            // the four warps of a group take the same decision, so none is left at a barrier
            const bool got = warp_wait(smem_u32(&ctl->acc_full), (uint32_t)(tl & 1), abort_flag, lane);
            ok = half ? epi_all_b(got) : epi_all(got);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
#pragma unroll 1
            for (int sub = 0; sub < 2; ++sub) {
#pragma unroll 1
                for (int g4 = 0; g4 < 4; ++g4) {
                    const int gi = sub * 8 + half * 4 + g4;       // group of 32 frames
                    if (f0 + gi * 32 >= M) break;                  // uniform over the warp
                    uint32_t acc[32];
                    tmem_ld32(taddr + gi * 32, acc);
                    tmem_ld_wait();
                    if (c < C) {
                        float* dst = Z + (size_t)(f0 + gi * 32) * ldz + c;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (f0 + gi * 32 + j < M) {
                                const float zv = fmaf(__uint_as_float(acc[j]), scl, bia);
                                asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(dst + (size_t)j * ldz), "f"(zv), "l"(pol) : "memory");
                            }
                    }
                }
                // this warp's share of accumulator `sub` has been read: once all eight warps are through,
                // the MMA thread may start the next tile on it
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[sub]));
            }
            if (done) {
                // this warp's logits of the tile are stored: count it in for the tile's 512 frames (release)
                __threadfence();
                __syncwarp();
                if (lane == 0)
                    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(done + tile / c_tiles) : "memory");
            }
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

size_t out_prepared_bytes(int C, int H) {
    const size_t ct = ceil_div(C, BC), hs = ceil_div(H, BK);
    return ct * hs * A_BYTES + ct * BC * sizeof(float);
}

int launch_out_prepare(const float* W, int ldw, int C, int H, void* prepared, cudaStream_t st) {
    const int ct = ceil_div(C, BC), hs = ceil_div(H, BK);
    uint8_t* img = static_cast<uint8_t*>(prepared);
    float* rs = reinterpret_cast<float*>(img + (size_t)ct * hs * A_BYTES);
    out_rowscale_kernel<<<ceil_div(ct * BC, 8), 256, 0, st>>>(W, ldw, C, H, ct * BC, rs);
    const long long chunks = (long long)ct * hs * 4 * BC;
    out_split_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(W, ldw, C, H, hs, rs, img, chunks);
    return launch_status();
}

int out_tc_group_rows() { return FN; }
int out_tc_group_arrivals(int C) { return ceil_div(C, BC) * EPI_WARPS; }
size_t out_tc_done_bytes(int M) { return (size_t)(ceil_div(M, FN) + 1) * sizeof(int); }
// With no more tiles than SMs every tile ends at about the same time: nothing for a following kernel to
// overlap with (measured: 1-2 % slower than two launches in a row on 256 frames).
bool out_tc_more_than_one_wave(int M, int C) { return ceil_div(M, FN) * ceil_div(C, BC) > device_sm_count(); }

int launch_out_tc(const uint32_t* Hp, int ldhp, const void* prepared, const float* bias,
                  int M, int C, int H, float* Z, int ldz, int zo, int* done, cudaStream_t st) {
    const int sms = device_sm_count();
    if (sms <= 0 || !ensure_dynamic_smem(reinterpret_cast<const void*>(out_tc_kernel<false>), SMEM_BYTES) ||
        !ensure_dynamic_smem(reinterpret_cast<const void*>(out_tc_kernel<true>), SMEM_BYTES))
        return BNN_ERR_CUDA;
    const int ct = ceil_div(C, BC), hs = ceil_div(H, BK);
    const uint8_t* img = static_cast<const uint8_t*>(prepared);
    const float* rs = reinterpret_cast<const float*>(img + (size_t)ct * hs * A_BYTES);
    const int tiles = ct * ceil_div(M, FN);
    const TcStatus status = tc_status();
    if (!status.word) return BNN_ERR_CUDA;
    if (zo)
        out_tc_kernel<true><<<tiles < sms ? tiles : sms, THREADS, SMEM_BYTES, st>>>(Hp, ldhp, img, rs, bias, M, C, H, Z, ldz, done, status);
    else
        out_tc_kernel<false><<<tiles < sms ? tiles : sms, THREADS, SMEM_BYTES, st>>>(Hp, ldhp, img, rs, bias, M, C, H, Z, ldz, done, status);
    return launch_status();
}

}  // namespace bnn
