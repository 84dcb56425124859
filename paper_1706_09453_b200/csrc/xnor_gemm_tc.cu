// XNOR GEMM on the 5th-generation tensor cores (tcgen05, kind::i8, accumulators in TMEM).
//
// Identity used: with bits a, w in {0,1} standing for -1/+1,
//     dot = K - 2 popc(a) - 2 popc(w) + 4 popc(a AND w),
// and popc(a AND w) is an ordinary integer dot product of the bit vectors, i.e. a dense
// contraction the tensor core can do.  Packed bits stay 1 bit per element in HBM/L2; they
// are widened to bytes only inside the SM, on the way into shared memory:
//   - the contraction index may be permuted freely as long as A and W use the same
//     permutation, so byte j of output word (w_i, t) is simply bit 8j+t of packed word w_i:
//     one AND with the mask 0x01010101 << t widens 4 bits to 4 bytes;
//   - that leaves the byte holding 2^t instead of 1.  A keeps 2^t, W is bit-reversed within
//     bytes first so its byte holds 2^(7-t); every product is then 2^7 * a * w and the
//     accumulator is exactly 128 * popc(a AND w) (u8 x u8 -> s32).
//
// One persistent CTA per SM, tile 128 frames x 192 units, 128 bits of K per pipeline stage.
// Tiles are numbered with the unit index fastest, so that the CTAs running at the same time
// share frame rows (L2 hits) and, with int32 output, fill whole output rows together.
// Warp roles: warps 0-3 epilogue (TMEM -> thresholds -> packed bits / int32), warp 4 issues
// the MMAs, warps 5-8 widen the frame rows and warps 9-14 the unit rows (one packed row per
// thread and stage).  The kernel is bound by the shared-memory pipe, not by the tensor pipe,
// so the frame operand never touches shared memory: its producers write the widened bytes
// straight into tensor memory (tcgen05.st, lane = frame) and the MMA reads A from there.
// TMEM budget (512 columns): two 192-column accumulators, so that the epilogue of tile i
// overlaps the MMAs of tile i+1, plus 4 stages x 32 columns of A.
// The packed rows themselves reach the SM by TMA: one 2-D tile load per operand brings the
// next four stages (64 bytes per row) of all rows of the tile into a small staging ring
// (64-byte swizzle, no multicast); each producer thread then reads its own row, 16 bytes per
// stage, free of bank conflicts.  No thread waits on a global load.
// The row popcounts the identity needs cost nothing extra: each producer thread sees every
// word of its row anyway, sums their popcounts and hands the total to the epilogue through a
// small ring in shared memory.
#include <cuda.h>

#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {

__device__ int g_tc_status = 0;  // set to 1 by a CTA whose bounded wait ran out
int* tc_status_ptr();

namespace {

using namespace tc;

constexpr int BM = 128, BN = 192, BK = 128;  // BK: bits of K per stage = bytes per widened row
constexpr int STAGES = 4;
constexpr int B_BYTES = BN * BK, STAGE_BYTES = B_BYTES;  // only the unit operand lives in shared memory
constexpr int EPI_WARPS = 4, MMA_WARP = 4, PROD_WARP0 = 5, A_WARPS = 4, B_WARPS = BN / 32;
constexpr int PROD_WARPS = A_WARPS + B_WARPS;
constexpr int TMA_WARP = PROD_WARP0 + PROD_WARPS;        // one more warp issues the tile loads
constexpr int THREADS = (TMA_WARP + 1) * 32;             // 512
constexpr int QUADS = 3;                                 // staging ring: 3 groups of 4 stages
constexpr int QA_BYTES = BM * 64, QB_BYTES = BN * 64, QUAD_BYTES = QA_BYTES + QB_BYTES;
constexpr uint32_t TMEM_A_COL = 2 * BN;                  // A stages start after the two accumulators
constexpr uint32_t A_COLS = BK / 4;                      // 32-bit columns per A stage
constexpr uint32_t TMEM_COLS = 512;

// Producers may run up to STAGES tiles ahead of the MMA warp (when a tile is a single stage)
// and the MMA warp up to 2 tiles ahead of the epilogue, hence the depth of the popcount ring.
constexpr int RING = 8;

struct Control {
    int T[BN];              // per-unit constant of the epilogue (threshold or 2 popc(w) - K)
    uint32_t flipw[BN / 32];
    int popc[RING][BM + BN];  // per tile: popcount of each frame row, then of each unit row
    uint64_t full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], popc_ready[RING];
    uint64_t quad_full[QUADS], quad_empty[QUADS];
    // int32 output: per warp two staging blocks of 32 rows x 128 bytes (pitch 144: conflict-free 16-byte accesses)
    __align__(16) int cstage[EPI_WARPS][2][32][36];
    uint32_t tmem_base;
    int abort;
};
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + QUADS * QUAD_BYTES + (int)sizeof(Control) + 1024;




struct ProducerArgs {
    uint32_t smem;        // shared-space address of stage 0
    uint32_t tmem;        // base of the tensor-memory allocation
    Control* ctl;
    volatile int* abort_flag;
    int tiles, m_tiles, nks, kw;
    uint32_t tmask;
    int lane;
};

__device__ __forceinline__ uint4 lds128u(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// 2-D tiled TMA load (no multicast): box at element coordinates (x = word, y = row).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Producer loop of one thread: row `r` of every tile of this CTA, stage by stage.  IS_A picks
// the operand (frames / units): byte weights 2^t / 2^(7-t), destination (tensor memory /
// shared memory) and the slot in the popcount ring are compile-time.
template <bool IS_A>
__device__ __forceinline__ void produce(const ProducerArgs& a, int r) {
    Control* ctl = a.ctl;
    const int my_tiles = (a.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
    const int total = my_tiles * a.nks;
    const uint32_t dst0 = a.smem + r * 16;
    // TMEM lane of this thread's frame row: a warp may only touch lanes 32*(warp%4)..+31
    const uint32_t tdst0 = a.tmem + ((uint32_t)(r & ~31) << 16) + TMEM_A_COL;
    // this row inside a staging slot: 64 bytes per row, 16-byte chunk c stored at c ^ ((r/2)%4)
    const uint32_t stg0 = a.smem + STAGES * STAGE_BYTES + (IS_A ? 0 : QA_BYTES) + r * 64;
    const uint32_t sw = (uint32_t)(r >> 1) & 3u;
    const int last_word = a.kw - 1 - 4 * (a.nks - 1);   // index of the last valid word in the last stage
    int qslot = 0;
    uint32_t qph = 0;
    int pc = 0, ks = 0, slot = 0, s = 0;
    uint32_t ph = 1;  // parity to wait for on `empty`: a fresh barrier passes parity 1
    for (int it = 0; it < total; ++it) {
        const int qi = ks & 3;   // stage inside its group of four
        if (qi == 0 && !warp_wait(smem_u32(&ctl->quad_full[qslot]), qph, a.abort_flag, a.lane)) break;
        uint4 v = lds128u(stg0 + qslot * QUAD_BYTES + (((uint32_t)qi ^ sw) << 4));
        if (qi == 3 || ks == a.nks - 1) {   // group used up (values are in registers): release its slot
            __syncwarp();
            if (a.lane == 0) mbar_arrive(smem_u32(&ctl->quad_empty[qslot]));
            if (++qslot == QUADS) { qslot = 0; qph ^= 1u; }
        }
        if (ks == a.nks - 1) {   // last stage of the row: clear the bits at positions >= K
            if (last_word == 0) { v.x &= a.tmask; v.y = 0u; v.z = 0u; v.w = 0u; }
            else if (last_word == 1) { v.y &= a.tmask; v.z = 0u; v.w = 0u; }
            else if (last_word == 2) { v.z &= a.tmask; v.w = 0u; }
            else { v.w &= a.tmask; }
        }
        pc += __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
        if (!IS_A) {  // reverse the bits inside each byte, so that bit t carries weight 2^(7-t)
            v.x = __brev(__byte_perm(v.x, 0, 0x0123));
            v.y = __brev(__byte_perm(v.y, 0, 0x0123));
            v.z = __brev(__byte_perm(v.z, 0, 0x0123));
            v.w = __brev(__byte_perm(v.w, 0, 0x0123));
        }
        if (!warp_wait(smem_u32(&ctl->empty[s]), ph, a.abort_flag, a.lane)) break;
        if (IS_A) {
            // column 4t+i of the stage holds bytes 16t+4i .. 16t+4i+3 of K: the same order as
            // the 16-byte chunks of the unit operand in shared memory
            uint32_t wr[32];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t mk = 0x01010101u << t;
                wr[4 * t + 0] = v.x & mk; wr[4 * t + 1] = v.y & mk;
                wr[4 * t + 2] = v.z & mk; wr[4 * t + 3] = v.w & mk;
            }
            tmem_st32(tdst0 + s * A_COLS, wr);
            tmem_st_wait();
            tc_fence_before_sync();
        } else {
            const uint32_t dst = dst0 + s * STAGE_BYTES;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t mk = 0x01010101u << (7 - t);
                sts128(dst + t * (BN * 16), v.x & mk, v.y & mk, v.z & mk, v.w & mk);
            }
            fence_proxy_async_smem();
        }
        __syncwarp();
        if (a.lane == 0) mbar_arrive(smem_u32(&ctl->full[s]));
        if (++s == STAGES) { s = 0; ph ^= 1u; }
        if (++ks == a.nks) {  // row finished: publish its popcount for this tile
            // The slot was last read by the epilogue of the tile RING tiles back, which is done:
            // this tile's stages could only be filled after the MMAs of the tile STAGES back had
            // run, and those waited for the epilogue two tiles before that.
            ctl->popc[slot][(IS_A ? 0 : BM) + r] = pc;
            __syncwarp();
            if (a.lane == 0) mbar_arrive(smem_u32(&ctl->popc_ready[slot]));
            pc = 0; ks = 0;
            slot = (slot + 1) % RING;
        }
    }
}

template <bool STORE_C, bool SIGN_PACK>
__global__ void __launch_bounds__(THREADS, 1)
xnor_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               int M, int N, int K, int32_t* __restrict__ C, int ldc,
               const int32_t* __restrict__ thr, const uint32_t* __restrict__ flip,
               uint32_t* __restrict__ out_bits, int ldob, int* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(smem + STAGES * STAGE_BYTES + QUADS * QUAD_BYTES);
    volatile int* abort_flag = &ctl->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kw = words_for(K);
    const uint32_t tmask = tail_mask(K);
    const int nks = ceil_div(K, BK);
    const int m_tiles = ceil_div(M, BM), n_tiles = ceil_div(N, BN);
    const int tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), PROD_WARPS);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), EPI_WARPS);
        }
        for (int b = 0; b < RING; ++b) mbar_init(smem_u32(&ctl->popc_ready[b]), PROD_WARPS);
        for (int b = 0; b < QUADS; ++b) {
            mbar_init(smem_u32(&ctl->quad_full[b]), 1);            // the issuing thread (+ bytes)
            mbar_init(smem_u32(&ctl->quad_empty[b]), PROD_WARPS);  // every producer warp has read it
        }
        ctl->abort = 0;
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
        // ---------------- producers: packed words -> widened byte tiles in shared memory
        ProducerArgs pa{smem_u32(smem), tmem, ctl, abort_flag, tiles, m_tiles, nks, kw, tmask, lane};
        if (warp == TMA_WARP) {
            // ---------------- one thread feeds the staging ring, a group of four stages at a time
            if (lane == 0) {
                const uint32_t stg = smem_u32(smem) + STAGES * STAGE_BYTES;
                const int nq = ceil_div(nks, 4);
                int qc = 0;
                bool ok = true;
                for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                    const int n0 = (tile % n_tiles) * BN, m0 = (tile / n_tiles) * BM;   // unit tiles vary fastest
                    for (int gq = 0; gq < nq; ++gq, ++qc) {
                        const int slot = qc % QUADS;
                        if (qc >= QUADS) {
                            ok = mbar_wait(smem_u32(&ctl->quad_empty[slot]), (uint32_t)(((qc / QUADS) - 1) & 1), abort_flag);
                            if (!ok) break;
                        }
                        const uint32_t bar = smem_u32(&ctl->quad_full[slot]);
                        mbar_arrive_expect_tx(bar, QUAD_BYTES);
                        tma_load_2d(stg + slot * QUAD_BYTES, &mapA, gq * 16, m0, bar);
                        tma_load_2d(stg + slot * QUAD_BYTES + QA_BYTES, &mapB, gq * 16, n0, bar);
                    }
                }
            }
            __syncwarp();
        } else if (warp < PROD_WARP0 + A_WARPS) {
            produce<true>(pa, (warp & 3) * 32 + lane);
        } else {
            produce<false>(pa, (warp - PROD_WARP0 - A_WARPS) * 32 + lane);
        }
    } else if (warp == MMA_WARP) {
        // ---------------- MMA issue: one thread
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kAccS32, kFmtU8, kFmtU8, BM, BN);
            int it = 0;
            int tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
                const int b = tl & 1;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), (uint32_t)(((tl >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d = tmem + (uint32_t)(b * BN);
                for (int ks = 0; ks < nks; ++ks, ++it) {
                    const int s = it % STAGES;
                    ok = mbar_wait(smem_u32(&ctl->full[s]), (uint32_t)((it / STAGES) & 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t b0 = smem_u32(smem + s * STAGE_BYTES);
                    const uint32_t ta = tmem + TMEM_A_COL + s * A_COLS;
#pragma unroll
                    for (int j = 0; j < BK / 32; ++j) {   // 32 bytes of K = 8 TMEM columns of A per MMA
                        const uint64_t db = smem_desc_kmajor(b0 + 2 * j * (BN * 16), BN * 16, 128);
                        mma_i8_ts(d, ta + 8 * j, db, idesc, (ks | j) != 0);
                    }
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                if (ok) mma_commit(smem_u32(&ctl->acc_full[b]));
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: 128 threads, thread = one frame (TMEM lane)
        const int row_in_tile = warp * 32 + lane;
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int n0 = (tile % n_tiles) * BN, m0 = (tile / n_tiles) * BM;   // unit tiles vary fastest
            const int m = m0 + row_in_tile;
            // row popcounts of this tile, published by the producers
            ok = epi_all(warp_wait(smem_u32(&ctl->popc_ready[tl % RING]), (uint32_t)((tl / RING) & 1), abort_flag, lane));
            if (!ok) break;
            const int* pcs = ctl->popc[tl % RING];
            const int pa = pcs[row_in_tile];
            epi_bar_sync();  // previous tile's readers of T are done
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int nl = row_in_tile + h * 128, n = n0 + nl;
                if (nl < BN) {
                    int t = 0;
                    if (n < N) {
                        const int pw = pcs[BM + nl];
                        t = (SIGN_PACK && !STORE_C) ? 32 * (thr[n] + 2 * pw - K) : 2 * pw - K;
                    }
                    ctl->T[nl] = t;
                }
            }
            if (SIGN_PACK && row_in_tile < BN / 32) {
                const int wi = (n0 >> 5) + row_in_tile;
                ctl->flipw[row_in_tile] = wi < words_for(N) ? flip[wi] : 0u;
            }
            epi_bar_sync();
            const int b = tl & 1;
            // all four epilogue warps take the same decision, so none is left at a barrier
            ok = epi_all(warp_wait(smem_u32(&ctl->acc_full[b]), (uint32_t)((tl >> 1) & 1), abort_flag, lane));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * BN);
            uint32_t words[BN / 32];
#pragma unroll
            for (int g = 0; g < BN / 32; ++g) {
                uint32_t acc[32];
                tmem_ld32(taddr + g * 32, acc);
                tmem_ld_wait();
                const int nb = n0 + g * 32;
                if (STORE_C) {
                    // dot = 4 popc(a&w) - 2 popc(a) - (2 popc(w) - K), acc = 128 popc(a&w)
                    int d[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) d[j] = (int)(acc[j] >> 5) - 2 * pa - ctl->T[g * 32 + j];
                    // Each thread parks its 32 integers (128 bytes of one output row) in shared
                    // memory; the warp then writes the 32 x 128-byte block with 16-byte stores in
                    // which 8 consecutive lanes cover one row: every store instruction writes four
                    // whole 128-byte lines.
                    const bool vec_ok = (ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && nb + 31 < N;
                    if (vec_ok) {
                        int (*blk)[36] = ctl->cstage[warp][g & 1];
                        const uint32_t row_smem = smem_u32(&blk[lane][0]);
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            sts128(row_smem + 16 * q, (uint32_t)d[4 * q], (uint32_t)d[4 * q + 1], (uint32_t)d[4 * q + 2], (uint32_t)d[4 * q + 3]);
                        __syncwarp();
                        const int rr = lane >> 3, qq = lane & 7;
                        const int mrow0 = m0 + warp * 32;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int row = 4 * i + rr;
                            const int4 v = *reinterpret_cast<const int4*>(&blk[row][4 * qq]);
                            if (mrow0 + row < M)
                                *reinterpret_cast<int4*>(C + (size_t)(mrow0 + row) * ldc + nb + 4 * qq) = v;
                        }
                        // the buffer is written again two blocks later: by then every lane has passed
                        // the __syncwarp of the next block, i.e. has finished reading this one
                    } else if (m < M) {
                        int32_t* dst = C + (size_t)m * ldc + nb;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + j < N) dst[j] = d[j];
                    }
                    if (SIGN_PACK) {
                        uint32_t wd = 0u;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int n = nb + j;
                            const bool bit = n < N && (d[j] >= __ldg(thr + (n < N ? n : 0)));
                            wd |= (uint32_t)bit << j;
                        }
                        words[g] = wd ^ ctl->flipw[g];
                    }
                } else {
                    // bit = (acc - 64 popc(a) - T[n] >= 0); the sign bits are shifted in from the
                    // top, element 31 first, so element j ends up in bit j, inverted.
                    const int cm = 64 * pa;
                    uint32_t wd = 0u;
#pragma unroll
                    for (int j = 31; j >= 0; --j) {
                        const int v = (int)acc[j] - cm - ctl->T[g * 32 + j];
                        wd = __funnelshift_l((uint32_t)v, wd, 1);
                    }
                    words[g] = ~wd ^ ctl->flipw[g];
                }
                if (SIGN_PACK) {
                    const int valid = N - nb;  // columns of this word that exist
                    if (valid < 32) words[g] = valid > 0 ? (words[g] & ((1u << valid) - 1u)) : 0u;
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
            if (SIGN_PACK && m < M) {
                const int nw = words_for(N), w0 = n0 >> 5;
                uint32_t* dst = out_bits + (size_t)m * ldob + w0;
                if (w0 + BN / 32 <= nw) {   // 6 words; rows are 16-byte aligned, n0/32 is a multiple of 6
#pragma unroll
                    for (int q = 0; q < BN / 64; ++q)
                        reinterpret_cast<uint2*>(dst)[q] = make_uint2(words[2 * q], words[2 * q + 1]);
                } else {
#pragma unroll
                    for (int g = 0; g < BN / 32; ++g)
                        if (w0 + g < nw) dst[g] = words[g];
                }
            }
        }
    }

    // ---------------- teardown: every thread arrives here, also after an aborted wait
    tc_fence_before_sync();
    __syncthreads();
    if (warp == MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, TMEM_COLS);
    }
    if (threadIdx.x == 0 && ctl->abort) atomicExch(status, 1);
}

int g_sm_count = 0;

template <bool STORE_C, bool SIGN_PACK>
int launch_variant(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N, int K,
                   int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                   uint32_t* out_bits, int ldob, cudaStream_t st) {
    auto kern = xnor_tc_kernel<STORE_C, SIGN_PACK>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return BNN_ERR_CUDA;
        configured = true;
    }
    if (g_sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return BNN_ERR_CUDA;
    }
    const int tiles = ceil_div(M, BM) * ceil_div(N, BN);
    const int grid = tiles < g_sm_count ? tiles : g_sm_count;
    int* status = tc_status_ptr();
    if (!status) return BNN_ERR_CUDA;
    // tensor maps of the two packed operands: [rows][ceil(K/32) words] with the caller's pitch;
    // boxes of 16 words x (128 | 192) rows; whatever lies outside the tensor reads as zero
    CUtensorMap mapA, mapB;
    if (!encode_packed_map(&mapA, Ap, ldap, M, K, BM) || !encode_packed_map(&mapB, Wp, ldwp, N, K, BN))
        return BNN_ERR_CUDA;
    kern<<<grid, THREADS, SMEM_BYTES, st>>>(mapA, mapB, M, N, K, C, ldc, thr, flip, out_bits, ldob, status);
    return launch_status();
}

}  // namespace

// The driver's tensor-map encoder is looked up through the runtime, so that the library does not
// link against the driver library (which only exists on machines with a GPU).
bool encode_packed_map(CUtensorMap* map, const uint32_t* base, int ld, int rows, int K, int box_rows) {
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess || !fn)
            return false;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    const cuuint64_t dims[2] = {(cuuint64_t)words_for(K), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(uint32_t)};   // bytes between rows (multiple of 16)
    const cuuint32_t box[2] = {16u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int launch_xnor_tc(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                   int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                   uint32_t* out_bits, int ldob, cudaStream_t st) {
    const bool sp = out_bits != nullptr;
    if (C && sp) return launch_variant<true, true>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, st);
    if (C) return launch_variant<true, false>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, st);
    return launch_variant<false, true>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, st);
}

// Device address of the status word (one per device would need a table; one device is used).
int* tc_status_ptr() {
    static int* ptr = nullptr;
    if (!ptr && cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_tc_status) != cudaSuccess) ptr = nullptr;
    return ptr;
}

int read_tc_status(int* out) {
    return cudaMemcpyFromSymbol(out, g_tc_status, sizeof(int)) == cudaSuccess ? BNN_OK : BNN_ERR_CUDA;
}

}  // namespace bnn
