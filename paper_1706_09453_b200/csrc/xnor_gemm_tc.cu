// XNOR GEMM on the 5th-generation tensor cores as a 4-bit floating-point contraction.
//
//   dot[m][n] = sum_k a[m][k] * w[n][k],  a, w in {-1, +1}  ( = K - 2 popc(a xor w) )
//
// The tensor cores have no 1-bit mode, so every bit is widened on the fly, in the SM, to the
// narrowest type they multiply: the 4-bit float e2m1, in which +1 is the nibble 0x2 and -1 the
// nibble 0xA (kind::mxf4; its per-32-element block scales are all set to 2^0).  The products are
// +-1 and the fp32 accumulator holds their integer sums exactly for K <= 2^22, so the result is
// the signed dot product itself: no popcount correction terms, no bias.  Padding (K rounded up
// to the stage size) is the nibble 0, i.e. +0.
//
// Widening costs 4 bits of shared memory per bit of input, half of what an 8-bit integer
// contraction needs, and the 4-bit MMA has twice its rate; both matter because this kernel
// is bound by the shared-memory pipe (stores of the widened operands + the tensor core's
// reads of them), not by HBM: the packed operands are tiny.
//
// K may be visited in any order as long as both operands use the same one.  The order here
// makes widening two instructions per 32-bit output word: output word t (0..3) of input word
// w holds, in nibble i, bit 4i + t of w:   ((w << (3 - t)) & 0x88888888) ^ 0xAAAAAAAA
// (sign bit = NOT the input bit, exponent field = 01).
//
// Roles in a CTA of 16 warps (persistent, one CTA per SM, tiles of 128 frames x 192 units):
//   warp 15      one thread issues 2-D TMA tile loads of the packed rows (64 bytes per row =
//                two stages) into a staging ring (64-byte swizzle, no multicast)
//   warps 5-8    widen the frame rows, thread = one row, 32 bytes -> 128 bytes per stage,
//                written to tensor memory (the MMA reads its A operand from there)
//   warps 9-14   widen the unit rows the same way into shared memory, two stages per iteration
//   warp 4       one thread issues the MMAs (4 per stage, K = 64 each) and the commits
//   warps 0-3    epilogue: accumulator -> Sign/threshold -> repacked bits (or int32 output);
//                two accumulators in tensor memory, so it overlaps the next tile's MMAs
// Every wait is bounded; a wait that runs out sets the CTA's abort flag, all roles fall
// through to the common teardown and the device status word is set.
#include "bnn_common.cuh"
#include "tcgen05.cuh"
#include "xnor_widen.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BM = 128, BN = 192;
constexpr int BK = 256;                                   // bits of K per stage = nibbles per widened row
constexpr int ROW_BYTES = BK / 2;                         // widened bytes per row and stage (128)
constexpr int B_BYTES = BN * ROW_BYTES, STAGE_BYTES = B_BYTES;   // only the unit operand lives in shared memory
constexpr int A_STAGES = 3, B_STAGES = 4;               // rings of the frame operand (tensor memory) and the unit operand
constexpr int EPI_WARPS = 4, MMA_WARP = 4, PROD_WARP0 = 5, A_WARPS = BM / 32, B_WARPS = BN / 32;
constexpr int PROD_WARPS = A_WARPS + B_WARPS;
constexpr int TMA_WARP = PROD_WARP0 + PROD_WARPS;
constexpr int THREADS = (TMA_WARP + 1) * 32;              // 512
constexpr int GROUPS = 4;                                 // staging ring: groups of two stages
constexpr int GA_BYTES = BM * 64, GB_BYTES = BN * 64, GROUP_BYTES = GA_BYTES + GB_BYTES;
constexpr uint32_t TMEM_A_COL = 2 * BN;                   // A stages start after the two accumulators
constexpr uint32_t A_COLS = ROW_BYTES / 4;                // 32-bit columns per A stage
constexpr uint32_t TMEM_SF_COL = TMEM_A_COL + A_STAGES * A_COLS, SF_COLS = 32;   // block scales: 16 columns per operand
constexpr uint32_t TMEM_COLS = 512;

// With int32 output each epilogue warp needs two staging blocks of 32 rows x 128 bytes.
template <bool STORE_C> struct Cfg {
    static constexpr int CSTAGE_BYTES = STORE_C ? EPI_WARPS * 2 * 32 * 36 * 4 : 0;
};

struct Control {
    int T[BN];               // per unit: threshold + kMagicBits (Sign epilogue only)
    uint32_t flipw[BN / 32];
    uint64_t full_a[A_STAGES], empty_a[A_STAGES], full_b[B_STAGES], empty_b[B_STAGES], acc_full[2], acc_empty[2];
    uint64_t group_full[GROUPS], group_empty[GROUPS];
    uint32_t tmem_base;
    WaitState wait;
};
template <bool STORE_C> constexpr int smem_bytes() {
    return B_STAGES * STAGE_BYTES + GROUPS * GROUP_BYTES + (int)sizeof(Control) + Cfg<STORE_C>::CSTAGE_BYTES + 1024;
}
static_assert(smem_bytes<false>() <= 232448 && smem_bytes<true>() <= 232448, "shared memory of one CTA");
static_assert(TMEM_SF_COL + SF_COLS <= TMEM_COLS, "tensor memory columns");
static_assert(sizeof(Control) % 16 == 0, "the int32 staging blocks follow the control block");

struct ProducerArgs {
    uint32_t smem;        // shared-space address of stage 0
    uint32_t tmem;        // base of the tensor-memory allocation
    Control* ctl;
    volatile int* abort_flag;
    int tiles, nks, kw;
    uint32_t tmask;
    int lane;
    int zo;               // the frame operand's bits stand for (0,1) instead of (-1,+1)
};

// The eight 16-byte chunks of one widened row and stage; `ks` is the stage's index in the row.
template <bool FRAMES>
__device__ __forceinline__ void widen_stage(const ProducerArgs& a, bool ragged, int ks, const uint4& v0, const uint4& v1, uint4 (&o)[8]) {
    const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
    if (FRAMES && a.zo) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int g = 8 * ks + c;   // index of the word in the row
            const uint32_t valid = (!ragged || g < a.kw - 1) ? 0xFFFFFFFFu : (g == a.kw - 1 ? a.tmask : 0u);
            o[c] = widen01_masked(w[c], valid);
        }
    } else if (ragged && ks == a.nks - 1) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int g = 8 * ks + c;   // index of the word in the row
            const uint32_t valid = g < a.kw - 1 ? 0xFFFFFFFFu : (g == a.kw - 1 ? a.tmask : 0u);
            o[c] = widen_masked(w[c], valid);
        }
    } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) o[c] = widen(w[c]);
    }
}

// Producer of the frame operand: thread = row `r` of every tile of this CTA, one stage per
// iteration, widened rows written to tensor memory (ring of A_STAGES stages).
__device__ __forceinline__ void produce_a(const ProducerArgs& a, int r) {
    Control* ctl = a.ctl;
    const int my_tiles = (a.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
    const int total = my_tiles * a.nks;
    // TMEM lane of this thread's frame row: a warp may only touch lanes 32*(warp%4)..+31
    const uint32_t tdst0 = a.tmem + ((uint32_t)(r & ~31) << 16) + TMEM_A_COL;
    // this row inside a staging group: 64 bytes per row, 16-byte chunk c stored at c ^ ((r/2)%4)
    const uint32_t stg0 = a.smem + B_STAGES * STAGE_BYTES + r * 64;
    const uint32_t sw = (uint32_t)(r >> 1) & 3u;
    const bool ragged = (a.kw % 8 != 0) || a.tmask != 0xFFFFFFFFu;   // last stage has positions >= K
    int gslot = 0;
    uint32_t gph = 0;
    int ks = 0, s = 0;
    uint32_t ph = 1;  // parity to wait for on `empty`: a fresh barrier passes parity 1
    for (int it = 0; it < total; ++it) {
        const uint32_t gi = (uint32_t)ks & 1u;   // stage inside its group of two
        if (gi == 0 && !warp_wait(smem_u32(&ctl->group_full[gslot]), gph, a.abort_flag, a.lane)) break;
        const uint32_t src = stg0 + gslot * GROUP_BYTES;
        const uint4 v0 = lds128u(src + (((2u * gi) ^ sw) << 4));
        const uint4 v1 = lds128u(src + (((2u * gi + 1u) ^ sw) << 4));
        if (!warp_wait(smem_u32(&ctl->empty_a[s]), ph, a.abort_flag, a.lane)) break;
        uint4 o[8];
        widen_stage<true>(a, ragged, ks, v0, v1, o);
        // 32-bit column 4c + t of the stage = word t of chunk c: the byte order of the
        // K-major shared-memory layout of the other operand
        uint32_t wr[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) { wr[4 * c] = o[c].x; wr[4 * c + 1] = o[c].y; wr[4 * c + 2] = o[c].z; wr[4 * c + 3] = o[c].w; }
        tmem_st32(tdst0 + s * A_COLS, wr);
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (a.lane == 0) mbar_arrive(smem_u32(&ctl->full_a[s]));
        // The staging slot is handed back only here, after the stores that consumed the loaded
        // words: a shared-memory load that has merely been issued does not hold back the TMA
        // write that refills the slot (that write belongs to the async proxy; only the data
        // dependency proves that the load has read its bytes).
        if (gi == 1 || ks == a.nks - 1) {
            if (a.lane == 0) mbar_arrive(smem_u32(&ctl->group_empty[gslot]));
            if (++gslot == GROUPS) { gslot = 0; gph ^= 1u; }
        }
        if (++s == A_STAGES) { s = 0; ph ^= 1u; }
        if (++ks == a.nks) ks = 0;
    }
}

// Producer of the unit operand: thread = row `r`, one staging group (two stages) per
// iteration, so the fixed costs of an iteration (group wait, proxy fence, warp barrier,
// release) are paid once per two stages; widened rows go to shared memory (ring of B_STAGES).
__device__ __forceinline__ void produce_b(const ProducerArgs& a, int r) {
    Control* ctl = a.ctl;
    const int my_tiles = (a.tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1;
    const int ng = ceil_div(a.nks, 2);
    const int total = my_tiles * ng;
    const uint32_t dst0 = a.smem + r * 16;
    const uint32_t stg0 = a.smem + B_STAGES * STAGE_BYTES + GA_BYTES + r * 64;
    const uint32_t sw = (uint32_t)(r >> 1) & 3u;
    const bool ragged = (a.kw % 8 != 0) || a.tmask != 0xFFFFFFFFu;
    int gslot = 0;
    uint32_t gph = 0;
    int kg = 0, s = 0;
    uint32_t ph = 1;
    for (int g = 0; g < total; ++g) {
        const bool two = 2 * kg + 1 < a.nks;   // the last group of a row may hold a single stage
        if (!warp_wait(smem_u32(&ctl->group_full[gslot]), gph, a.abort_flag, a.lane)) break;
        const uint32_t src = stg0 + gslot * GROUP_BYTES;
        const uint4 v0 = lds128u(src + ((0u ^ sw) << 4)), v1 = lds128u(src + ((1u ^ sw) << 4));
        const uint4 v2 = lds128u(src + ((2u ^ sw) << 4)), v3 = lds128u(src + ((3u ^ sw) << 4));
        const int s2 = s + 1 == B_STAGES ? 0 : s + 1;
        const uint32_t ph2 = s + 1 == B_STAGES ? ph ^ 1u : ph;
        if (!warp_wait(smem_u32(&ctl->empty_b[s]), ph, a.abort_flag, a.lane)) break;
        uint4 o[8];
        widen_stage<false>(a, ragged, 2 * kg, v0, v1, o);
#pragma unroll
        for (int c = 0; c < 8; ++c) sts128(dst0 + s * STAGE_BYTES + c * (BN * 16), o[c].x, o[c].y, o[c].z, o[c].w);
        if (two) {
            if (!warp_wait(smem_u32(&ctl->empty_b[s2]), ph2, a.abort_flag, a.lane)) break;
            widen_stage<false>(a, ragged, 2 * kg + 1, v2, v3, o);
#pragma unroll
            for (int c = 0; c < 8; ++c) sts128(dst0 + s2 * STAGE_BYTES + c * (BN * 16), o[c].x, o[c].y, o[c].z, o[c].w);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (a.lane == 0) {
            mbar_arrive(smem_u32(&ctl->full_b[s]));
            if (two) mbar_arrive(smem_u32(&ctl->full_b[s2]));
            mbar_arrive(smem_u32(&ctl->group_empty[gslot]));   // after the stores that consumed the loaded words (see produce_a)
        }
        if (++gslot == GROUPS) { gslot = 0; gph ^= 1u; }
        if (two) { s = s2; ph = ph2; }
        if (++s == B_STAGES) { s = 0; ph ^= 1u; }
        if (++kg == ng) kg = 0;
    }
}

template <bool STORE_C, bool SIGN_PACK>
__global__ void __launch_bounds__(THREADS, 1)
xnor_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                int M, int N, int K, int32_t* __restrict__ C, int ldc,
                const int32_t* __restrict__ thr, const uint32_t* __restrict__ flip,
                uint32_t* __restrict__ out_bits, int ldob, int zo, TcStatus status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(smem + B_STAGES * STAGE_BYTES + GROUPS * GROUP_BYTES);
    int (*cstage)[2][32][36] = reinterpret_cast<int (*)[2][32][36]>(reinterpret_cast<uint8_t*>(ctl) + sizeof(Control));
    volatile int* abort_flag = &ctl->wait.abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kw = words_for(K);
    const int nks = ceil_div(K, BK);
    const int m_tiles = ceil_div(M, BM), n_tiles = ceil_div(N, BN);
    const int tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < A_STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full_a[s]), A_WARPS);
            mbar_init(smem_u32(&ctl->empty_a[s]), 1);
        }
        for (int s = 0; s < B_STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full_b[s]), B_WARPS);
            mbar_init(smem_u32(&ctl->empty_b[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), EPI_WARPS);
        }
        for (int b = 0; b < GROUPS; ++b) {
            mbar_init(smem_u32(&ctl->group_full[b]), 1);            // the issuing thread (+ bytes)
            mbar_init(smem_u32(&ctl->group_empty[b]), PROD_WARPS);  // every producer warp has read it
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
    if (warp < EPI_WARPS) {
        // Block scales of both operands: every byte 127, the ue8m0 code of 2^0.  The whole
        // region is filled, so the values do not depend on how the scales are laid out in it.
        uint32_t ones[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) ones[j] = 0x7F7F7F7Fu;
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + TMEM_SF_COL, ones);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (warp >= PROD_WARP0) {
        ProducerArgs pa{smem_u32(smem), tmem, ctl, abort_flag, tiles, nks, kw, tail_mask(K), lane, zo};
        if (warp == TMA_WARP) {
            // ---------------- one thread feeds the staging ring, a group of two stages at a time
            if (lane == 0) {
                const uint32_t stg = smem_u32(smem) + B_STAGES * STAGE_BYTES;
                const int ng = ceil_div(nks, 2);
                int gc = 0;
                bool ok = true;
                for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                    const int n0 = (tile % n_tiles) * BN, m0 = (tile / n_tiles) * BM;   // unit tiles vary fastest
                    for (int g = 0; g < ng; ++g, ++gc) {
                        const int slot = gc % GROUPS;
                        if (gc >= GROUPS) {
                            ok = mbar_wait_relaxed(smem_u32(&ctl->group_empty[slot]), (uint32_t)(((gc / GROUPS) - 1) & 1), abort_flag);
                            if (!ok) break;
                        }
                        const uint32_t bar = smem_u32(&ctl->group_full[slot]);
                        mbar_arrive_expect_tx(bar, GROUP_BYTES);
                        tma_load_2d(stg + slot * GROUP_BYTES, &mapA, g * 16, m0, bar);
                        tma_load_2d(stg + slot * GROUP_BYTES + GA_BYTES, &mapB, g * 16, n0, bar);
                    }
                }
            }
            __syncwarp();
        } else if (warp < PROD_WARP0 + A_WARPS) {
            produce_a(pa, (warp & 3) * 32 + lane);
        } else {
            produce_b(pa, (warp - PROD_WARP0 - A_WARPS) * 32 + lane);
        }
    } else if (warp == MMA_WARP) {
        // ---------------- MMA issue: one thread.  Two stages per iteration: whatever this thread
        // does between two MMAs (polls, commits, bookkeeping) is time the tensor pipe idles, so
        // the waits of two stages are taken together and their eight MMAs issued back to back.
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_mxf4(BM, BN);
            const uint32_t sfa = tmem + TMEM_SF_COL, sfb = tmem + TMEM_SF_COL + SF_COLS / 2;
            const uint32_t smem0 = smem_u32(smem);
            int sa = 0, sb = 0;        // ring slots and the parities their `full` barriers show next
            uint32_t pa = 0, pb = 0;
            int tl = 0;
            bool ok = true;
            auto issue = [&](uint32_t d, int slot_a, int slot_b, bool first) {
                const uint32_t b0 = smem0 + slot_b * STAGE_BYTES;
                const uint32_t ta = tmem + TMEM_A_COL + slot_a * A_COLS;
#pragma unroll
                for (int j = 0; j < BK / 64; ++j) {   // 64 positions of K = 32 bytes: 8 columns of A, two 16-byte chunks of B
                    const uint64_t db = smem_desc_kmajor(b0 + 2 * j * (BN * 16), BN * 16, 128);
                    mma_mxf4_ts(d, ta + 8 * j, db, idesc, sfa, sfb, !(first && j == 0));
                }
                mma_commit(smem_u32(&ctl->empty_a[slot_a]));
                mma_commit(smem_u32(&ctl->empty_b[slot_b]));
            };
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
                const int b = tl & 1;
                ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), (uint32_t)(((tl >> 1) & 1) ^ 1), abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d = tmem + (uint32_t)(b * BN);
                int ks = 0;
                for (; ks + 1 < nks; ks += 2) {
                    const int sa2 = sa + 1 == A_STAGES ? 0 : sa + 1, sb2 = sb + 1 == B_STAGES ? 0 : sb + 1;
                    const uint32_t pa2 = sa + 1 == A_STAGES ? pa ^ 1u : pa, pb2 = sb + 1 == B_STAGES ? pb ^ 1u : pb;
                    ok = mbar_wait(smem_u32(&ctl->full_b[sb]), pb, abort_flag) && mbar_wait(smem_u32(&ctl->full_b[sb2]), pb2, abort_flag) &&
                         mbar_wait(smem_u32(&ctl->full_a[sa]), pa, abort_flag) && mbar_wait(smem_u32(&ctl->full_a[sa2]), pa2, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue(d, sa, sb, ks == 0);
                    issue(d, sa2, sb2, false);
                    sa = sa2; pa = pa2; sb = sb2; pb = pb2;
                    if (++sa == A_STAGES) { sa = 0; pa ^= 1u; }
                    if (++sb == B_STAGES) { sb = 0; pb ^= 1u; }
                }
                if (ok && ks < nks) {   // odd number of stages: the last one alone
                    ok = mbar_wait(smem_u32(&ctl->full_b[sb]), pb, abort_flag) && mbar_wait(smem_u32(&ctl->full_a[sa]), pa, abort_flag);
                    if (ok) {
                        tc_fence_after_sync();
                        issue(d, sa, sb, ks == 0);
                        if (++sa == A_STAGES) { sa = 0; pa ^= 1u; }
                        if (++sb == B_STAGES) { sb = 0; pb ^= 1u; }
                    }
                }
                if (ok) mma_commit(smem_u32(&ctl->acc_full[b]));
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: 128 threads, thread = one frame (TMEM lane)
        const int row_in_tile = warp * 32 + lane;
        const float magic = __int_as_float(kMagicBits);
        int tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int n0 = (tile % n_tiles) * BN, m0 = (tile / n_tiles) * BM;   // unit tiles vary fastest
            const int m = m0 + row_in_tile;
            if (SIGN_PACK) {
                epi_bar_sync();  // previous tile's readers of T are done
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int nl = row_in_tile + h * 128, n = n0 + nl;
                    if (nl < BN) ctl->T[nl] = kMagicBits + (n < N ? thr[n] : 0);
                }
                if (row_in_tile < BN / 32) {
                    const int wi = (n0 >> 5) + row_in_tile;
                    ctl->flipw[row_in_tile] = wi < words_for(N) ? flip[wi] : 0u;
                }
                epi_bar_sync();
            }
            const int b = tl & 1;
            // all four epilogue warps take the same decision, so none is left at a barrier
            ok = epi_all(warp_wait_relaxed(smem_u32(&ctl->acc_full[b]), (uint32_t)((tl >> 1) & 1), abort_flag, lane));
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
                // The accumulator holds the integer dot product as a float; adding 1.5 * 2^23
                // leaves that integer, offset by kMagicBits, in the bit pattern of the sum.
                int q[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) q[j] = __float_as_int(__uint_as_float(acc[j]) + magic);
                if (STORE_C) {
                    // Each thread parks its 32 integers (128 bytes of one output row) in shared
                    // memory; the warp then writes the 32 x 128-byte block with 16-byte stores in
                    // which 8 consecutive lanes cover one row: every store instruction writes four
                    // whole 128-byte lines.
                    const bool vec_ok = (ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && nb + 31 < N;
                    if (vec_ok) {
                        int (*blk)[36] = cstage[warp][g & 1];
                        const uint32_t row_smem = smem_u32(&blk[lane][0]);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            sts128(row_smem + 16 * i, (uint32_t)(q[4 * i] - kMagicBits), (uint32_t)(q[4 * i + 1] - kMagicBits),
                                   (uint32_t)(q[4 * i + 2] - kMagicBits), (uint32_t)(q[4 * i + 3] - kMagicBits));
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
                            if (nb + j < N) dst[j] = q[j] - kMagicBits;
                    }
                }
                if (SIGN_PACK) {
                    // bit = (dot - thr >= 0); the sign bits are shifted in from the top, element 31
                    // first, so element j ends up in bit j, inverted.
                    uint32_t wd = 0u;
#pragma unroll
                    for (int j = 31; j >= 0; --j)
                        wd = __funnelshift_l((uint32_t)(q[j] - ctl->T[g * 32 + j]), wd, 1);
                    words[g] = ~wd ^ ctl->flipw[g];
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
                    for (int i = 0; i < BN / 64; ++i)
                        reinterpret_cast<uint2*>(dst)[i] = make_uint2(words[2 * i], words[2 * i + 1]);
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
    if (threadIdx.x == 0 && ctl->wait.abort) atomicExch(status.word, 1);
}

template <bool STORE_C, bool SIGN_PACK>
int launch_variant(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N, int K,
                   int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                   uint32_t* out_bits, int ldob, int zo, cudaStream_t st) {
    auto kern = xnor_tc_kernel<STORE_C, SIGN_PACK>;
    constexpr int SMEM = smem_bytes<STORE_C>();
    const int sm_count = device_sm_count();
    if (sm_count <= 0 || !ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SMEM)) return BNN_ERR_CUDA;
    const int tiles = ceil_div(M, BM) * ceil_div(N, BN);
    const int grid = tiles < sm_count ? tiles : sm_count;
    const TcStatus status = tc_status();
    if (!status.word) return BNN_ERR_CUDA;
    // tensor maps of the two packed operands: [rows][ceil(K/32) words] with the caller's pitch;
    // boxes of 16 words x (128 | 192) rows; whatever lies outside the tensor reads as zero
    CUtensorMap mapA, mapB;
    if (!encode_packed_map(&mapA, Ap, ldap, M, K, BM) || !encode_packed_map(&mapB, Wp, ldwp, N, K, BN))
        return BNN_ERR_CUDA;
    kern<<<grid, THREADS, SMEM, st>>>(mapA, mapB, M, N, K, C, ldc, thr, flip, out_bits, ldob, zo, status);
    return launch_status();
}

}  // namespace

int launch_xnor_tc(const uint32_t* Ap, int ldap, const uint32_t* Wp, int ldwp, int M, int N,
                   int K, int32_t* C, int ldc, const int32_t* thr, const uint32_t* flip,
                   uint32_t* out_bits, int ldob, int zo, cudaStream_t st) {
    const bool sp = out_bits != nullptr;
    if (C && sp) return launch_variant<true, true>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, zo, st);
    if (C) return launch_variant<true, false>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, zo, st);
    return launch_variant<false, true>(Ap, ldap, Wp, ldwp, M, N, K, C, ldc, thr, flip, out_bits, ldob, zo, st);
}

}  // namespace bnn
