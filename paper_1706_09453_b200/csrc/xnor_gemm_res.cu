// Fused binary hidden layer on the tensor cores with the layer's weights RESIDENT in shared
// memory:  bits[m][n] = Sign(scale[n] * sum_k a[m][k] * w[n][k] + shift[n]),  a, w in {-1, +1}.
//
// Same contraction as xnor_gemm_tc.cu / xnor_gemm_img.cu (every +-1 widened to a 4-bit e2m1
// nibble, kind::mxf4, unit block scales, exact fp32 sums).  Measured on B200, streaming the
// widened weights from L2 for every tile of frames holds the tensor pipe at about a third of
// its rate (24 KB per 384 MMA clocks and SM is more than L2 delivers to 148 SMs at once).  So
// here a CTA owns ONE tile of units for the whole launch: it loads that tile's slice of the
// prepared weight image (all of K, up to 192 KB) into shared memory once and then walks over
// frame tiles, for which only the packed frame bits (4 KB per stage) cross L2.  CTA c works on
// unit tile c mod n_tiles and shares that tile's frame tiles with the other CTAs of the same
// residue.
//
// The image is the one xnor_gemm_img.cu describes: a tile of BN units is, per stage of 256
// positions of K, eight contiguous runs of BN x 16 bytes, copied to offsets c * BN * 16 of the
// stage's block (K-major core matrices).  BN = 192 while K <= 2048 and BN = 128 while
// K <= 3072 keep the slice within 192 KB; other shapes are left to the streaming kernel.
//
// Roles in a CTA of 15 warps (one CTA per SM):
//   warp 13      one thread issues the bulk copies of the weight slice (once) and the 2-D TMA
//                tile loads of the packed frame rows (64 bytes per row = two stages) into a
//                staging ring (64-byte swizzle, no multicast)
//   warps 5-12   two teams of four warps widen the frame rows, thread = one row, 32 bytes ->
//                128 bytes per stage, into tensor memory (the MMA reads its A operand from
//                there); the teams take alternate stages
//   warps 4, 14  issue the MMAs (4 per stage, K = 64 each) and the commits, one lane each; the two
//                warps take a tile's stages in turn and accumulate into the same accumulator
//   warps 0-3    epilogue: accumulator -> threshold -> repacked bits; two accumulators in
//                tensor memory, so it overlaps the next tile's MMAs
// Every wait is bounded; a wait that runs out sets the CTA's abort flag, all roles fall
// through to the common teardown and the device status word is set.
//
// A run of consecutive hidden layers of the same shape (the forward loop of Algorithm 2 over
// l = 2 .. L-1) is ONE launch: the roles above loop over the layers.  Between layers nothing is
// torn down; a CTA keeps its unit tile index and its frame tiles.  What a layer needs from the
// one before it is tracked per frame tile: a counter in global memory that every CTA increments
// (release) once its bits of that frame tile and layer are stored, and the thread that loads a
// frame tile waits (acquire, bounded) until all unit tiles have arrived.  The weight slice of the
// next layer replaces the current one stage by stage, each stage as soon as the last frame tile's
// MMAs of that stage have completed, so the reload overlaps the tail of the layer.  (Measured on
// B200: five launches of one layer each spent 6 us per layer between the end of one kernel and
// the first MMA of the next.)
#include "bnn_common.cuh"
#include "tcgen05.cuh"
#include "xnor_widen.cuh"

namespace bnn {

namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 256;                                   // positions of K per stage
constexpr int ROW_BYTES = BK / 2;                         // widened bytes per row and stage (128)
constexpr int B_REGION = 192 * 1024;                      // shared memory that holds the weight slice
constexpr int EPI_WARPS = 4, MMA_WARP = 4, PROD_WARP0 = 5, A_WARPS = BM / 32, TEAMS = 2;
constexpr int TMA_WARP = PROD_WARP0 + TEAMS * A_WARPS;
constexpr int MMA_WARP2 = TMA_WARP + 1;                   // the second issuing warp
constexpr int THREADS = (MMA_WARP2 + 1) * 32;             // 480
constexpr int GROUPS = 4;                                 // staging ring of the packed frame rows: groups of two stages
constexpr int GROUP_BYTES = BM * 64;
constexpr uint32_t A_COLS = ROW_BYTES / 4;                // 32-bit columns per A stage
constexpr uint32_t SF_COLS = 32, TMEM_COLS = 512;
constexpr int MAX_NKS = 16;

template <int BN> struct Cfg {
    static constexpr int B_BYTES = BN * ROW_BYTES;                 // one stage of the unit operand
    static constexpr int NKS = B_REGION / B_BYTES;                 // stages that fit: 8 (BN 192), 12 (BN 128)
    static constexpr int A_STAGES = (int)((TMEM_COLS - SF_COLS - 2 * BN) / A_COLS) > 6 ? 6 : (int)((TMEM_COLS - SF_COLS - 2 * BN) / A_COLS);
    static constexpr uint32_t TMEM_A_COL = 2 * BN;                 // A stages start after the two accumulators
    static constexpr uint32_t TMEM_SF_COL = TMEM_A_COL + A_STAGES * A_COLS;
    static_assert(NKS <= MAX_NKS && A_STAGES >= 3 && TMEM_SF_COL + SF_COLS <= TMEM_COLS, "tile configuration");
};

constexpr int MAX_STACK = kXnorStackMax;

struct Control {
    int T[192];              // per unit: threshold + kMagicBits
    uint32_t flipw[8];
    uint64_t full_a[6], empty_a[6], full_b[MAX_NKS], b_free[MAX_NKS], acc_full[2], acc_empty[2];
    uint64_t group_full[GROUPS], group_empty[GROUPS];
    uint64_t started[2];
    uint32_t tmem_base;
    WaitState wait;
};
constexpr int SMEM_BYTES = B_REGION + GROUPS * GROUP_BYTES + (int)sizeof(Control) + 1024;
static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");

// 1-D bulk asynchronous copy global -> shared; completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Frame tiles of this CTA: mt = first, first + step, ... < m_tiles.
struct Share {
    int first, step, count;
};
__device__ __forceinline__ Share my_share(int m_tiles, int n_tiles) {
    const int nt = (int)blockIdx.x % n_tiles, r = (int)blockIdx.x / n_tiles;
    const int peers = ((int)gridDim.x - 1 - nt) / n_tiles + 1;    // CTAs that work on unit tile nt
    Share s;
    s.first = r; s.step = peers;
    s.count = r < m_tiles ? (m_tiles - 1 - r) / peers + 1 : 0;
    return s;
}

struct ProducerArgs {
    uint32_t smem_stage;  // shared-space address of the staging ring
    uint32_t tmem_a;      // tensor-memory address of A stage 0 (lane 0)
    Control* ctl;
    volatile int* abort_flag;
    int my_tiles, nks, kw;
    uint32_t tmask;
    int lane;
    int zo;               // the frame operand's bits stand for (0,1) instead of (-1,+1)
};

// Producer of the frame operand: thread = row `r` of every tile of this CTA; team `team`
// takes the stages it = team, team + TEAMS, ... of the CTA's sequence of (tile, stage) pairs.
template <int A_STAGES>
__device__ __forceinline__ void produce_a(const ProducerArgs& a, int r, int team) {
    Control* ctl = a.ctl;
    const int total = a.my_tiles * a.nks;
    const int ng = ceil_div(a.nks, 2);
    // TMEM lane of this thread's frame row: a warp may only touch lanes 32*(warp%4)..+31
    const uint32_t tdst0 = a.tmem_a + ((uint32_t)(r & ~31) << 16);
    // this row inside a staging group: 64 bytes per row, 16-byte chunk c stored at c ^ ((r/2)%4)
    const uint32_t stg0 = a.smem_stage + r * 64;
    const uint32_t sw = (uint32_t)(r >> 1) & 3u;
    const bool ragged = (a.kw % 8 != 0) || a.tmask != 0xFFFFFFFFu;   // last stage has positions >= K
    int ks = team, tl = 0;
    while (ks >= a.nks) { ks -= a.nks; ++tl; }
    for (int it = team; it < total; it += TEAMS) {
        const int gidx = tl * ng + (ks >> 1);          // staging group that holds this stage
        const int gslot = gidx % GROUPS;
        const uint32_t gi = (uint32_t)ks & 1u;         // stage inside its group of two
        if (!warp_wait(smem_u32(&ctl->group_full[gslot]), (uint32_t)((gidx / GROUPS) & 1), a.abort_flag, a.lane)) break;
        const uint32_t src = stg0 + gslot * GROUP_BYTES;
        const uint4 v0 = lds128u(src + (((2u * gi) ^ sw) << 4));
        const uint4 v1 = lds128u(src + (((2u * gi + 1u) ^ sw) << 4));
        const int s = it % A_STAGES;
        if (!warp_wait(smem_u32(&ctl->empty_a[s]), (uint32_t)(((it / A_STAGES) & 1) ^ 1), a.abort_flag, a.lane)) break;
        const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        // 32-bit column 4c + t of the stage = word t of chunk c: the byte order of the
        // K-major shared-memory layout of the other operand
        uint32_t wr[32];
        if (a.zo) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int g = 8 * ks + c;   // index of the word in the row
                const uint32_t valid = (!ragged || g < a.kw - 1) ? 0xFFFFFFFFu : (g == a.kw - 1 ? a.tmask : 0u);
                const uint4 o = widen01_masked(w[c], valid);
                wr[4 * c] = o.x; wr[4 * c + 1] = o.y; wr[4 * c + 2] = o.z; wr[4 * c + 3] = o.w;
            }
        } else if (ragged && ks == a.nks - 1) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int g = 8 * ks + c;   // index of the word in the row
                const uint32_t valid = g < a.kw - 1 ? 0xFFFFFFFFu : (g == a.kw - 1 ? a.tmask : 0u);
                const uint4 o = widen_masked(w[c], valid);
                wr[4 * c] = o.x; wr[4 * c + 1] = o.y; wr[4 * c + 2] = o.z; wr[4 * c + 3] = o.w;
            }
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint4 o = widen(w[c]);
                wr[4 * c] = o.x; wr[4 * c + 1] = o.y; wr[4 * c + 2] = o.z; wr[4 * c + 3] = o.w;
            }
        }
        tmem_st32(tdst0 + s * A_COLS, wr);
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (a.lane == 0) {
            mbar_arrive(smem_u32(&ctl->full_a[s]));
            // The staging slot is handed back only after the stores that consumed the loaded
            // words: a shared-memory load that has merely been issued does not hold back the
            // TMA write that refills the slot.  A group counts one arrival per warp and stage;
            // the last group of a row with an odd number of stages holds a single stage, whose
            // consumers arrive twice.
            mbar_arrive(smem_u32(&ctl->group_empty[gslot]));
            if (gi == 0 && ks == a.nks - 1) mbar_arrive(smem_u32(&ctl->group_empty[gslot]));
        }
        ks += TEAMS;
        while (ks >= a.nks) { ks -= a.nks; ++tl; }
    }
}

// One layer of the run: its prepared weight image, folded thresholds and output.
struct StackLayer {
    const uint8_t* img;
    const int32_t* thr;
    const uint32_t* flip;
    uint32_t* out_bits;
};
struct StackArgs {
    StackLayer layer[MAX_STACK];
    int n_layers;
    int M, N, K, ldob, zo;
    TcStatus status;
    int* progress;           // [n_layers - 1][frame tiles] arrival counters, zero at launch (unused for one layer)
};
struct StackMaps {
    CUtensorMap m[MAX_STACK];   // packed input of each layer
};

// Wait until `*p` has reached `target` (acquire at GPU scope); bounded like the mbarrier waits.
__device__ __forceinline__ bool wait_counter(const int* p, int target, volatile int* abort_flag) {
    const long long t0 = clock64(), limit = wait_limit_of(abort_flag);
#pragma unroll 1
    while (true) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        if (v >= target) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
        __nanosleep(64);
    }
}

template <int BN>
__global__ void __launch_bounds__(THREADS, 1)
xnor_res_kernel(const __grid_constant__ StackMaps maps, const __grid_constant__ StackArgs g) {
    using C = Cfg<BN>;
    const int M = g.M, N = g.N, K = g.K, ldob = g.ldob, zo = g.zo, L = g.n_layers;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control* ctl = reinterpret_cast<Control*>(smem + B_REGION + GROUPS * GROUP_BYTES);
    volatile int* abort_flag = &ctl->wait.abort;

    // The kernel that follows in the stream may be scheduled as soon as this one's CTAs leave
    // their SMs.  This kernel's own set-up and the copy of its weight slice need nothing the
    // kernel before it writes; it waits (pdl_wait, below) before it touches the frames.
    pdl_trigger();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kw = words_for(K);
    const int nks = ceil_div(K, BK);
    const int m_tiles = ceil_div(M, BM), n_tiles = ceil_div(N, BN);
    const Share share = my_share(m_tiles, n_tiles);
    const int nt = (int)blockIdx.x % n_tiles, n0 = nt * BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::A_STAGES; ++s) {
            mbar_init(smem_u32(&ctl->full_a[s]), A_WARPS);
            mbar_init(smem_u32(&ctl->empty_a[s]), 1);
        }
        for (int s = 0; s < MAX_NKS; ++s) {
            mbar_init(smem_u32(&ctl->full_b[s]), 1);   // the copying thread (+ bytes)
            mbar_init(smem_u32(&ctl->b_free[s]), 1);   // the MMA thread's commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl->acc_full[b]), 2);       // one commit of each issuing warp
            mbar_init(smem_u32(&ctl->started[b]), 1);
            mbar_init(smem_u32(&ctl->acc_empty[b]), EPI_WARPS);
        }
        for (int b = 0; b < GROUPS; ++b) {
            mbar_init(smem_u32(&ctl->group_full[b]), 1);              // the issuing thread (+ bytes)
            mbar_init(smem_u32(&ctl->group_empty[b]), 2 * A_WARPS);   // per stage of the group, every warp of its team
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
    if (warp < EPI_WARPS) {
        // Block scales of both operands: every byte 127, the ue8m0 code of 2^0.  The whole
        // region is filled, so the values do not depend on how the scales are laid out in it.
        uint32_t ones[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) ones[j] = 0x7F7F7F7Fu;
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + C::TMEM_SF_COL, ones);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (warp == TMA_WARP) {
        // ---------------- one thread: per layer the weight slice, then the staging ring of frame rows
        if (lane == 0 && share.count > 0) {
            const uint32_t stg = smem_u32(smem) + B_REGION;
            const int ng = ceil_div(nks, 2);
            const size_t run = (size_t)xnor_image_npad(N) * 16;   // bytes between chunks of the image
            int gc = 0;   // groups issued so far, over all layers: slot gc % GROUPS, < GROUPS ahead of its consumers
            int gl = 0, gt = 0, gi = 0;   // the next group to issue: layer, index of the frame tile, group inside the tile
            bool ok = true;
            auto issue_group = [&]() {
                const int mt = share.first + gt * share.step;
                if (gi == 0 && gl > 0) {
                    // the frame tile's bits of the layer before: every unit tile's CTA has stored them
                    ok = wait_counter(g.progress + (size_t)(gl - 1) * m_tiles + mt, n_tiles, abort_flag);
                    if (!ok) return;
                    asm volatile("fence.proxy.async;" ::: "memory");   // generic-proxy writes of other CTAs -> this thread's TMA reads
                }
                const int slot = gc % GROUPS;
                if (gc >= GROUPS) {
                    ok = mbar_wait_relaxed(smem_u32(&ctl->group_empty[slot]), (uint32_t)(((gc / GROUPS) - 1) & 1), abort_flag);
                    if (!ok) return;
                }
                const uint32_t bar = smem_u32(&ctl->group_full[slot]);
                mbar_arrive_expect_tx(bar, GROUP_BYTES);
                tma_load_2d(stg + slot * GROUP_BYTES, &maps.m[gl], gi * 16, mt * BM, bar);
                ++gc;
                if (++gi == ng) { gi = 0; if (++gt == share.count) { gt = 0; ++gl; } }
            };
            for (int l = 0; l < L && ok; ++l) {
                // A later layer's first frame rows go into the staging ring before its weights: the
                // producers widen them into tensor memory while the weight stages arrive.
                if (l > 0)
                    for (int i = 0; i < GROUPS && gl == l && ok; ++i) issue_group();
                if (!ok) break;
                // The weights do not depend on the kernel before this one in the stream (layer 0) nor on
                // other CTAs (later layers).  A stage of the previous layer's slice is overwritten once
                // the MMAs of this CTA's last frame tile that read it have completed.
                const uint8_t* src = g.layer[l].img + (size_t)n0 * 16;
                for (int ks = 0; ks < nks && ok; ++ks) {
                    if (l > 0) ok = mbar_wait(smem_u32(&ctl->b_free[ks]), (uint32_t)((l - 1) & 1), abort_flag);
                    if (!ok) break;
                    const uint32_t bar = smem_u32(&ctl->full_b[ks]);
                    mbar_arrive_expect_tx(bar, C::B_BYTES);
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        bulk_g2s(smem_u32(smem + ks * C::B_BYTES + c * (BN * 16)), src + (size_t)(ks * 8 + c) * run, BN * 16, bar);
                }
                if (!ok) break;
                // the frames of layer 0 are the previous kernel's output: wait until that kernel has
                // completed and its writes are visible (returns at once when there is no such dependency)
                if (l == 0) pdl_wait();
                while (gl == l && ok) issue_group();
            }
        }
        __syncwarp();
    } else if (warp >= PROD_WARP0 && warp < TMA_WARP) {
        // the layers follow one another in the producers' sequence of (tile, stage) pairs
        ProducerArgs pa{smem_u32(smem) + B_REGION, tmem + C::TMEM_A_COL, ctl, abort_flag, L * share.count, nks, kw, tail_mask(K), lane, zo};
        produce_a<C::A_STAGES>(pa, (warp & 3) * 32 + lane, (warp - PROD_WARP0) / A_WARPS);
    } else if (warp == MMA_WARP || warp == MMA_WARP2) {
        // ---------------- MMA issue: two warps, one issuing lane each; the warps stay converged and the
        // MMAs and commits are predicated on lane 0.  A tile's stages go to the two warps in turn, and both
        // accumulate into the tile's accumulator: the sums are exact integers (|sum| <= K < 2^24), so the
        // order of the accumulations does not matter.  Only the stage that overwrites the accumulator has
        // to come first: warp 0 commits its first MMA of a tile to `started`, and warp 1 waits for that
        // before its first MMA of the tile.  (Measured on B200: what an issuing thread does between MMAs
        // -- polls, commits, bookkeeping -- is time the tensor pipe idles; with two issuers one thread's
        // waits overlap the other's MMAs.  2 % off the WSJ-scale step against one issuer that takes the
        // stages in pairs; two issuers taking pairs, and a deeper ring of narrower tiles, gained less.)
        {
            const int w = warp == MMA_WARP ? 0 : 1;
            const uint32_t issue = lane == 0;
            constexpr uint32_t idesc = instr_desc_mxf4(BM, BN);
            const uint32_t sfa = tmem + C::TMEM_SF_COL, sfb = tmem + C::TMEM_SF_COL + SF_COLS / 2;
            const uint64_t desc0 = smem_desc_kmajor(smem_u32(smem), BN * 16, 128);
            constexpr uint32_t kStepJ = (2 * BN * 16) >> 4, kStepS = C::B_BYTES >> 4;
            const uint32_t tmem_a = tmem + C::TMEM_A_COL;
            bool ok = true;
            int tl = 0;          // tiles so far, over all layers
            int it_base = 0;     // stages before this tile, over all layers
            for (int l = 0; l < L && ok; ++l) {
                const uint32_t pb = (uint32_t)(l & 1);   // a layer's weight stages arrive once and then stay
                for (int t = 0; t < share.count && ok; ++t, ++tl, it_base += nks) {
                    const bool first = t == 0;
                    const bool hand_over = t == share.count - 1 && l + 1 < L;   // the next layer's slice follows
                    const int b = tl & 1;
                    ok = mbar_wait(smem_u32(&ctl->acc_empty[b]), (uint32_t)(((tl >> 1) & 1) ^ 1), abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d = tmem + (uint32_t)(b * BN);
                    for (int ks = w; ks < nks; ks += 2) {
                        const int it = it_base + ks;             // this stage in the CTA's sequence: slot and parity of the A ring
                        const int sa = it % C::A_STAGES;
                        const uint32_t pa = (uint32_t)((it / C::A_STAGES) & 1);
                        ok = (!first || mbar_wait(smem_u32(&ctl->full_b[ks]), pb, abort_flag)) &&
                             mbar_wait(smem_u32(&ctl->full_a[sa]), pa, abort_flag) &&
                             (ks != 1 || mbar_wait(smem_u32(&ctl->started[b]), (uint32_t)((tl >> 1) & 1), abort_flag));
                        if (!ok) break;
                        tc_fence_after_sync();
                        // descriptor of stage ks, chunk pair 0; the address field (16-byte units) of the others is
                        // reached by plain additions: the whole region lies below 2^14 * 16 bytes
                        const uint64_t db = desc0 + (uint64_t)((uint32_t)ks * kStepS);
                        const uint32_t ta = tmem_a + sa * A_COLS;
#pragma unroll
                        for (int j = 0; j < BK / 64; ++j) {  // 64 positions of K = 32 bytes: 8 columns of A, two 16-byte chunks of B
                            mma_mxf4_ts_if(issue, d, ta + 8 * j, db + j * kStepJ, idesc, sfa, sfb, (ks | j) != 0);
                            if (j == 0 && ks == 0) mma_commit_if(issue, smem_u32(&ctl->started[b]));
                        }
                        mma_commit_if(issue, smem_u32(&ctl->empty_a[sa]));
                        if (hand_over) mma_commit_if(issue, smem_u32(&ctl->b_free[ks]));
                    }
                    if (ok) mma_commit_if(issue, smem_u32(&ctl->acc_full[b]));
                }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: 128 threads, thread = one frame (TMEM lane)
        const int row_in_tile = warp * 32 + lane;
        const float magic = __int_as_float(kMagicBits);
        bool ok = true;
        int tl = 0;              // tiles so far, over all layers
        for (int l = 0; l < L && ok; ++l) {
            // thresholds of this CTA's units for this layer (the unit tile never changes); the
            // barriers keep them apart from the previous layer's last readers
            const int32_t* __restrict__ thr = g.layer[l].thr;
            const uint32_t* __restrict__ flip = g.layer[l].flip;
            uint32_t* __restrict__ out_bits = g.layer[l].out_bits;
            if (l > 0) epi_bar_sync();
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
            for (int t = 0; t < share.count && ok; ++t, ++tl) {
                const int mt = share.first + t * share.step;
                const int m = mt * BM + row_in_tile;
                const int b = tl & 1;
                // all four epilogue warps take the same decision, so none is left at a barrier
                ok = epi_all(warp_wait_relaxed(smem_u32(&ctl->acc_full[b]), (uint32_t)((tl >> 1) & 1), abort_flag, lane));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * BN);
                const int nw = words_for(N), w0 = n0 >> 5;
                uint32_t* dst = out_bits + (size_t)(m < M ? m : 0) * ldob + w0;
                const bool whole = w0 + BN / 32 <= nw;   // rows are 16-byte aligned and BN/32 is even: 8-byte stores
#pragma unroll
                for (int gp = 0; gp < BN / 64; ++gp) {
                    uint32_t pair[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int gq = 2 * gp + h;
                        uint32_t acc[32];
                        tmem_ld32(taddr + gq * 32, acc);
                        tmem_ld_wait();
                        // The accumulator holds the integer dot product as a float; adding 1.5 * 2^23
                        // leaves that integer, offset by kMagicBits, in the bit pattern of the sum.
                        // bit = (dot - thr >= 0); the sign bits are shifted in from the top, element 31
                        // first, so element j ends up in bit j, inverted.
                        uint32_t wd = 0u;
#pragma unroll
                        for (int j = 31; j >= 0; --j)
                            wd = __funnelshift_l((uint32_t)(__float_as_int(__uint_as_float(acc[j]) + magic) - ctl->T[gq * 32 + j]), wd, 1);
                        wd = ~wd ^ ctl->flipw[gq];
                        const int valid = N - (n0 + gq * 32);  // columns of this word that exist
                        if (valid < 32) wd = valid > 0 ? (wd & ((1u << valid) - 1u)) : 0u;
                        pair[h] = wd;
                    }
                    if (m < M) {
                        if (whole) {
                            reinterpret_cast<uint2*>(dst)[gp] = make_uint2(pair[0], pair[1]);
                        } else {
                            if (w0 + 2 * gp < nw) dst[2 * gp] = pair[0];
                            if (w0 + 2 * gp + 1 < nw) dst[2 * gp + 1] = pair[1];
                        }
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[b]));
                if (l + 1 < L) {
                    // this CTA's share of frame tile mt is stored: tell the CTAs that read it in the next layer
                    __threadfence();
                    epi_bar_sync();
                    if (threadIdx.x == 0) {
                        asm volatile("fence.proxy.async;" ::: "memory");
                        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(g.progress + (size_t)l * m_tiles + mt) : "memory");
                    }
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
    if (threadIdx.x == 0 && ctl->wait.abort) atomicExch(g.status.word, 1);
}

template <int BN>
int launch_bn(const uint32_t* Ap, int ldap, const XnorStackLayer* layers, int n_layers, int M, int N, int K, int ldob,
              int zo, int* progress, bool chained, int sm_count, cudaStream_t st) {
    auto kern = xnor_res_kernel<BN>;
    if (!ensure_dynamic_smem(reinterpret_cast<const void*>(kern), SMEM_BYTES)) return BNN_ERR_CUDA;
    const long long tiles = (long long)ceil_div(M, BM) * ceil_div(N, BN);
    const int grid = tiles < sm_count ? (int)tiles : sm_count;
    StackArgs a{};
    StackMaps maps{};
    a.n_layers = n_layers; a.M = M; a.N = N; a.K = K; a.ldob = ldob; a.zo = zo;
    a.status = tc_status();
    a.progress = progress;
    if (!a.status.word) return BNN_ERR_CUDA;
    for (int l = 0; l < n_layers; ++l) {
        a.layer[l] = StackLayer{static_cast<const uint8_t*>(layers[l].image), layers[l].thr, layers[l].flip, layers[l].out_bits};
        // a layer reads what the layer before it wrote
        const uint32_t* in = l == 0 ? Ap : layers[l - 1].out_bits;
        if (!encode_packed_map(&maps.m[l], in, l == 0 ? ldap : ldob, M, K, BM)) return BNN_ERR_CUDA;
    }
    // Programmatic dependent launch only inside a forward pass: there the kernel before this one is a
    // layer's kernel and everything read before the wait (weights, thresholds) was complete before the
    // forward pass started.  A stand-alone call may follow the kernel that wrote its thresholds or its
    // weight image on the same stream, so it is launched the ordinary way.
    if (chained) {
        if (launch_pdl(kern, dim3(grid), dim3(THREADS), SMEM_BYTES, st, maps, a) != cudaSuccess) return BNN_ERR_CUDA;
    } else {
        kern<<<grid, THREADS, SMEM_BYTES, st>>>(maps, a);
    }
    return launch_status();
}

}  // namespace

// Units per tile for a layer of this shape, or 0 when the kernel does not apply: the slice of
// a tile must fit the shared-memory region, and every unit tile needs a CTA of its own.
static int tile_units(int N, int K, int sm_count) {
    const int nks = ceil_div(K, BK);
    const int bn = nks <= Cfg<192>::NKS ? 192 : (nks <= Cfg<128>::NKS ? 128 : 0);
    if (bn == 0 || ceil_div(N, bn) > sm_count) return 0;
    return bn;
}

static int sm_count_of_device() { return device_sm_count(); }

bool xnor_res_applicable(int N, int K) {
    const int sms = sm_count_of_device();
    return sms > 0 && tile_units(N, K, sms) != 0;
}

size_t xnor_stack_sync_bytes(int M, int n_layers) {
    return n_layers > 1 ? (size_t)(n_layers - 1) * ceil_div(M, BM) * sizeof(int) : 0;
}

int launch_xnor_stack(const uint32_t* Ap, int ldap, const XnorStackLayer* layers, int n_layers, int M, int N, int K,
                      int ldob, int zo, int* progress, bool chained, cudaStream_t st) {
    const int sms = sm_count_of_device();
    if (sms <= 0) return BNN_ERR_CUDA;
    if (n_layers < 1 || n_layers > kXnorStackMax || (n_layers > 1 && (N != K || !progress))) return BNN_ERR_UNSUPPORTED;
    const int bn = tile_units(N, K, sms);
    if (bn == 192) return launch_bn<192>(Ap, ldap, layers, n_layers, M, N, K, ldob, zo, progress, chained, sms, st);
    if (bn == 128) return launch_bn<128>(Ap, ldap, layers, n_layers, M, N, K, ldob, zo, progress, chained, sms, st);
    return BNN_ERR_UNSUPPORTED;
}

int launch_xnor_res(const uint32_t* Ap, int ldap, const void* image, int M, int N, int K,
                    const int32_t* thr, const uint32_t* flip, uint32_t* out_bits, int ldob, int zo, cudaStream_t st) {
    const XnorStackLayer one{image, thr, flip, out_bits};
    return launch_xnor_stack(Ap, ldap, &one, 1, M, N, K, ldob, zo, nullptr, false, st);
}

}  // namespace bnn
