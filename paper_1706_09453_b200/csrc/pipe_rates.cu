// Micro-benchmarks of the execution pipes that bound the forward pass: the integer and FP32
// pipes (popc, lop3, iadd, fadd/ffma), the tensor pipe in the kinds the kernels use
// (kind::mxf4 on 4-bit operands, kind::f16), and the L2 read path.  Measurement support: the
// paper has no counterpart.  Each entry performs ONE launch of a fixed amount of work on the
// caller's stream and reports that amount; the caller times the launch with CUDA events.
#include "bnn_common.cuh"
#include "tcgen05.cuh"

namespace bnn {
namespace {

using namespace tc;

constexpr int ALU_THREADS = 256, ALU_BLOCKS_PER_SM = 8, CHAINS = 8, ALU_UNROLL = 32;

// 8 independent dependency chains per thread, ALU_UNROLL instructions of the chosen kind per
// chain and loop trip; the results are stored so that nothing is dead.
template <int KIND>
__global__ void __launch_bounds__(ALU_THREADS)
alu_rate_kernel(int trips, uint32_t* __restrict__ sink) {
    uint32_t a[CHAINS];
    float f[CHAINS];
    const uint32_t b = 0x9E3779B9u * (threadIdx.x + 1), c = 0x85EBCA6Bu ^ blockIdx.x;
    const float fb = 1.0f + 1e-7f * threadIdx.x, fc = 1e-9f * blockIdx.x;
#pragma unroll
    for (int j = 0; j < CHAINS; ++j) { a[j] = b + j; f[j] = fb + j; }
    for (int t = 0; t < trips; ++t) {
#pragma unroll
        for (int u = 0; u < ALU_UNROLL; ++u) {
#pragma unroll
            for (int j = 0; j < CHAINS; ++j) {
                if (KIND == BNN_RATE_POPC) asm volatile("popc.b32 %0, %0;" : "+r"(a[j]));
                if (KIND == BNN_RATE_LOP3) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(a[j]) : "r"(b), "r"(c));
                if (KIND == BNN_RATE_IADD) asm volatile("add.u32 %0, %0, %1;" : "+r"(a[j]) : "r"(b));
                if (KIND == BNN_RATE_FADD) asm volatile("add.rn.f32 %0, %0, %1;" : "+f"(f[j]) : "f"(fc));
                if (KIND == BNN_RATE_FFMA) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[j]) : "f"(fb), "f"(fc));
            }
        }
    }
    uint32_t r = 0;
#pragma unroll
    for (int j = 0; j < CHAINS; ++j) r ^= a[j] ^ __float_as_uint(f[j]);
    sink[(size_t)blockIdx.x * ALU_THREADS + threadIdx.x] = r;
}

// Every SM reads the same `bytes` (a multiple of 16 KB that fits L2) `trips` times.
__global__ void __launch_bounds__(512)
l2_read_kernel(const uint4* __restrict__ src, size_t vecs, int trips, uint32_t* __restrict__ sink) {
    uint32_t r = 0;
    for (int t = 0; t < trips; ++t) {
        // start every CTA at a different offset so that the SMs do not read the same lines at once
        const size_t off = ((size_t)blockIdx.x * 7919u + (size_t)t * 104729u) * 512u;
        for (size_t i = threadIdx.x; i < vecs; i += 512) {
            const uint4 v = __ldcg(src + ((i + off) & (vecs - 1)));   // vecs is a power of two
            r ^= v.x ^ v.y ^ v.z ^ v.w;
        }
    }
    sink[(size_t)blockIdx.x * 512 + threadIdx.x] = r;
}

// One CTA per SM; one thread issues `n_mma` MMAs of 128 x N x (K of the kind) on operands that
// sit in shared memory (whatever bytes are there: the rate does not depend on the values),
// with a commit and a bounded wait every 64 MMAs.  MXF4: kind::mxf4 with unit block scales;
// A_TMEM: A operand read from tensor memory instead of shared memory.
constexpr int MMA_SMEM = 128 * 32 + 256 * 32 + 1024;   // one K step of A and of B, K-major 16-byte chunks
template <bool MXF4, bool A_TMEM, int N>
__global__ void __launch_bounds__(128, 1)
mma_rate_kernel(int n_mma, TcStatus status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ WaitState wait;
    const int warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < (128 * 32 + 256 * 32) / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x22222222u;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        wait_state_init(&wait, status);
        mbar_init_fence();
    }
    fence_proxy_async_smem();
    if (warp == 0) {
        tmem_alloc(smem_u32(&tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    {   // columns 256..319: the A operand (when read from tensor memory) and the block scales
        uint32_t v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 0x22222222u;
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + 256, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 0x7F7F7F7Fu;
        tmem_st32(tmem + ((uint32_t)(warp * 32) << 16) + 288, v);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (threadIdx.x == 0) {
        const uint32_t a0 = smem_u32(smem), b0 = a0 + 128 * 32;
        const uint64_t da = smem_desc_kmajor(a0, 128 * 16, 128), db = smem_desc_kmajor(b0, 256 * 16, 128);
        const uint32_t idesc = MXF4 ? instr_desc_mxf4(128, N) : instr_desc(kAccF32, kFmtF16, kFmtF16, 128, N);
        uint32_t phase = 0;
        bool ok = true;
        for (int i = 0; i < n_mma && ok; i += 64) {
            for (int j = 0; j < 64; ++j) {
                const uint32_t d = tmem;   // one accumulator: back-to-back MMAs into it, as in a K loop
                if (MXF4 && A_TMEM) mma_mxf4_ts(d, tmem + 256, db, idesc, tmem + 288, tmem + 304, 1u);
                else if (MXF4) mma_mxf4(d, da, db, idesc, tmem + 288, tmem + 304, 1u);
                else mma_f16(d, da, db, idesc, 1u);
            }
            mma_commit(smem_u32(&bar));
            ok = mbar_wait(smem_u32(&bar), phase, &wait.abort);
            phase ^= 1u;
        }
        if (!ok) atomicExch(status.word, 1);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

template <int KIND>
int launch_alu(int repeat, uint32_t* sink, int sms, double* work, cudaStream_t st) {
    alu_rate_kernel<KIND><<<sms * ALU_BLOCKS_PER_SM, ALU_THREADS, 0, st>>>(repeat, sink);
    *work = (double)sms * ALU_BLOCKS_PER_SM * ALU_THREADS * CHAINS * ALU_UNROLL * (double)repeat *
            (KIND == BNN_RATE_POPC ? 32.0 * 2.0 : KIND == BNN_RATE_FFMA ? 2.0 : 1.0);
    return launch_status();
}

template <bool MXF4, bool A_TMEM, int N>
int launch_mma(int repeat, int sms, double* work, cudaStream_t st) {
    const TcStatus status = tc_status();
    if (!status.word) return BNN_ERR_CUDA;
    const int n_mma = repeat * 64;
    mma_rate_kernel<MXF4, A_TMEM, N><<<sms, 128, MMA_SMEM, st>>>(n_mma, status);
    *work = (double)sms * n_mma * 2.0 * 128.0 * N * (MXF4 ? 64.0 : 16.0);
    return launch_status();
}

}  // namespace

size_t pipe_rate_scratch_bytes(int which) {
    return which == BNN_RATE_L2_READ ? (size_t)(32u << 20) + (1u << 20) : (size_t)(8u << 20);
}

int launch_pipe_rate(int which, int repeat, void* scratch, size_t scratch_bytes, double* work, cudaStream_t st) {
    if (!scratch || !work) return BNN_ERR_NULL;
    if (repeat < 1 || repeat > (1 << 20)) return BNN_ERR_SHAPE;
    if (scratch_bytes < pipe_rate_scratch_bytes(which)) return BNN_ERR_WORKSPACE;
    if (!aligned16(scratch)) return BNN_ERR_ALIGN;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return BNN_ERR_CUDA;
    if ((size_t)sms * ALU_BLOCKS_PER_SM * ALU_THREADS * 4 > ((size_t)8u << 20)) return BNN_ERR_UNSUPPORTED;
    uint32_t* sink = static_cast<uint32_t*>(scratch);
    switch (which) {
        case BNN_RATE_POPC: return launch_alu<BNN_RATE_POPC>(repeat, sink, sms, work, st);
        case BNN_RATE_LOP3: return launch_alu<BNN_RATE_LOP3>(repeat, sink, sms, work, st);
        case BNN_RATE_IADD: return launch_alu<BNN_RATE_IADD>(repeat, sink, sms, work, st);
        case BNN_RATE_FADD: return launch_alu<BNN_RATE_FADD>(repeat, sink, sms, work, st);
        case BNN_RATE_FFMA: return launch_alu<BNN_RATE_FFMA>(repeat, sink, sms, work, st);
        case BNN_RATE_MMA_MXF4_N256: return launch_mma<true, false, 256>(repeat, sms, work, st);
        case BNN_RATE_MMA_MXF4_N192: return launch_mma<true, false, 192>(repeat, sms, work, st);
        case BNN_RATE_MMA_MXF4_N192_ATMEM: return launch_mma<true, true, 192>(repeat, sms, work, st);
        case BNN_RATE_MMA_F16_N256: return launch_mma<false, false, 256>(repeat, sms, work, st);
        case BNN_RATE_L2_READ: {
            // first 32 MB: the data read (whatever it holds); last 1 MB: the sink
            const size_t vecs = ((size_t)32u << 20) / 16;
            uint32_t* snk = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(scratch) + ((size_t)32u << 20));
            l2_read_kernel<<<sms, 512, 0, st>>>(static_cast<const uint4*>(scratch), vecs, repeat, snk);
            *work = (double)sms * repeat * (double)((size_t)32u << 20);
            return launch_status();
        }
        default: return BNN_ERR_UNSUPPORTED;
    }
}

}  // namespace bnn
