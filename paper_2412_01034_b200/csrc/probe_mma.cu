// Measurement helper (not part of the method): how fast this GPU's tensor cores run tcgen05.mma when nothing else
// is in the way.  One CTA per SM keeps two operand tiles resident in shared memory (128 x 128 bytes and 256 x 128
// bytes, K-major, no swizzle) and one thread issues 128 x 256 MMAs over them back to back - kind::i8 (K = 32 per
// instruction) or kind::f16 with bf16 operands (K = 16) - into one accumulator in tensor memory.  The host times the
// launch; operations / time is the roof the integer and bf16 GEMM kernels of this library are compared with.
#include "qil_common.cuh"

namespace qil {

namespace {

constexpr int kRowsA = 128, kRowsB = 256, kRowBytes = 128;
constexpr int kThreads = 128;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (t - t0 > kWaitLimitNs) return false;
    }
}
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}

// kI8: kind::i8 (s8 x s8 -> s32), else kind::f16 (bf16 x bf16 -> f32)
template <bool kI8>
__global__ void __launch_bounds__(kThreads, 1) probe_mma_kernel(int iters, int commit_every, int* status) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* sa = smem;                              // [8 chunks][128 rows][16 bytes]
    unsigned char* sb = smem + kRowsA * kRowBytes;         // [8 chunks][256 rows][16 bytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sb + kRowsB * kRowBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
    const int tid = threadIdx.x;
    // operands: small values, so that neither accumulator type overflows or loses meaning over the run
    for (int i = tid; i < (kRowsA + kRowsB) * kRowBytes / 4; i += kThreads)
        reinterpret_cast<uint32_t*>(smem)[i] = kI8 ? ((i & 1) ? 0x01FF0001u : 0x00010100u) : ((i & 1) ? 0x3C003C00u : 0x00000000u);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars)));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + 1)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    if (tid == 0) {
        // instruction descriptor: D type at bit 4 (f32 = 1, s32 = 2), A and B type at bits 7 and 10 (bf16 = 1, s8 = 1),
        // N >> 3 at bit 17, M >> 4 at bit 24
        constexpr uint32_t idesc = ((kI8 ? 2u : 1u) << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
        const uint32_t a0 = smem_u32(sa), b0 = smem_u32(sb);
        bool ok = true;
        // The queue is bounded: a commit every `commit_every` iterations, on two barriers in turn; before a barrier is committed to
        // again its previous commit is waited for (a barrier's parity can only tell neighbouring phases apart).
        const uint32_t bar[2] = {smem_u32(bars), smem_u32(bars + 1)};
        uint32_t ph[2] = {0u, 0u};
        int ncommit = 0, since = 0;
        auto commit = [&]() {
            const int b = ncommit & 1;
            if (ncommit >= 2) {
                ok = mbar_wait(bar[b], ph[b]);
                ph[b] ^= 1u;
            }
            if (ok) {
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar[b]) : "memory");
                ++ncommit;
            }
        };
        for (int it = 0; ok && it < iters; ++it) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {  // 32 bytes of K per instruction
                const uint64_t ad = smem_desc(a0 + 2 * k * (kRowsA * 16), kRowsA * 16, 128);
                const uint64_t bd = smem_desc(b0 + 2 * k * (kRowsB * 16), kRowsB * 16, 128);
                if (kI8)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                                 ::"r"(tmem), "l"(ad), "l"(bd), "r"(idesc), "r"((it | k) ? 1u : 0u), "r"(0u) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
                                 ::"r"(tmem), "l"(ad), "l"(bd), "r"(idesc), "r"((it | k) ? 1u : 0u), "r"(0u) : "memory");
            }
            if (++since == commit_every) { since = 0; commit(); }
        }
        // everything issued is complete before tensor memory is released: the last two commits are still unwaited
        if (ok) commit();
        for (int back = 2; back >= 1; --back)
            if (ncommit >= back) {
                const int b = (ncommit - back) & 1;
                if (!mbar_wait(bar[b], ph[b])) ok = false;
                ph[b] ^= 1u;
            }
        if (!ok && status) atomicOr(status, (int)QIL_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256));
}

constexpr size_t kSmem = (size_t)(kRowsA + kRowsB) * kRowBytes + 16 + 16;

}  // namespace

// ops_out (host): operations of one launch (2 per multiply-add, all CTAs)
qil_status launch_probe_mma(bool i8, int iters, int commit_every, double* ops_out, int* status, cudaStream_t st) {
    const int C = num_sms();
    const double k_per_mma = i8 ? 32.0 : 16.0;
    if (ops_out) *ops_out = 2.0 * 128.0 * 256.0 * k_per_mma * 4.0 * (double)iters * (double)C;
    cudaError_t e;
    if (i8) {
        e = cudaFuncSetAttribute(probe_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) probe_mma_kernel<true><<<C, kThreads, kSmem, st>>>(iters, commit_every, status);
    } else {
        e = cudaFuncSetAttribute(probe_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) probe_mma_kernel<false><<<C, kThreads, kSmem, st>>>(iters, commit_every, status);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return QIL_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace qil
