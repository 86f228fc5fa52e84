// Measurement helper, not part of the embedding path: one tile product on the fifth-generation tensor cores
// (tcgen05.mma kind::tf32, operands in shared memory, accumulator in tensor memory), checked against a plain FP32
// loop and timed.  It answers the design question of where this path could use tcgen05 at all: the products of the
// path (paper Sec. 3.2: C = A.B, E = C.D) have between 4 and 128 output columns, and the instruction's rate depends
// on that width (it reads its operands from shared memory: 4 KB of A per M128.k8 instruction whatever N is).
//
// D[128 x N] = A[128 x 32] . B[32 x N], both operands K-major without swizzle: a 16-byte piece (row r, k-chunk c)
// lies at ((r / 8) * 8 + c) * 128 + (r % 8) * 16 bytes (8 x 16-byte core matrices; stride between row groups 1024
// bytes, between k chunks 128 bytes).  One CTA of 128 threads; one thread issues; completion through an mbarrier
// with a bounded wait; tensor memory is freed on every path.
#include "common.cuh"

#define TP_TILE_BYTES 16384   // 128 rows x 32 floats

__device__ __forceinline__ uint32_t tp_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// shared-memory matrix descriptor: start address, leading (k chunk) and stride (row group) offsets in 16-byte units
__device__ __forceinline__ uint64_t tp_desc(uint32_t saddr, uint32_t lbo16, uint32_t sbo16)
{
    return (uint64_t)((saddr >> 4) & 0x3fffu) | ((uint64_t)(lbo16 & 0x3fffu) << 16) | ((uint64_t)(sbo16 & 0x3fffu) << 32) | (1ull << 46);
}

// fp32 accumulator, TF32 operands, both K-major, M = 128
__device__ __forceinline__ uint32_t tp_idesc(int n) { return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24); }

__device__ __forceinline__ void tp_mma(uint32_t taddr, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(taddr), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ bool tp_wait(uint64_t* mbar, uint32_t parity)
{
    for (int it = 0; it < (1 << 22); ++it) {   // bounded: a product that never completes is reported, not waited for
        uint32_t f;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(f) : "r"(tp_smem(mbar)), "r"(parity) : "memory");
        if (f) return true;
    }
    return false;
}

// rounds x per_round products into the same accumulator; with check != 0 the first product (4 k steps, K = 32) is read
// back and compared with a plain loop over the same operands: out[0] = max |difference|, out[1] = 1 on a timeout
template <int N>
__global__ void __launch_bounds__(128) k_probe_tcgen05(int rounds, int per_round, int check, float* out)
{
    static_assert(N == 32 || N == 128, "validated output widths");
    extern __shared__ __align__(1024) unsigned char tp_sm[];
    float* sA = reinterpret_cast<float*>(tp_sm);
    float* sB = reinterpret_cast<float*>(tp_sm + TP_TILE_BYTES);
    uint64_t* mbar = reinterpret_cast<uint64_t*>(tp_sm + 2 * TP_TILE_BYTES);
    uint32_t* tslot = reinterpret_cast<uint32_t*>(tp_sm + 2 * TP_TILE_BYTES + 8);
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    // operands: small multiples of 1/4 (exact in TF32, sums exact in fp32), A[r][k] and B[n][k] from a hash of the indices
    auto aval = [](int r, int k) { return (float)(((r * 131 + k * 71 + 3) % 17) - 8) * 0.25f; };
    auto bval = [](int n, int k) { return (float)(((n * 37 + k * 113 + 5) % 17) - 8) * 0.25f; };
    for (int i = tid; i < 128 * 32; i += 128) {
        const int r = i >> 5, k = i & 31;
        const int off = (((r >> 3) * 8 + (k >> 2)) * 128 + (r & 7) * 16 + (k & 3) * 4) >> 2;
        sA[off] = aval(r, k);
        sB[off] = r < N ? bval(r, k) : 0.f;
    }
    if (tid == 0) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tp_smem(mbar)));
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads shared memory through the async proxy
    __syncthreads();
    if (wid == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tp_smem(tslot)), "r"(128u));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t taddr = *tslot;
    const uint32_t idesc = tp_idesc(N);
    __shared__ int s_ok;
    if (tid == 0) {
        s_ok = 1;
        uint32_t parity = 0;
        if (check) {
            for (int ks = 0; ks < 4; ++ks)
                tp_mma(taddr, tp_desc(tp_smem(sA) + ks * 256, 8, 64), tp_desc(tp_smem(sB) + ks * 256, 8, 64), idesc, ks > 0 ? 1u : 0u);
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tp_smem(mbar)) : "memory");
            if (!tp_wait(mbar, parity)) s_ok = 0;
            parity ^= 1u;
        }
        for (int r = 0; r < rounds && s_ok && !check; ++r) {
            for (int i = 0; i < per_round; ++i) {
                const int ks = i & 3;
                tp_mma(taddr, tp_desc(tp_smem(sA) + ks * 256, 8, 64), tp_desc(tp_smem(sB) + ks * 256, 8, 64), idesc, 1u);
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tp_smem(mbar)) : "memory");
            if (!tp_wait(mbar, parity)) s_ok = 0;
            parity ^= 1u;
        }
    }
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (!s_ok && tid == 0) out[1] = 1.f;
    if (check && s_ok) {
        // row wid * 32 + lane of D sits in lane wid * 32 + lane of tensor memory, column n in column n
        float worst = 0.f;
        for (int c0 = 0; c0 < N; c0 += 32) {
            uint32_t v[32];
            const uint32_t a = taddr + ((uint32_t)(wid * 32) << 16) + (uint32_t)c0;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                           "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                         : "r"(a));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int r = wid * 32 + lane;
#pragma unroll 1
            for (int j = 0; j < 32; ++j) {
                float ref = 0.f;
                for (int k = 0; k < 32; ++k) ref = fmaf(aval(r, k), bval(c0 + j, k), ref);
                const float d = fabsf(__uint_as_float(v[j]) - ref);
                worst = d > worst ? d : worst;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { const float y = __shfl_xor_sync(0xffffffffu, worst, o); worst = y > worst ? y : worst; }
        if (lane == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(worst));   // non-negative floats order like their bit patterns
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (wid == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(128u));
}

template <int N>
static int tp_run(double* mma_per_second, double* max_abs_err, cudaStream_t s, int sms)
{
    const size_t smem = 2 * TP_TILE_BYTES + 64;
    float* dout = nullptr;
    cudaError_t e = cudaFuncSetAttribute(k_probe_tcgen05<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaMalloc(&dout, 2 * sizeof(float));   // a probe, not the path: the path allocates nothing
    if (e != cudaSuccess) { tt_set_last_cuda_error(e); return TT_EMB_ERR_CUDA; }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    float host[2] = {0.f, 0.f};
    float ms = 0.f;
    const int rounds = 50, per_round = 256;
    e = cudaMemsetAsync(dout, 0, 2 * sizeof(float), s);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) {
        k_probe_tcgen05<N><<<1, 128, smem, s>>>(0, 0, 1, dout);            // the checked product
        k_probe_tcgen05<N><<<sms, 128, smem, s>>>(2, per_round, 0, dout);  // warm-up
        cudaEventRecord(e0, s);
        k_probe_tcgen05<N><<<sms, 128, smem, s>>>(rounds, per_round, 0, dout);
        cudaEventRecord(e1, s);
        tt_note_launch(); tt_note_launch(); tt_note_launch();
        e = cudaEventSynchronize(e1);
    }
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e == cudaSuccess) e = cudaMemcpy(host, dout, 2 * sizeof(float), cudaMemcpyDeviceToHost);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(dout);
    if (e != cudaSuccess) { tt_set_last_cuda_error(e); return TT_EMB_ERR_CUDA; }
    if (host[1] != 0.f) return TT_EMB_ERR_CUDA;   // a product did not complete within the bounded wait
    *mma_per_second = (double)sms * rounds * per_round / (ms * 1e-3);
    *max_abs_err = (double)host[0];
    return TT_EMB_OK;
}

extern "C" int tt_emb_probe_tcgen05(int32_t n_cols, double* mma_per_second, double* max_abs_err, tt_emb_stream_t stream)
{
    if (!mma_per_second || !max_abs_err || (n_cols != 32 && n_cols != 128)) return TT_EMB_ERR_ARG;
    int sms = 0;
    if (!tt_device_ok(&sms)) return TT_EMB_ERR_ARCH;
    return n_cols == 32 ? tp_run<32>(mma_per_second, max_abs_err, (cudaStream_t)stream, sms)
                        : tp_run<128>(mma_per_second, max_abs_err, (cudaStream_t)stream, sms);
}
