// Weight-streaming skinny GEMM, first version (warp-level mma.sync, cp.async pipeline).
//
// Y[split][r][f] = sum_{k in split} X[r][k] * W[f][k]
// The weight matrix is the large operand (each element is read once per pass); the R <= 128 activation
// rows are the small one.  "Swap-AB": a CTA owns 128 weight rows (the MMA M dimension, 16 per warp) and
// all activation rows of its row chunk (the MMA N dimension), so weights stream through shared memory
// exactly once.  Split-K partial sums are written to separate planes and reduced by the consumer
// kernel in a fixed order, which keeps results bit-reproducible.
#include "kernels.cuh"

namespace glance {

namespace {

constexpr int BM = 128;     // weight rows per CTA
constexpr int BK = 64;      // k per stage (128 bytes per row)
constexpr int STAGES = 4;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// 128-byte rows, 16-byte chunks XOR-swizzled by the row
__device__ __forceinline__ uint32_t toff(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// NT = activation rows per CTA / 8
template <int NT>
__global__ void __launch_bounds__(256) gemm_mma_kernel(const bf16 *__restrict__ W, const bf16 *__restrict__ X,
                                                       float *__restrict__ Y, int Nout, int K, int R, int ldy,
                                                       size_t split_stride, int S) {
    constexpr int XR = NT * 8;
    constexpr int STAGE_BYTES = (BM + XR) * 128;
    extern __shared__ __align__(128) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int f0 = blockIdx.x * BM;
    const int split = blockIdx.y;
    const int r0 = blockIdx.z * XR;
    const int ktiles = K / BK;
    const int kt0 = (int)((long long)split * ktiles / S), kt1 = (int)((long long)(split + 1) * ktiles / S);
    const int nk = kt1 - kt0;

    auto load_stage = [&](int kt, int stage) {
        unsigned char *sW = smem + stage * STAGE_BYTES;
        unsigned char *sX = sW + BM * 128;
        const int k0 = kt * BK;
        for (int it = tid; it < BM * 8; it += 256) {
            const int r = it >> 3, c = it & 7;
            const int f = min(f0 + r, Nout - 1);
            cp_async16(smem_u32(sW + toff(r, c)), W + (size_t)f * K + k0 + c * 8);
        }
        for (int it = tid; it < XR * 8; it += 256) {
            const int r = it >> 3, c = it & 7;
            const int row = min(r0 + r, R - 1);
            cp_async16(smem_u32(sX + toff(r, c)), X + (size_t)row * K + k0 + c * 8);
        }
    };

    float acc[NT][4];
#pragma unroll
    for (int j = 0; j < NT; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < nk) load_stage(kt0 + s, s);
        cp_async_commit();
    }
    for (int i = 0; i < nk; ++i) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        if (i + STAGES - 1 < nk) load_stage(kt0 + i + STAGES - 1, (i + STAGES - 1) % STAGES);
        cp_async_commit();
        const unsigned char *sW = smem + (i % STAGES) * STAGE_BYTES;
        const unsigned char *sX = sW + BM * 128;
#pragma unroll
        for (int kk = 0; kk < BK / 16; ++kk) {
            uint32_t a0, a1, a2, a3;
            ldsm_x4(smem_u32(sW + toff(warp * 16 + (lane & 15), kk * 2 + (lane >> 4))), a0, a1, a2, a3);
#pragma unroll
            for (int j = 0; j < NT; j += 2) {
                uint32_t b0, b1, b2, b3;
                const int mtx = lane >> 3;
                ldsm_x4(smem_u32(sX + toff(j * 8 + (lane & 7) + (mtx >> 1) * 8, kk * 2 + (mtx & 1))), b0, b1, b2, b3);
                mma_bf16(acc[j], a0, a1, a2, a3, b0, b1);
                mma_bf16(acc[j + 1], a0, a1, a2, a3, b2, b3);
            }
        }
    }
    cp_async_wait<0>();

    const int g8 = lane >> 2, t4 = lane & 3;
    float *Ys = Y + (size_t)split * split_stride;
#pragma unroll
    for (int j = 0; j < NT; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int f = f0 + warp * 16 + g8 + (e >> 1) * 8;
            const int r = r0 + j * 8 + t4 * 2 + (e & 1);
            if (f < Nout && r < R) Ys[(size_t)r * ldy + f] = acc[j][e];
        }
    }
}

template <int NT>
void launch_nt(const bf16 *W, const bf16 *X, float *Y, int Nout, int K, int R, int ldy, size_t split_stride, int S,
               cudaStream_t st) {
    constexpr int XR = NT * 8;
    constexpr int smem = STAGES * (BM + XR) * 128;
    static bool once = false;
    if (!once) {
        cudaFuncSetAttribute(gemm_mma_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        once = true;
    }
    dim3 grid((Nout + BM - 1) / BM, S, (R + XR - 1) / XR);
    gemm_mma_kernel<NT><<<grid, 256, smem, st>>>(W, X, Y, Nout, K, R, ldy, split_stride, S);
}

}  // namespace

void launch_gemm(const bf16 *W, const bf16 *X, float *Y, int Nout, int K, int R, int ldy, size_t split_stride,
                 int S, cudaStream_t st) {
    if (R <= 16) launch_nt<2>(W, X, Y, Nout, K, R, ldy, split_stride, S, st);
    else if (R <= 32) launch_nt<4>(W, X, Y, Nout, K, R, ldy, split_stride, S, st);
    else if (R <= 64) launch_nt<8>(W, X, Y, Nout, K, R, ldy, split_stride, S, st);
    else launch_nt<16>(W, X, Y, Nout, K, R, ldy, split_stride, S, st);
}

}  // namespace glance
