// Plain-FMA projection kernel: y[n,N] (fp32) = or += x[n,K] . W[N,K]^T, fp32 accumulation.
// It is the fp32 model path (the tensor cores have no fp32-input mode that keeps 1e-4) and the
// on-GPU cross-check of the bf16 tensor-core path.
#include "cdb_internal.h"

namespace cdbk {

bool launch_linear_tc(const cdb* h, const void* x, const void* W, float* y, int n, int N, int K, Epilogue ep, cudaStream_t st);
bool linear_tc_supported(const cdb* h, int n, int N, int K);

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T, int EP>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                        float* __restrict__ C, int n, int N, int K) {
    pdl_trigger();
    pdl_wait();
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const int lr = tid / 4, lk = (tid % 4) * 4;          // each thread stages 4 consecutive k of one row
    for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int k = k0 + lk + q;
            As[lk + q][lr] = (m0 + lr < n && k < K) ? ldf<T>(A + (size_t)(m0 + lr) * K + k) : 0.f;
            Ws[lk + q][lr] = (n0 + lr < N && k < K) ? ldf<T>(W + (size_t)(n0 + lr) * K + k) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Ws[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = m0 + ty * 4 + i;
        if (r >= n) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int cidx = n0 + tx * 4 + j;
            if (cidx >= N) continue;
            float* dst = C + (size_t)r * N + cidx;
            if (EP == (int)Epilogue::ResidualAdd) *dst += acc[i][j]; else *dst = acc[i][j];
        }
    }
}

template <typename T>
static void launch_simt(const void* x, const void* W, float* y, int n, int N, int K, Epilogue ep, cudaStream_t st) {
    dim3 grid((N + BN - 1) / BN, (n + BM - 1) / BM);
    if (ep == Epilogue::ResidualAdd)
        launch_pdl(gemm_simt_kernel<T, 1>, dim3(grid), dim3(256), 0, st, (const T*)x, (const T*)W, y, n, N, K);
    else
        launch_pdl(gemm_simt_kernel<T, 0>, dim3(grid), dim3(256), 0, st, (const T*)x, (const T*)W, y, n, N, K);
}

void launch_linear(const cdb* h, const void* x, const void* W, float* y, int n, int N, int K, Epilogue ep, cudaStream_t st) {
    if (n <= 0 || N <= 0) return;
    ProfScope ps(h, kProfLinear, st);
    CDB_LAUNCH(h);
    if (h->cfg.dtype == CDB_FP32) { launch_simt<float>(x, W, y, n, N, K, ep, st); return; }
    if (!(h->cfg.flags & CDB_FLAG_SIMT_GEMM) && linear_tc_supported(h, n, N, K)) {
        if (!launch_linear_tc(h, x, W, y, n, N, K, ep, st)) h->launch_error = 1;      // reported by the entry point
        return;
    }
    launch_simt<__nv_bfloat16>(x, W, y, n, N, K, ep, st);
}

}  // namespace cdbk
