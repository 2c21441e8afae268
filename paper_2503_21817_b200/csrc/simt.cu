// Plain-FMA (CUDA-core) GEMM kernels with the Skip-FFN epilogues.  They serve the fp32 mode
// (true fp32 multiply-add, no TF32) and act as an on-device second opinion for the bf16
// tensor-core kernels.  One generic tile kernel, specialised by epilogue.
#include "common.cuh"

namespace skipffn {

constexpr int ST_BM = 64, ST_BN = 64, ST_BK = 16, ST_THREADS = 256;

template <typename T>
__device__ __forceinline__ void load_tile(float (*sm)[ST_BM + 4], const T *__restrict__ base,
                                          int64_t ld_mn, int64_t ld_k, int mn0, int k0, int MN,
                                          int K)
{
    const int tid = threadIdx.x;
#pragma unroll
    for (int i = 0; i < (ST_BM * ST_BK) / ST_THREADS; ++i) {
        int e = tid + i * ST_THREADS;
        int k, m;
        if (ld_k == 1) { k = e % ST_BK; m = e / ST_BK; }
        else           { m = e % ST_BM; k = e / ST_BM; }
        int gm = mn0 + m, gk = k0 + k;
        float v = 0.0f;
        if (gm < MN && gk < K) v = to_f32(base[(int64_t)gm * ld_mn + (int64_t)gk * ld_k]);
        sm[k][m] = v;
    }
}

template <typename T, int EPI>
__global__ void __launch_bounds__(ST_THREADS) k_simt_gemm(GemmArgs a)
{
    constexpr bool DUAL = (EPI == EPI_GATEUP);   // two accumulators sharing A (gate and up)
    __shared__ float As[ST_BK][ST_BM + 4];
    __shared__ float Bs[ST_BK][ST_BN + 4];
    __shared__ float Bs2[DUAL ? ST_BK : 1][ST_BN + 4];

    const int nk = a.status[ST_NK];
    const int M = a.m_from_nk ? nk : a.M;
    const int N = a.N;
    const int K = a.k_from_nk ? nk : a.K;
    const int m0 = blockIdx.y * ST_BM, n0 = blockIdx.x * ST_BN;
    if (m0 >= M) return;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

    float acc[4][4] = {}, acc2[DUAL ? 4 : 1][4] = {};
    const int segments = (EPI == EPI_DX) ? 2 : 1;   // dx sums dG*W_gate and dU*W_up
    for (int seg = 0; seg < segments; ++seg) {
        const T *A = (const T *)(seg == 0 ? a.A : a.A2);
        const T *B = (const T *)((seg == 0) ? a.B : a.B2);
        for (int k0 = 0; k0 < K; k0 += ST_BK) {
            load_tile<T>(As, A, a.lda_m, a.lda_k, m0, k0, M, K);
            load_tile<T>(Bs, B, a.ldb_n, a.ldb_k, n0, k0, N, K);
            if (DUAL) load_tile<T>(Bs2, (const T *)a.B2, a.ldb_n, a.ldb_k, n0, k0, N, K);
            __syncthreads();
#pragma unroll
            for (int k = 0; k < ST_BK; ++k) {
                float av[4], bv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) av[i] = As[k][ty + 16 * i];
#pragma unroll
                for (int j = 0; j < 4; ++j) bv[j] = Bs[k][tx + 16 * j];
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
                if (DUAL) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) bv[j] = Bs2[k][tx + 16 * j];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int j = 0; j < 4; ++j) acc2[DUAL ? i : 0][j] = fmaf(av[i], bv[j], acc2[DUAL ? i : 0][j]);
                }
            }
            __syncthreads();
        }
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty + 16 * i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx + 16 * j;
            if (n >= N) continue;
            float v = acc[i][j];
            int64_t o = (int64_t)m * a.ldo + n;
            if (EPI == EPI_GATEUP) {             // G, U, H = silu(G) * U   (compacted rows)
                float u = acc2[DUAL ? i : 0][j];
                if (a.out0) ((T *)a.out0)[o] = from_f32<T>(v);   // a recomputing forward stores H only
                if (a.out1) ((T *)a.out1)[o] = from_f32<T>(u);
                ((T *)a.out2)[o] = from_f32<T>(swiglu(v, u));   // from the fp32 accumulators
            } else if (EPI == EPI_DX && a.out_fp32) {        // pre-norm variant: raw fp32 rows, compact
                ((float *)a.out0)[o] = v;
            } else if (EPI == EPI_DOWN || EPI == EPI_DX) {   // residual add + row scatter
                float res = to_f32(((const T *)a.in0)[o]);   // compacted residual row
                int64_t tok = a.idx[m];
                ((T *)a.out0)[tok * a.ldo + n] = from_f32<T>(res + v);
            } else if (EPI == EPI_DH) {          // dG, dU from dH and the saved G, U
                float g = to_f32(((const T *)a.in0)[o]), u = to_f32(((const T *)a.in1)[o]);
                float dg, du;
                swiglu_bwd(v, g, u, dg, du);
                ((T *)a.out0)[o] = from_f32<T>(dg);
                ((T *)a.out1)[o] = from_f32<T>(du);
            } else {                             // EPI_DW
                if (a.out_fp32) {
                    float *d = (float *)a.out0 + o;
                    *d = a.accumulate ? *d + v : v;
                } else {
                    T *d = (T *)a.out0 + o;
                    *d = from_f32<T>(a.accumulate ? to_f32(*d) + v : v);
                }
            }
        }
    }
    // the tile row holding the last kept row also zeroes the padding rows Nk .. round_up(Nk, ROW_PAD)-1
    if ((EPI == EPI_GATEUP || EPI == EPI_DH) && m0 + ST_BM >= M) {
        int end = (M + ROW_PAD - 1) / ROW_PAD * ROW_PAD;
        for (int m = M + ty; m < end; m += 16)
            for (int n = n0 + tx; n < n0 + ST_BN && n < N; n += 16) {
                int64_t o = (int64_t)m * a.ldo + n;
                if (a.out0) ((T *)a.out0)[o] = from_f32<T>(0.0f);
                if (a.out1) ((T *)a.out1)[o] = from_f32<T>(0.0f);
                if (EPI == EPI_GATEUP) ((T *)a.out2)[o] = from_f32<T>(0.0f);
            }
    }
}

template <typename T>
static cudaError_t launch_t(int epi, const GemmArgs &a, cudaStream_t s)
{
    dim3 grid((a.N + ST_BN - 1) / ST_BN, (a.M + ST_BM - 1) / ST_BM);
    if (grid.x == 0 || grid.y == 0) return cudaSuccess;
    switch (epi) {
    case EPI_GATEUP: k_simt_gemm<T, EPI_GATEUP><<<grid, ST_THREADS, 0, s>>>(a); break;
    case EPI_DOWN:   k_simt_gemm<T, EPI_DOWN><<<grid, ST_THREADS, 0, s>>>(a); break;
    case EPI_DH:     k_simt_gemm<T, EPI_DH><<<grid, ST_THREADS, 0, s>>>(a); break;
    case EPI_DW:     k_simt_gemm<T, EPI_DW><<<grid, ST_THREADS, 0, s>>>(a); break;
    case EPI_DX:     k_simt_gemm<T, EPI_DX><<<grid, ST_THREADS, 0, s>>>(a); break;
    default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_simt_gemm(int epi, int dtype, const GemmArgs &a, cudaStream_t s)
{
    return dtype == SKIPFFN_FP32 ? launch_t<float>(epi, a, s) : launch_t<bf16>(epi, a, s);
}

}  // namespace skipffn
