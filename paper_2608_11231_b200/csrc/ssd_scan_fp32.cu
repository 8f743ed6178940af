// Chunkwise Mamba-2 (SSD) scan in plain fp32 FMA (Eq. 1 with Eq. 2).
//
// One CTA owns one (sequence, head); the N x P state stays in shared memory and the CTA
// walks the sequence in blocks of kQ tokens.  With l the running sum of dt * A_h inside
// the block and S the incoming state:
//     y_t = e^{l_t} S^T C_t + sum_{i<=t} e^{l_t-l_i} (C_t.B_i) dt_i x_i
//     S  <- e^{l_Q} S + sum_i e^{l_Q-l_i} dt_i B_i x_i^T .
// Exponents are differences <= 0 (A < 0, dt >= 0).  A padded token has dt = 0.
#include "common.cuh"

namespace lkv {

namespace {

constexpr int kQ = 32;

template <typename T, int P>
__global__ void __launch_bounds__(256) ssd_scan_fp32_kernel(const __grid_constant__ SsdArgs a) {
    constexpr int NG = 256 / P;
    constexpr int TPER = kQ / NG;
    static_assert(kQ % NG == 0 && TPER >= 1, "block shape");
    extern __shared__ float smem[];
    const int N = a.N;
    const int ns = N + 1;
    float *S = smem;                  // [N][P]
    float *Bs = S + N * P;            // [kQ][ns]
    float *Cs = Bs + kQ * ns;         // [kQ][ns]
    float *Xs = Cs + kQ * ns;         // [kQ][P]
    float *Gm = Xs + kQ * P;          // [kQ][kQ+1]
    float *ls = Gm + kQ * (kQ + 1);   // [kQ]
    float *dts = ls + kQ;             // [kQ]

    const int h = blockIdx.x, seq = a.cu[a.n_seq + 1 + blockIdx.y];   // launch order: longest sequence first
    const int grp = h / (a.H / a.G);
    const int tid = threadIdx.x;
    const int p = tid % P, tg = tid / P;
    const int t_begin = a.cu[seq], t_end = a.cu[seq + 1];
    const T *x = static_cast<const T *>(a.x);
    const T *Bg = static_cast<const T *>(a.B);
    const T *Cg = static_cast<const T *>(a.C);
    T *y = static_cast<T *>(a.y);
    const float Ah = a.A[h];
    const size_t sbase = (static_cast<size_t>(seq) * a.H + h) * N * P;

    for (int idx = tid; idx < N * P; idx += 256) S[idx] = a.S0 ? a.S0[sbase + idx] : 0.f;

    for (int t0 = t_begin; t0 < t_end; t0 += kQ) {
        const int n = min(kQ, t_end - t0);
        for (int idx = tid; idx < kQ * N; idx += 256) {
            const int t = idx / N, m = idx % N;
            const size_t off = (static_cast<size_t>(t0 + t) * a.G + grp) * N + m;
            Bs[t * ns + m] = t < n ? to_f32<T>(Bg[off]) : 0.f;
            Cs[t * ns + m] = t < n ? to_f32<T>(Cg[off]) : 0.f;
        }
        for (int idx = tid; idx < kQ * P; idx += 256) {
            const int t = idx / P, c = idx % P;
            Xs[idx] = t < n ? to_f32<T>(x[(static_cast<size_t>(t0 + t) * a.H + h) * P + c]) : 0.f;
        }
        if (tid < kQ) dts[tid] = tid < n ? a.dt[static_cast<size_t>(t0 + tid) * a.H + h] : 0.f;
        __syncthreads();
        if (tid == 0) {
            float run = 0.f;
            for (int t = 0; t < kQ; ++t) { run += dts[t] * Ah; ls[t] = run; }
        }
        __syncthreads();
        // masked, decayed C B^T with dt folded in: warp <-> t, lane <-> i
        for (int idx = tid; idx < kQ * kQ; idx += 256) {
            const int t = idx / kQ, i = idx % kQ;
            float gm = 0.f;
            if (i <= t) {
                float cb = 0.f;
                for (int m = 0; m < N; ++m) cb = fmaf(Cs[t * ns + m], Bs[i * ns + m], cb);
                gm = expf(ls[t] - ls[i]) * dts[i] * cb;
            }
            Gm[t * (kQ + 1) + i] = gm;
        }
        // C S: thread (tg, p) owns tokens tg, tg + NG, ...
        float cS[TPER];
#pragma unroll
        for (int u = 0; u < TPER; ++u) cS[u] = 0.f;
        for (int m = 0; m < N; ++m) {
            const float s = S[m * P + p];
#pragma unroll
            for (int u = 0; u < TPER; ++u) cS[u] = fmaf(Cs[(tg + NG * u) * ns + m], s, cS[u]);
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < TPER; ++u) {
            const int t = tg + NG * u;
            float acc = expf(ls[t]) * cS[u];
            for (int i = 0; i <= t; ++i) acc = fmaf(Gm[t * (kQ + 1) + i], Xs[i * P + p], acc);
            if (y && t < n) y[(static_cast<size_t>(t0 + t) * a.H + h) * P + p] = from_f32<T>(acc);
        }
        {
            float w[kQ];
            const float ll = ls[kQ - 1];
#pragma unroll
            for (int i = 0; i < kQ; ++i) w[i] = expf(ll - ls[i]) * dts[i] * Xs[i * P + p];
            const float gam = expf(ll);
            for (int m = tg; m < N; m += NG) {
                float acc = gam * S[m * P + p];
#pragma unroll
                for (int i = 0; i < kQ; ++i) acc = fmaf(Bs[i * ns + m], w[i], acc);
                S[m * P + p] = acc;
            }
        }
        __syncthreads();
    }
    if (a.S_T) {
        __syncthreads();
        for (int idx = tid; idx < N * P; idx += 256) store_state(a.S_T, a.st_bf16, sbase + idx, S[idx]);
    }
}

size_t smem_bytes(int N, int P) {
    return sizeof(float) * (static_cast<size_t>(N) * P + 2 * kQ * (N + 1) + kQ * P + kQ * (kQ + 1) + 2 * kQ);
}

template <typename T, int P>
cudaError_t launch(const SsdArgs &a, cudaStream_t s) {
    const size_t smem = smem_bytes(a.N, P);
    cudaError_t e = cudaFuncSetAttribute(ssd_scan_fp32_kernel<T, P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    ssd_scan_fp32_kernel<T, P><<<dim3(a.H, a.n_seq), 256, smem, s>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const SsdArgs &a, cudaStream_t s) {
    switch (a.P) {
        case 16: return launch<T, 16>(a, s);
        case 32: return launch<T, 32>(a, s);
        case 64: return launch<T, 64>(a, s);
        case 128: return launch<T, 128>(a, s);
        case 256: return launch<T, 256>(a, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool ssd_scan_fp32_supported(int N, int P) {
    const bool pow2 = P >= 16 && P <= 256 && (P & (P - 1)) == 0;
    return pow2 && N >= 1 && smem_bytes(N, P) <= 227 * 1024;
}

cudaError_t launch_ssd_scan_fp32(const SsdArgs &a, bool io_bf16, cudaStream_t s) {
    return io_bf16 ? dispatch<__nv_bfloat16>(a, s) : dispatch<float>(a, s);
}

}  // namespace lkv
