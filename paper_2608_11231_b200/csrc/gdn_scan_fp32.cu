// Chunkwise Gated DeltaNet scan in plain fp32 FMA (Eq. 1 with Eq. 3).
//
// The tight-tolerance path (fp32 I/O, small or unusual head sizes).  One CTA owns one
// (sequence, value head): the state stays in shared memory and the CTA walks the
// sequence in blocks of kC tokens.  Inside a block, with cg the running sum of g and
// S the incoming state, the per-token pseudo-values u_t solve the unit lower-triangular
// system
//     u_t + sum_{i<t} beta_t e^{cg_t-cg_i} (k_t.k_i) u_i = beta_t (v_t - e^{cg_t} S^T k_t)
// (solved here by forward substitution, one thread per state column), then
//     o_t = scale ( e^{cg_t} S^T q_t + sum_{i<=t} e^{cg_t-cg_i} (q_t.k_i) u_i )
//     S  <- e^{cg_C} S + sum_i e^{cg_C-cg_i} k_i u_i^T .
// Every exponent is a difference that is <= 0 for g <= 0, so nothing overflows.
#include "common.cuh"

namespace lkv {

namespace {

constexpr int kC = 32;  // tokens per block

template <typename T, int DV>
__global__ void __launch_bounds__(256) gdn_scan_fp32_kernel(const __grid_constant__ GdnArgs a) {
    constexpr int NG = 256 / DV;   // thread groups along tokens / state rows
    constexpr int TPER = kC / NG;  // tokens per thread in the token-parallel steps
    static_assert(kC % NG == 0 && TPER >= 1, "block shape");
    extern __shared__ float smem[];
    const int dk = a.d_k;
    const int ks = dk + 1;  // padded row stride of Qs / Ks
    float *S = smem;                       // [dk][DV]
    float *Qs = S + dk * DV;               // [kC][ks]
    float *Ks = Qs + kC * ks;              // [kC][ks]
    float *Vs = Ks + kC * ks;              // [kC][DV]
    float *Us = Vs + kC * DV;              // [kC][DV]   right-hand side, then u
    float *Am = Us + kC * DV;              // [kC][kC+1]
    float *Pm = Am + kC * (kC + 1);        // [kC][kC+1]
    float *cg = Pm + kC * (kC + 1);        // [kC]
    float *bs = cg + kC;                   // [kC]
    float *gs = bs + kC;                   // [kC]

    const int h = blockIdx.x, seq = a.cu[a.n_ranges + 1 + blockIdx.y];   // launch order: longest sequence first
    const bool tr = seq >= a.tr_first;                                    // transition sequence
    const int rg = tr ? seq - a.tr_first + a.tr_src0 : seq;
    const int hk = h / (a.H_v / a.H_k);
    const int tid = threadIdx.x;
    const int j = tid % DV, tg = tid / DV;
    const int t_begin = a.cu[rg], t_end = a.cu[rg + 1];
    const T *q = static_cast<const T *>(a.q);
    const T *k = static_cast<const T *>(a.k);
    const T *v = tr ? nullptr : static_cast<const T *>(a.v);
    T *o = tr ? nullptr : static_cast<T *>(a.o);
    const size_t sbase = (static_cast<size_t>(seq) * a.H_v + h) * dk * DV;
    float *ST = (tr && a.tr_out) ? a.tr_out : a.S_T;   // final state of this sequence
    const size_t obase = (tr && a.tr_out) ? (static_cast<size_t>(seq - a.tr_first) * a.H_v + h) * dk * DV : sbase;

    for (int idx = tid; idx < dk * DV; idx += 256)
        S[idx] = (a.s0_identity || tr) ? (idx / DV == idx % DV ? 1.f : 0.f) : (a.S0 ? a.S0[sbase + idx] : 0.f);

    for (int t0 = t_begin; t0 < t_end; t0 += kC) {
        const int n = min(kC, t_end - t0);
        for (int idx = tid; idx < kC * dk; idx += 256) {
            const int t = idx / dk, m = idx % dk;
            const size_t off = (static_cast<size_t>(t0 + t) * a.H_k + hk) * dk + m;
            Qs[t * ks + m] = t < n ? to_f32<T>(q[off]) : 0.f;
            Ks[t * ks + m] = t < n ? to_f32<T>(k[off]) : 0.f;
        }
        for (int idx = tid; idx < kC * DV; idx += 256) {
            const int t = idx / DV, c = idx % DV;
            Vs[idx] = (v && t < n) ? to_f32<T>(v[(static_cast<size_t>(t0 + t) * a.H_v + h) * DV + c]) : 0.f;
        }
        if (tid < kC) {
            const bool ok = tid < n;  // a padded token is the identity step: g = 0, beta = 0
            gs[tid] = ok ? a.g[static_cast<size_t>(t0 + tid) * a.H_v + h] : 0.f;
            bs[tid] = ok ? a.beta[static_cast<size_t>(t0 + tid) * a.H_v + h] : 0.f;
        }
        __syncthreads();
        if (tid == 0) {
            float run = 0.f;
            for (int t = 0; t < kC; ++t) { run += gs[t]; cg[t] = run; }
        }
        __syncthreads();
        // coupling matrices: warp <-> token t, lane <-> earlier token i
        for (int idx = tid; idx < kC * kC; idx += 256) {
            const int t = idx / kC, i = idx % kC;
            float am = 0.f, pm = 0.f;
            if (i <= t) {
                float kk = 0.f, qk = 0.f;
                for (int m = 0; m < dk; ++m) {
                    const float ki = Ks[i * ks + m];
                    kk = fmaf(Ks[t * ks + m], ki, kk);
                    qk = fmaf(Qs[t * ks + m], ki, qk);
                }
                const float dec = expf(cg[t] - cg[i]);
                pm = dec * qk;
                am = (i < t) ? bs[t] * dec * kk : 0.f;
            }
            Am[t * (kC + 1) + i] = am;
            Pm[t * (kC + 1) + i] = pm;
        }
        // state products K S and Q S: thread (tg, j) owns tokens tg, tg + NG, ... of column j
        float kS[TPER], qS[TPER];
#pragma unroll
        for (int u = 0; u < TPER; ++u) { kS[u] = 0.f; qS[u] = 0.f; }
        for (int m = 0; m < dk; ++m) {
            const float s = S[m * DV + j];
#pragma unroll
            for (int u = 0; u < TPER; ++u) {
                const int t = tg + NG * u;
                kS[u] = fmaf(Ks[t * ks + m], s, kS[u]);
                qS[u] = fmaf(Qs[t * ks + m], s, qS[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < TPER; ++u) {
            const int t = tg + NG * u;
            Us[t * DV + j] = bs[t] * (Vs[t * DV + j] - expf(cg[t]) * kS[u]);
        }
        __syncthreads();
        // forward substitution down the block, one thread per state column
        if (tid < DV) {
            float u[kC];
#pragma unroll
            for (int t = 0; t < kC; ++t) {
                float acc = Us[t * DV + tid];
#pragma unroll
                for (int i = 0; i < t; ++i) acc = fmaf(-Am[t * (kC + 1) + i], u[i], acc);
                u[t] = acc;
            }
#pragma unroll
            for (int t = 0; t < kC; ++t) Us[t * DV + tid] = u[t];
        }
        __syncthreads();
        // outputs
#pragma unroll
        for (int u = 0; u < TPER; ++u) {
            const int t = tg + NG * u;
            float acc = expf(cg[t]) * qS[u];
            for (int i = 0; i <= t; ++i) acc = fmaf(Pm[t * (kC + 1) + i], Us[i * DV + j], acc);
            if (o && t < n) o[(static_cast<size_t>(t0 + t) * a.H_v + h) * DV + j] = from_f32<T>(a.scale * acc);
        }
        // state carry: thread (tg, j) owns rows tg, tg + NG, ... of column j
        {
            float w[kC];
            const float cl = cg[kC - 1];
#pragma unroll
            for (int i = 0; i < kC; ++i) w[i] = expf(cl - cg[i]) * Us[i * DV + j];
            const float gam = expf(cl);
            for (int m = tg; m < dk; m += NG) {
                float acc = gam * S[m * DV + j];
#pragma unroll
                for (int i = 0; i < kC; ++i) acc = fmaf(Ks[i * ks + m], w[i], acc);
                S[m * DV + j] = acc;
            }
        }
        __syncthreads();
    }
    if (ST) {
        __syncthreads();
        for (int idx = tid; idx < dk * DV; idx += 256)
            store_state(ST, a.st_bf16, obase + idx, S[idx] + (a.S_add ? a.S_add[sbase + idx] : 0.f));
    }
}

size_t smem_bytes(int dk, int dv) {
    return sizeof(float) * (static_cast<size_t>(dk) * dv + 2 * kC * (dk + 1) + 2 * kC * dv + 2 * kC * (kC + 1) + 3 * kC);
}

template <typename T, int DV>
cudaError_t launch(const GdnArgs &a, cudaStream_t s) {
    const size_t smem = smem_bytes(a.d_k, DV);
    cudaError_t e = cudaFuncSetAttribute(gdn_scan_fp32_kernel<T, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    gdn_scan_fp32_kernel<T, DV><<<dim3(a.H_v, a.n_seq), 256, smem, s>>>(a);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const GdnArgs &a, cudaStream_t s) {
    switch (a.d_v) {
        case 16: return launch<T, 16>(a, s);
        case 32: return launch<T, 32>(a, s);
        case 64: return launch<T, 64>(a, s);
        case 128: return launch<T, 128>(a, s);
        case 256: return launch<T, 256>(a, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

// Shapes this kernel takes: d_v a power of two in [16, 256], and the whole working set
// within the 227 KB of shared memory a CTA may use.
bool gdn_scan_fp32_supported(int dk, int dv) {
    const bool pow2 = dv >= 16 && dv <= 256 && (dv & (dv - 1)) == 0;
    return pow2 && dk >= 1 && smem_bytes(dk, dv) <= 227 * 1024;
}

cudaError_t launch_gdn_scan_fp32(const GdnArgs &a, bool io_bf16, cudaStream_t s) {
    return io_bf16 ? dispatch<__nv_bfloat16>(a, s) : dispatch<float>(a, s);
}

}  // namespace lkv
