// State-initialisation kernels (Eq. 4): single cached state, and exact composition
// (Eq. 6 as the chain of Eq. 5) for Mamba-2 (scalar decay, HBM-bound) and for GDN in
// plain fp32 FMA (the tight-tolerance / small-shape path; the tensor-core path for
// d_k = d_v = 128 lives in init_gdn_tensor.cu).
#include "common.cuh"

namespace lkv {

namespace {

// 16 bytes of pool state -> 4 (fp32 pool) or 8 (bf16 pool) floats.
template <bool BF16>
struct PoolVec;
template <>
struct PoolVec<false> {
    static constexpr int kElems = 4;
    __device__ static __forceinline__ void load(const void *base, size_t elem, float (&out)[4]) {
        const float4 v = __ldcs(reinterpret_cast<const float4 *>(static_cast<const float *>(base) + elem));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <>
struct PoolVec<true> {
    static constexpr int kElems = 8;
    __device__ static __forceinline__ void load(const void *base, size_t elem, float (&out)[8]) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(base) + elem));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
};

template <int E>
__device__ __forceinline__ void store_vec(float *dst, const float (&v)[E]) {
#pragma unroll
    for (int i = 0; i < E; i += 4) __stcs(reinterpret_cast<float4 *>(dst + i), make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]));
}

// ---------------------------------------------------------------- single cached state
// S0[r] = states[ids[cu_k[r] + b_r]], b_r = sel[r] or the last position.  A pure copy: with
// an fp32 pool the bits are untouched.  grid = (vectors per state / 256, n_req).
template <bool BF16>
__global__ void __launch_bounds__(256) init_single_kernel(const __grid_constant__ InitArgs a, size_t state_elems) {
    using PV = PoolVec<BF16>;
    const int r = blockIdx.y;
    const int k0 = a.cu_k(r), k1 = a.cu_k(r + 1);
    const size_t e = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * PV::kElems;
    if (e >= state_elems) return;
    float v[PV::kElems];
    if (k1 == k0) {
#pragma unroll
        for (int i = 0; i < PV::kElems; ++i) v[i] = 0.f;
    } else {
        const int b = a.sel(r, k1 - k0);
        const size_t chunk = static_cast<size_t>(a.id(k0 + b));
        PV::load(a.states, chunk * state_elems + e, v);
    }
    store_vec<PV::kElems>(a.S0 + static_cast<size_t>(r) * state_elems + e, v);
}

// ---------------------------------------------------------------- Mamba-2 exact composition
// S <- S_{c_1};  S <- exp(lambda_{c_j,h}) S + S_{c_j}.  Pure streaming: every thread owns
// one 16-byte vector of the state and walks the K chunks with kUnroll independent loads
// in flight; the decays are K scalars per head.  grid = (vectors per state / 256, n_req).
template <bool BF16>
__global__ void __launch_bounds__(256) init_mamba_exact_kernel(const __grid_constant__ InitArgs a, size_t state_elems, int head_elems) {
    using PV = PoolVec<BF16>;
    constexpr int E = PV::kElems;
    constexpr int kUnroll = 8;
    const int r = blockIdx.y;
    const int k0 = a.cu_k(r), K = a.cu_k(r + 1) - k0;
    const size_t e = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * E;
    if (e >= state_elems) return;
    const int h = static_cast<int>(e / head_elems);
    float acc[E];
#pragma unroll
    for (int i = 0; i < E; ++i) acc[i] = 0.f;
    int j = 0;
    if (K > 0) {
        PV::load(a.states, static_cast<size_t>(a.id(k0)) * state_elems + e, acc);
        j = 1;
    }
    for (; j < K; j += kUnroll) {
        float v[kUnroll][E];
        float dec[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (j + u < K) {
                const size_t c = static_cast<size_t>(a.id(k0 + j + u));
                PV::load(a.states, c * state_elems + e, v[u]);
                dec[u] = expf(__ldg(a.transitions + c * a.H + h));
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (j + u < K) {
#pragma unroll
                for (int i = 0; i < E; ++i) acc[i] = fmaf(dec[u], acc[i], v[u][i]);
            }
        }
    }
    store_vec<E>(a.S0 + static_cast<size_t>(r) * state_elems + e, acc);
}

// ---------------------------------------------------------------- GDN exact composition, fp32 FMA
// One CTA owns kTN columns of one head's state for one request: the chain
// S <- T_{c_j} S + S_{c_j} acts on the left, so columns never mix.  The current column
// block sits in shared memory; T_j streams through shared memory kTM rows at a time.
constexpr int kTN = 32;  // state columns per CTA
constexpr int kTM = 32;  // transition rows staged per step

template <bool BF16>
__global__ void __launch_bounds__(256) init_gdn_exact_fp32_kernel(const __grid_constant__ InitArgs a) {
    extern __shared__ float smem[];
    const int dk = a.d_k, dv = a.d_v;
    float *Scur = smem;                 // [dk][kTN]
    float *Snew = Scur + dk * kTN;      // [dk][kTN]
    float *Tt = Snew + dk * kTN;        // [kTM][dk + 1]
    const int tstride = dk + 1;
    const int col0 = blockIdx.x * kTN;
    const int h = blockIdx.y, r = blockIdx.z;
    const int k0 = a.cu_k(r), K = a.cu_k(r + 1) - k0;
    const size_t ss = static_cast<size_t>(dk) * dv;
    const int tid = threadIdx.x;
    const int c = tid % kTN;   // column inside the block
    const int rg = tid / kTN;  // row group 0..7
    const bool col_ok = col0 + c < dv;

    auto load_state = [&](int chunk, int i) -> float {
        const size_t off = (static_cast<size_t>(chunk) * a.H + h) * ss + static_cast<size_t>(i) * dv + col0 + c;
        if (!col_ok) return 0.f;
        if (BF16) return __bfloat162float(static_cast<const __nv_bfloat16 *>(a.states)[off]);
        return static_cast<const float *>(a.states)[off];
    };

    for (int i = rg; i < dk; i += 8) Scur[i * kTN + c] = (K > 0) ? load_state(a.id(k0), i) : 0.f;
    __syncthreads();
    for (int j = 1; j < K; ++j) {
        const int chunk = a.id(k0 + j);
        const float *Tj = a.transitions + (static_cast<size_t>(chunk) * a.H + h) * dk * dk;
        for (int i0 = 0; i0 < dk; i0 += kTM) {
            for (int idx = tid; idx < kTM * dk; idx += 256) {
                const int ii = idx / dk, m = idx % dk;
                Tt[ii * tstride + m] = (i0 + ii < dk) ? __ldg(Tj + static_cast<size_t>(i0 + ii) * dk + m) : 0.f;
            }
            __syncthreads();
            // thread (rg, c) produces rows i0 + rg, i0 + rg + 8, ... of column c
            float acc[kTM / 8];
#pragma unroll
            for (int u = 0; u < kTM / 8; ++u) acc[u] = 0.f;
            for (int m = 0; m < dk; ++m) {
                const float s = Scur[m * kTN + c];
#pragma unroll
                for (int u = 0; u < kTM / 8; ++u) acc[u] = fmaf(Tt[(rg + 8 * u) * tstride + m], s, acc[u]);
            }
#pragma unroll
            for (int u = 0; u < kTM / 8; ++u) {
                const int i = i0 + rg + 8 * u;
                if (i < dk) Snew[i * kTN + c] = acc[u] + load_state(chunk, i);
            }
            __syncthreads();
        }
        float *t = Scur; Scur = Snew; Snew = t;
    }
    if (col_ok)
        for (int i = rg; i < dk; i += 8)
            a.S0[(static_cast<size_t>(r) * a.H + h) * ss + static_cast<size_t>(i) * dv + col0 + c] = Scur[i * kTN + c];
}

}  // namespace

cudaError_t launch_init_single(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    const size_t elems = static_cast<size_t>(a.H) * a.d_k * a.d_v;
    const int per = pool_bf16 ? 8 : 4;
    dim3 grid(static_cast<unsigned>((elems / per + 255) / 256), a.n_req);
    if (pool_bf16) init_single_kernel<true><<<grid, 256, 0, s>>>(a, elems);
    else init_single_kernel<false><<<grid, 256, 0, s>>>(a, elems);
    return cudaGetLastError();
}

cudaError_t launch_init_mamba_exact(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    const size_t elems = static_cast<size_t>(a.H) * a.d_k * a.d_v;
    const int per = pool_bf16 ? 8 : 4;
    dim3 grid(static_cast<unsigned>((elems / per + 255) / 256), a.n_req);
    if (pool_bf16) init_mamba_exact_kernel<true><<<grid, 256, 0, s>>>(a, elems, a.d_k * a.d_v);
    else init_mamba_exact_kernel<false><<<grid, 256, 0, s>>>(a, elems, a.d_k * a.d_v);
    return cudaGetLastError();
}

cudaError_t launch_init_gdn_exact_fp32(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    const size_t smem = (static_cast<size_t>(2) * a.d_k * kTN + static_cast<size_t>(kTM) * (a.d_k + 1)) * sizeof(float);
    dim3 grid((a.d_v + kTN - 1) / kTN, a.H, a.n_req);
    cudaError_t e;
    if (pool_bf16) {
        e = cudaFuncSetAttribute(init_gdn_exact_fp32_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        init_gdn_exact_fp32_kernel<true><<<grid, 256, smem, s>>>(a);
    } else {
        e = cudaFuncSetAttribute(init_gdn_exact_fp32_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        init_gdn_exact_fp32_kernel<false><<<grid, 256, smem, s>>>(a);
    }
    return cudaGetLastError();
}

namespace {

// One warp per (sequence, group of 32 heads): lanes walk consecutive heads, so every token's dt row is read with
// coalesced 128-byte accesses; four partial sums per lane keep several loads in flight.
__global__ void mamba_logdecay_kernel(const __grid_constant__ SsdArgs a, float *__restrict__ out) {
    const int seq = blockIdx.y;
    const int h = blockIdx.x * 32 + (threadIdx.x & 31);
    const int part = threadIdx.x >> 5, nparts = blockDim.x >> 5;
    __shared__ float red[8][32];
    const int t0 = a.cu[seq], t1 = a.cu[seq + 1];
    float acc = 0.f;
    if (h < a.H)
        for (int t = t0 + part; t < t1; t += nparts) acc += a.dt[static_cast<size_t>(t) * a.H + h];
    red[part][threadIdx.x & 31] = acc;
    __syncthreads();
    if (part == 0 && h < a.H) {
        float sum = 0.f;
        for (int p = 0; p < nparts; ++p) sum += red[p][threadIdx.x];
        out[static_cast<size_t>(seq) * a.H + h] = a.A[h] * sum;
    }
}

}  // namespace

cudaError_t launch_mamba_logdecay(const SsdArgs &a, float *logdecay, cudaStream_t s) {
    mamba_logdecay_kernel<<<dim3((a.H + 31) / 32, a.n_seq), 256, 0, s>>>(a, logdecay);
    return cudaGetLastError();
}

namespace {

constexpr int kErrThreads = 256;
constexpr size_t kErrElemsPerCta = 16384;   // 64 KB of each input per CTA: 16 float4 per thread

// Squared norms of (x - r) and r over one slice of one state; one (num, den) pair per CTA, summed in a fixed order.
__global__ void state_err_partial_kernel(const float *__restrict__ x, const float *__restrict__ r, size_t elems, int parts,
                                         float *__restrict__ partials) {
    const int state = blockIdx.y, part = blockIdx.x;
    const size_t vecs = elems / 4;
    const size_t v0 = vecs * part / parts, v1 = vecs * (part + 1) / parts;
    const float4 *xv = reinterpret_cast<const float4 *>(x + static_cast<size_t>(state) * elems);
    const float4 *rv = reinterpret_cast<const float4 *>(r + static_cast<size_t>(state) * elems);
    float num = 0.f, den = 0.f;
    for (size_t i = v0 + threadIdx.x; i < v1; i += kErrThreads) {
        const float4 a = __ldcs(xv + i), b = __ldcs(rv + i);
        const float d0 = a.x - b.x, d1 = a.y - b.y, d2 = a.z - b.z, d3 = a.w - b.w;
        num += d0 * d0 + d1 * d1 + d2 * d2 + d3 * d3;
        den += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, o);
        den += __shfl_xor_sync(0xffffffffu, den, o);
    }
    __shared__ float sn[kErrThreads / 32], sd[kErrThreads / 32];
    if ((threadIdx.x & 31) == 0) { sn[threadIdx.x >> 5] = num; sd[threadIdx.x >> 5] = den; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float n = 0.f, d = 0.f;
        for (int w = 0; w < kErrThreads / 32; ++w) { n += sn[w]; d += sd[w]; }
        partials[2 * (static_cast<size_t>(state) * parts + part)] = n;
        partials[2 * (static_cast<size_t>(state) * parts + part) + 1] = d;
    }
}

__global__ void state_err_final_kernel(const float *__restrict__ partials, int parts, int n_states, float *__restrict__ rel_err) {
    const int state = blockIdx.x * blockDim.x + threadIdx.x;
    if (state >= n_states) return;
    float n = 0.f, d = 0.f;
    for (int p = 0; p < parts; ++p) {
        n += partials[2 * (static_cast<size_t>(state) * parts + p)];
        d += partials[2 * (static_cast<size_t>(state) * parts + p) + 1];
    }
    rel_err[state] = sqrtf(n) / sqrtf(d);
}

}  // namespace

int state_err_parts(size_t elems) {
    const size_t parts = (elems + kErrElemsPerCta - 1) / kErrElemsPerCta;
    return static_cast<int>(parts < 1 ? 1 : (parts > 4096 ? 4096 : parts));
}

cudaError_t launch_state_rel_error(const float *x, const float *r, float *rel_err, int n_states, size_t elems,
                                   float *partials, cudaStream_t s) {
    const int parts = state_err_parts(elems);
    state_err_partial_kernel<<<dim3(parts, n_states), kErrThreads, 0, s>>>(x, r, elems, parts, partials);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    state_err_final_kernel<<<(n_states + 127) / 128, 128, 0, s>>>(partials, parts, n_states, rel_err);
    return cudaGetLastError();
}

}  // namespace lkv
