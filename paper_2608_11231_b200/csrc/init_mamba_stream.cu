// Mamba-2 exact composition (Eq. 6 with the scalar transitions of Eq. 2 / Eq. 5) as a persistent streaming
// kernel: S <- S_{c_1};  S <- exp(lambda_{c_j,h}) S + S_{c_j}, fp32 or bf16 pool, same arithmetic and order as
// init_mamba_exact_kernel (so the results are identical bit for bit, K = 1 is a plain copy).
//
// The work is cut into units (request, 16 KB tile of the state).  Every CTA walks its units one after the other
// and, inside a unit, the K chunks of the request; one producer thread copies each chunk's tile into a ring of
// shared-memory stages with bulk asynchronous copies (mbarrier transaction counts), 256 consumer threads hold
// the running tile in registers.  The ring never drains between units, so about 190 KB of loads are in flight
// per SM all the time -- more than per-thread loads can keep in flight with the registers a thread has.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kTileBytes = 16384;   // of one chunk's state per stage: 4096 fp32 or 8192 bf16 values
constexpr int kStages = 12;
constexpr int kConsumers = 256;
constexpr int kDecSlots = 64;       // decay ring: >= 32 (chunks prepared at once) + kStages + 1
constexpr int kSmemBytes = kStages * kTileBytes + 128;

__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :
                 : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gmem_src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

template <bool BF16>
__global__ void __launch_bounds__(kConsumers + 32, 1)
init_mamba_exact_stream_kernel(const __grid_constant__ InitArgs a, size_t state_elems, int head_elems, int tiles_per_state) {
    constexpr int kTileElems = kTileBytes / (BF16 ? 2 : 4);
    constexpr int kElemBytes = BF16 ? 2 : 4;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ float dec[kDecSlots];
    __shared__ volatile int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        dead = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumers / 32);
        }
        mbar_fence_init();
    }
    __syncthreads();
    const int n_units = a.n_req * tiles_per_state;
    const unsigned char *pool = static_cast<const unsigned char *>(a.states);

    if (warp == kConsumers / 32) {
        // ------------------------------------------------ producer warp: lane 0 issues the copies; all lanes fetch decays
        uint32_t it = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int r = u / tiles_per_state, tile = u % tiles_per_state;
            const int k0 = a.cu_k(r), K = a.cu_k(r + 1) - k0;
            const size_t off = static_cast<size_t>(tile) * kTileElems;
            const int h = static_cast<int>(off / head_elems);
            for (int j0 = 0; j0 < K; j0 += 32) {
                // decays of the next (up to) 32 chunks, one global latency for all of them
                const int nj = min(32, K - j0);
                if (lane < nj) {
                    const int j = j0 + lane;
                    const size_t c = static_cast<size_t>(a.id(k0 + j));
                    dec[(it + lane) % kDecSlots] = j > 0 ? expf(__ldg(a.transitions + c * a.H + h)) : 0.f;
                }
                __syncwarp();
                if (lane == 0) {
                    for (int jj = 0; jj < nj; ++jj, ++it) {
                        const int s = it % kStages;
                        if (it >= kStages) mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, &dead, a.status);
                        const size_t c = static_cast<size_t>(a.id(k0 + j0 + jj));
                        mbar_expect_tx(&full[s], kTileBytes);
                        bulk_load(ring + s * kTileBytes, pool + (c * state_elems + off) * kElemBytes, kTileBytes, &full[s]);
                    }
                }
                it = __shfl_sync(0xffffffffu, it, 0);
            }
        }
    } else {
        // ------------------------------------------------ consumers: thread owns 4 x 16 bytes of the tile
        constexpr int E = BF16 ? 8 : 4;   // values per 16 bytes
        uint32_t it = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int r = u / tiles_per_state, tile = u % tiles_per_state;
            const int K = a.cu_k(r + 1) - a.cu_k(r);
            float acc[4][E];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
            for (int j = 0; j < K; ++j, ++it) {
                const int s = it % kStages;
                mbar_wait(&full[s], (it / kStages) & 1, &dead, a.status);
                const float d = dec[it % kDecSlots];
                const uint4 *src = reinterpret_cast<const uint4 *>(ring + s * kTileBytes);
                uint4 raw[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) raw[i] = src[i * kConsumers + tid];
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float v[E];
                    const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
                    if (BF16) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            v[(2 * q) % E] = __uint_as_float(w[q] << 16);
                            v[(2 * q + 1) % E] = __uint_as_float(w[q] & 0xFFFF0000u);
                        }
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) v[q] = __uint_as_float(w[q]);
                    }
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[i][e] = (j == 0) ? v[e] : fmaf(d, acc[i][e], v[e]);
                }
            }
            float *dst = a.S0 + static_cast<size_t>(r) * state_elems + static_cast<size_t>(tile) * kTileElems;
            if (dead) continue;   // a wait ran out: the status word says so, S0 is left alone
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < E; e += 4)
                    __stcs(reinterpret_cast<float4 *>(dst + static_cast<size_t>(i * kConsumers + tid) * E + e),
                           make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]));
        }
    }
}

}  // namespace

bool init_mamba_stream_supported(const InitArgs &a, bool pool_bf16) {
    const size_t head = static_cast<size_t>(a.d_k) * a.d_v;
    return head % (kTileBytes / (pool_bf16 ? 2 : 4)) == 0;
}

cudaError_t launch_init_mamba_exact_stream(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    const size_t elems = static_cast<size_t>(a.H) * a.d_k * a.d_v;
    const int tiles = static_cast<int>(elems / (kTileBytes / (pool_bf16 ? 2 : 4)));
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const long long units = static_cast<long long>(a.n_req) * tiles;
    const int grid = static_cast<int>(units < sms ? units : sms);
    if (pool_bf16) {
        e = cudaFuncSetAttribute(init_mamba_exact_stream_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_mamba_exact_stream_kernel<true><<<grid, kConsumers + 32, kSmemBytes, s>>>(a, elems, a.d_k * a.d_v, tiles);
    } else {
        e = cudaFuncSetAttribute(init_mamba_exact_stream_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_mamba_exact_stream_kernel<false><<<grid, kConsumers + 32, kSmemBytes, s>>>(a, elems, a.d_k * a.d_v, tiles);
    }
    return cudaGetLastError();
}

}  // namespace lkv
