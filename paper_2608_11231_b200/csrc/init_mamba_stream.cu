// Mamba-2 exact composition (Eq. 6 with the scalar transitions of Eq. 2 / Eq. 5) as a persistent streaming
// kernel: S <- S_{c_1};  S <- exp(lambda_{c_j,h}) S + S_{c_j}, fp32 or bf16 pool, same arithmetic and order as
// init_mamba_exact_kernel (so the results are identical bit for bit, K = 1 is a plain copy).
//
// The work is cut into units (request, tile of the state).  A tile is PER pieces of 4 KB of pool bytes (one 16-byte
// vector per consumer thread and piece), 16 KB by default; it may straddle heads (a piece never does), so every piece
// carries the decay of its own head.  Every CTA walks its units one after the other and, inside a unit, the K chunks of
// the request; one producer thread copies each chunk's tile into a ring of shared-memory stages with bulk asynchronous
// copies (mbarrier transaction counts), 256 consumer threads hold the running tile in registers.  The ring never drains
// between units, so about 190 KB of loads are in flight per SM all the time -- more than per-thread loads can keep in
// flight with the registers a thread has.  A launch whose 16 KB tiles would number between one and two per SM (a single
// request) takes the smallest larger tile that gives every SM at most one unit: with 160 units on 148 SMs a dozen SMs
// did two rounds and set the time of the launch.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kPieceBytes = 4096;    // 256 consumer threads x 16 bytes
constexpr int kRingBytes = 12 * 16384;
constexpr int kConsumers = 256;
constexpr int kMaxHeads = 3;         // heads a tile can touch (a head is at least 16 KB of pool bytes, a tile at most 32 KB)
constexpr int kDecSlots = 64;        // decay ring (per slot one decay per touched head): >= 32 (chunks prepared at once) + stages + 1
constexpr int kSmemBytes = kRingBytes + 128;

__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gmem_src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :
                 : "r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gmem_src)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

template <bool BF16, int PER>
__global__ void __launch_bounds__(kConsumers + 32, 1)
init_mamba_exact_stream_kernel(const __grid_constant__ InitArgs a, size_t state_elems, int head_elems, int tiles_per_state) {
    constexpr int kElemBytes = BF16 ? 2 : 4;
    constexpr int kPieceElems = kPieceBytes / kElemBytes;
    constexpr int kTileBytes = PER * kPieceBytes;
    constexpr int kTileElems = PER * kPieceElems;
    constexpr int kStages = kRingBytes / kTileBytes;
    static_assert(32 + kStages + 1 <= kDecSlots, "decay ring too small");
    extern __shared__ unsigned char smem_raw[];
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ float dec[kDecSlots][kMaxHeads];
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
    const int pieces_per_state = static_cast<int>(state_elems / kPieceElems);
    const unsigned char *pool = static_cast<const unsigned char *>(a.states);

    if (warp == kConsumers / 32) {
        // ------------------------------------------------ producer warp: lane 0 issues the copies; all lanes fetch decays
        uint32_t it = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int r = u / tiles_per_state, tile = u % tiles_per_state;
            const int k0 = a.cu_k(r), K = a.cu_k(r + 1) - k0;
            const size_t off = static_cast<size_t>(tile) * kTileElems;
            const int n_p = min(PER, pieces_per_state - tile * PER);            // pieces of this tile (the last one may be short)
            const int h0 = static_cast<int>(off / head_elems);                  // first head the tile touches
            const int n_h = static_cast<int>((off + static_cast<size_t>(n_p) * kPieceElems - 1) / head_elems) - h0 + 1;
            for (int j0 = 0; j0 < K; j0 += 32) {
                // decays of the next (up to) 32 chunks, one global latency for all of them
                const int nj = min(32, K - j0);
                if (lane < nj) {
                    const int j = j0 + lane;
                    const size_t c = static_cast<size_t>(a.id(k0 + j));
                    for (int hh = 0; hh < n_h; ++hh)
                        dec[(it + lane) % kDecSlots][hh] = j > 0 ? expf(__ldg(a.transitions + c * a.H + h0 + hh)) : 0.f;
                }
                __syncwarp();
                if (lane == 0) {
                    for (int jj = 0; jj < nj; ++jj, ++it) {
                        if (dead) break;   // a wait ran out: nothing more is issued
                        const int s = it % kStages;
                        if (it >= kStages) mbar_wait(&empty[s], ((it / kStages) & 1) ^ 1, &dead, a.status);
                        const size_t c = static_cast<size_t>(a.id(k0 + j0 + jj));
                        mbar_expect_tx(&full[s], n_p * kPieceBytes);
                        bulk_load(ring + s * kTileBytes, pool + (c * state_elems + off) * kElemBytes, n_p * kPieceBytes, &full[s]);
                    }
                }
                it = __shfl_sync(0xffffffffu, it, 0);
            }
        }
    } else {
        // ------------------------------------------------ consumers: thread owns one 16-byte vector of every piece of the tile
        constexpr int E = BF16 ? 8 : 4;   // values per 16 bytes
        uint32_t it = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int r = u / tiles_per_state, tile = u % tiles_per_state;
            const int K = a.cu_k(r + 1) - a.cu_k(r);
            const size_t off = static_cast<size_t>(tile) * kTileElems;
            const int n_p = min(PER, pieces_per_state - tile * PER);
            const int h0 = static_cast<int>(off / head_elems);
            int hsel[PER];   // which of the tile's heads piece i belongs to
#pragma unroll
            for (int i = 0; i < PER; ++i) hsel[i] = static_cast<int>((off + static_cast<size_t>(i) * kPieceElems) / head_elems) - h0;
            float acc[PER][E];
#pragma unroll
            for (int i = 0; i < PER; ++i)
#pragma unroll
                for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
            for (int j = 0; j < K; ++j, ++it) {
                const int s = it % kStages;
                mbar_wait(&full[s], (it / kStages) & 1, &dead, a.status);
                const float *dj = dec[it % kDecSlots];
                const uint4 *src = reinterpret_cast<const uint4 *>(ring + s * kTileBytes);
                uint4 raw[PER];
                float d[PER];
#pragma unroll
                for (int i = 0; i < PER; ++i) {
                    raw[i] = i < n_p ? src[i * kConsumers + tid] : make_uint4(0u, 0u, 0u, 0u);
                    d[i] = dj[min(hsel[i], kMaxHeads - 1)];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
#pragma unroll
                for (int i = 0; i < PER; ++i) {
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
                    for (int e = 0; e < E; ++e) acc[i][e] = (j == 0) ? v[e] : fmaf(d[i], acc[i][e], v[e]);
                }
            }
            float *dst = a.S0 + static_cast<size_t>(r) * state_elems + off;
            if (dead) continue;   // a wait ran out: the status word says so, S0 is left alone
#pragma unroll
            for (int i = 0; i < PER; ++i)
                if (i < n_p)
#pragma unroll
                    for (int e = 0; e < E; e += 4)
                        __stcs(reinterpret_cast<float4 *>(dst + static_cast<size_t>(i * kConsumers + tid) * E + e),
                               make_float4(acc[i][e], acc[i][e + 1], acc[i][e + 2], acc[i][e + 3]));
        }
    }
    grace_after_timeout(&dead);   // copies still in flight land before the ring is given back
}

}  // namespace

bool init_mamba_stream_supported(const InitArgs &a, bool pool_bf16) {
    // pieces never straddle heads, and a tile of up to 32 KB touches at most kMaxHeads heads
    const size_t head_bytes = static_cast<size_t>(a.d_k) * a.d_v * (pool_bf16 ? 2 : 4);
    return head_bytes % kPieceBytes == 0 && head_bytes >= 16384;
}

template <bool BF16, int PER>
static cudaError_t launch_stream(const InitArgs &a, int sms, cudaStream_t s) {
    const size_t elems = static_cast<size_t>(a.H) * a.d_k * a.d_v;
    const size_t pieces = elems / (kPieceBytes / (BF16 ? 2 : 4));
    const int tiles = static_cast<int>((pieces + PER - 1) / PER);
    const long long units = static_cast<long long>(a.n_req) * tiles;
    const int grid = static_cast<int>(units < sms ? units : sms);
    auto kern = init_mamba_exact_stream_kernel<BF16, PER>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kConsumers + 32, kSmemBytes, s>>>(a, elems, a.d_k * a.d_v, tiles);
    return cudaGetLastError();
}

cudaError_t launch_init_mamba_exact_stream(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    // 16 KB tiles (4 pieces) unless they would number between one and two per SM: then the smallest larger tile that
    // leaves every SM at most one unit (the results do not depend on the tile size)
    const long long pieces = static_cast<long long>(a.n_req) * a.H * a.d_k * a.d_v / (kPieceBytes / (pool_bf16 ? 2 : 4));
    int per = 4;
    if (a.n_req == 1 && pieces > 4ll * sms && pieces <= 8ll * sms) per = pieces <= 5ll * sms ? 5 : pieces <= 6ll * sms ? 6 : 8;
    if (pool_bf16)
        return per == 4 ? launch_stream<true, 4>(a, sms, s) : per == 5 ? launch_stream<true, 5>(a, sms, s)
             : per == 6 ? launch_stream<true, 6>(a, sms, s) : launch_stream<true, 8>(a, sms, s);
    return per == 4 ? launch_stream<false, 4>(a, sms, s) : per == 5 ? launch_stream<false, 5>(a, sms, s)
         : per == 6 ? launch_stream<false, 6>(a, sms, s) : launch_stream<false, 8>(a, sms, s);
}

}  // namespace lkv
