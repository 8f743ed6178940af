// GDN exact composition on the 5th-generation tensor cores (Eq. 6 as the chain of Eq. 5):
//     S <- S_{c_1};   S <- T_{c_j} S + S_{c_j},  j = 2..K          (d_k = d_v = 128)
// One CTA owns one (request, head) chain and works on the transposed problem
//     S^T <- S^T T_j^T + S_j^T
// so that the carried state never leaves tensor memory:
//   - S^T (128 state columns = TMEM lanes, 128 state rows = TMEM columns, fp32 read as tf32) is the
//     A operand of tcgen05.mma, taken straight from TMEM;
//   - T_j, row-major fp32 as cached, is exactly the K-major B operand; a producer warp streams it
//     (and the S_j tiles) through shared memory with TMA, and a separate warp issues the MMAs, so
//     neither waits for the other's instructions.  (No L2 prefetch of later chunks: with one CTA per
//     SM the prefetched lines were evicted before their use and DRAM traffic grew by half.)
//   - D = S^T T_j^T lands in a TMEM accumulator in two 64-column halves; two epilogue warpgroups
//     (thread = one state column, warpgroup = one half of the state rows) add S_j^T, round, and
//     store the result as the next step's A operand (double-buffered in TMEM), the first half
//     while the tensor core still works on the second; after the last chunk they write S0.
// The tensor cores drop the low 13 mantissa bits of fp32 operands, which would shrink every product
// a little and add up along the chain, so S is rounded to nearest tf32 when it is stored as an
// operand, and T_{j+1} is rounded to nearest in place in its stage while the MMAs of step j run.
// Every wait on an mbarrier is bounded; a wait that runs out marks the workspace status word.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kD = 128;                      // d_k = d_v = MMA M = MMA N (two halves of 64)
constexpr int kTStageBytes = kD * kD * 4;    // one transition: 4 K-blocks of [128 rows x 128 B]
constexpr int kStages = 2;                   // transitions in the shared-memory ring
constexpr int kSHalfBytes = 64 * kD * 4;     // half of a cached state: 4 column blocks of [64 rows x 128 B]
constexpr int kEpiThreads = 256;             // two epilogue warpgroups
constexpr int kThreads = kEpiThreads + 64;   // + MMA warp + TMA warp
constexpr int kSmemBytes = kStages * kTStageBytes + 2 * kSHalfBytes + 1024;
constexpr uint32_t kTmemCols = 512;          // D: 0..127, A buffers: 128..255 and 256..383

__device__ __forceinline__ uint32_t rn_tf32_bits(float x) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return u;
}

__device__ __forceinline__ void umma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        :
        : "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}

// Transition j (1 <= j < K) travels through ring stage (j-1) % kStages; this is its barrier phase.
__device__ __forceinline__ int stage_of(int j) { return (j - 1) % kStages; }
__device__ __forceinline__ uint32_t phase_of(int j) { return static_cast<uint32_t>((j - 1) / kStages) & 1u; }

// SBF16: the cached states are stored as bf16 (the transitions are fp32 either way); S0 is written as fp32.
template <bool SBF16>
__global__ void __launch_bounds__(kThreads, 1)
init_gdn_exact_tensor_kernel(const __grid_constant__ InitArgs a, const __grid_constant__ CUtensorMap mapT,
                             const __grid_constant__ CUtensorMap mapS) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // fp32 pool: [half][4 column blocks][64 rows][32 floats]; bf16 pool: [half][2 column blocks][64 rows][64 bf16]
    unsigned char *sS = sm + kStages * kTStageBytes;
    constexpr int kSHalf = SBF16 ? kSHalfBytes / 2 : kSHalfBytes;   // bytes of half a cached state in the pool's dtype
    __shared__ uint64_t bar_fullT[kStages], bar_freeT[kStages], bar_fullS[2], bar_freeS[2], bar_mma[2], bar_sready;
    __shared__ uint32_t tmem_base;
    __shared__ volatile int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, r = blockIdx.y;
    const int k0 = a.cu_k(r), K = a.cu_k(r + 1) - k0;
    constexpr size_t ss = static_cast<size_t>(kD) * kD;
    float *out = a.S0 + (static_cast<size_t>(r) * a.H + h) * ss;

    if (K == 0) {  // empty request: zero state
        for (int e = tid * 4; e < kD * kD; e += kThreads * 4) *reinterpret_cast<float4 *>(out + e) = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    if (tid == 0) {
        dead = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_fullT[s], 1); mbar_init(&bar_freeT[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&bar_fullS[s], 1); mbar_init(&bar_freeS[s], 128); mbar_init(&bar_mma[s], 1); }
        mbar_init(&bar_sready, kEpiThreads);
        mbar_fence_init();
    }
    if (warp == 8) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tacc = tmem_base;

    if (warp == 9) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&mapT);
            tma_prefetch_desc(&mapS);
            auto prow = [&](int j) { return (a.id(k0 + j) * a.H + h) * kD; };
            auto load_T = [&](int j) {
                const int st = stage_of(j);
                mbar_expect_tx(&bar_fullT[st], kTStageBytes);
                for (int kb = 0; kb < 4; ++kb) tma_load_2d(sm + st * kTStageBytes + kb * kD * 128, &mapT, kb * 32, prow(j), &bar_fullT[st]);
            };
            auto load_S = [&](int j, int half) {
                mbar_expect_tx(&bar_fullS[half], kSHalf);
                constexpr int ncb = SBF16 ? 2 : 4, cols = SBF16 ? 64 : 32;   // 128-byte rows either way
                for (int cb = 0; cb < ncb; ++cb)
                    tma_load_2d(sS + half * kSHalfBytes + cb * 64 * 128, &mapS, cb * cols, prow(j) + 64 * half, &bar_fullS[half]);
            };
            load_S(0, 0);
            load_S(0, 1);
            for (int j = 1; j < K && j <= kStages; ++j) load_T(j);
            for (int j = 1; j < K; ++j) {
                // T_{j+1} takes over the stage of T_{j-1} as soon as the MMAs of step j-1 are done
                if (j >= 2 && j + 1 < K) {
                    mbar_wait(&bar_freeT[stage_of(j - 1)], phase_of(j - 1), &dead, a.status);
                    load_T(j + 1);
                }
                // S_j takes over the tile halves as the epilogue of step j-1 lets go of them
                for (int half = 0; half < 2; ++half) {
                    mbar_wait(&bar_freeS[half], (j - 1) & 1, &dead, a.status);
                    load_S(j, half);
                }
            }
        }
    } else if (warp == 8) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(kFmtTF32, false, false, kD, 64);
            const uint64_t desc_hi = umma_desc(0, 0, 1024) & 0xFFFFFFFF00000000ull;
            for (int j = 1; j < K; ++j) {
                // epilogue j-1 is done: S^T sits in A buffer (j-1)&1 and T_j has been rounded
                mbar_wait(&bar_sready, (j - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
                const uint32_t lo0 = (smem_u32(sm + stage_of(j) * kTStageBytes) & 0x3FFFFu) >> 4;
                const uint32_t abuf = tacc + 128 + 128 * ((j - 1) & 1);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    // rows 64*half .. 64*half+63 of T_j are the N extent of this half
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        const uint32_t off = ((k >> 2) * (kD * 128) + half * (64 * 128) + (k & 3) * 32) >> 4;
                        umma_tf32_ts(tacc + 64 * half, abuf + 8 * k, desc_hi | (lo0 + off), idesc, k > 0);
                    }
                    umma_commit(&bar_mma[half]);
                }
                umma_commit(&bar_freeT[stage_of(j)]);
            }
        }
    } else {
        // ------------------------------------------------ epilogue: thread = state column c, warpgroup = half of the rows
        const int half = warp >> 2;                 // rows 64*half .. 64*half+63
        const int c = tid & 127;                    // state column = TMEM lane
        const int i0 = 64 * half;
        const uint32_t lane_base = tacc + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const float *tile = reinterpret_cast<const float *>(sS + half * kSHalfBytes + (c >> 5) * 64 * 128) + (c & 31);
        const __nv_bfloat16 *tile16 = reinterpret_cast<const __nv_bfloat16 *>(sS + half * kSHalfBytes + (c >> 6) * 64 * 128) + (c & 63);
        for (int j = 0; j < K; ++j) {
            if (j + 1 < K) {  // round the next transition to nearest tf32 while this step's MMAs run
                const int st = stage_of(j + 1);
                mbar_wait(&bar_fullT[st], phase_of(j + 1), &dead, a.status);
                uint4 *t4 = reinterpret_cast<uint4 *>(sm + st * kTStageBytes);
#pragma unroll 4
                for (int q = 0; q < kTStageBytes / 16 / kEpiThreads; ++q) {
                    uint4 v = t4[q * kEpiThreads + tid];
                    v.x = rn_tf32_bits(__uint_as_float(v.x)); v.y = rn_tf32_bits(__uint_as_float(v.y));
                    v.z = rn_tf32_bits(__uint_as_float(v.z)); v.w = rn_tf32_bits(__uint_as_float(v.w));
                    t4[q * kEpiThreads + tid] = v;
                }
                fence_async_smem();
            }
            float val[64];
            if (j > 0) {
                mbar_wait(&bar_mma[half], (j - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    uint32_t rr[32];
                    tmem_ld32(lane_base + i0 + 32 * q, rr);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) val[32 * q + i] = __uint_as_float(rr[i]);
                }
            }
            // add this chunk's cached state, column c, rows i0..i0+63, from the TMA-filled tile
            mbar_wait(&bar_fullS[half], j & 1, &dead, a.status);
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                const float s = SBF16 ? __bfloat162float(tile16[i * 64]) : tile[i * 32];
                val[i] = (j > 0) ? val[i] + s : s;  // j == 0 hands the first chunk through untouched
            }
            mbar_arrive(&bar_freeS[half]);
            if (j == K - 1) {
                if (!dead) {   // a wait ran out: the status word says so, S0 is left alone
#pragma unroll
                    for (int i = 0; i < 64; ++i) __stcs(out + static_cast<size_t>(i0 + i) * kD + c, val[i]);
                }
            } else {
                const uint32_t abuf = lane_base + 128 + 128 * (j & 1) + i0;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    uint32_t rr[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) rr[i] = rn_tf32_bits(val[32 * q + i]);
                    tmem_st32(abuf + 32 * q, rr);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(&bar_sready);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tacc, kTmemCols);
}

}  // namespace

bool init_gdn_exact_tensor_supported(const InitArgs &a, bool) {
    return a.d_k == kD && a.d_v == kD && a.n_chunks >= 1 &&
           static_cast<long long>(a.n_chunks) * a.H * kD < (1ll << 31);
}

cudaError_t launch_init_gdn_exact_tensor(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    CUtensorMap mapT, mapS;
    const uint64_t rows = static_cast<uint64_t>(a.n_chunks) * a.H * kD;
    if (!make_tensor_map_2d(&mapT, a.transitions, 4, kD, rows, kD * 4, 32, kD, true)) return cudaErrorInvalidValue;
    if (pool_bf16 ? !make_tensor_map_2d(&mapS, a.states, 2, kD, rows, kD * 2, 64, 64, false)
                  : !make_tensor_map_2d(&mapS, a.states, 4, kD, rows, kD * 4, 32, 64, false))
        return cudaErrorInvalidValue;
    cudaError_t e;
    if (pool_bf16) {
        e = cudaFuncSetAttribute(init_gdn_exact_tensor_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_gdn_exact_tensor_kernel<true><<<dim3(a.H, a.n_req), kThreads, kSmemBytes, s>>>(a, mapT, mapS);
    } else {
        e = cudaFuncSetAttribute(init_gdn_exact_tensor_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_gdn_exact_tensor_kernel<false><<<dim3(a.H, a.n_req), kThreads, kSmemBytes, s>>>(a, mapT, mapS);
    }
    return cudaGetLastError();
}

}  // namespace lkv
