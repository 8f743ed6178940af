// GDN exact composition on the 5th-generation tensor cores (Eq. 6 as the chain of Eq. 5):
//     S <- S_{c_1};   S <- T_{c_j} S + S_{c_j},  j = 2..K          (d_k = d_v = 128)
// One CTA owns one (request, head) chain and works on the transposed problem
//     S^T <- S^T T_j^T + S_j^T
// so that the carried state never leaves tensor memory:
//   - S^T (128 state columns = TMEM lanes, 128 state rows = TMEM columns, fp32 read as tf32) is the
//     A operand of tcgen05.mma, taken straight from TMEM;
//   - T_j, row-major fp32 as cached, is exactly the K-major B operand; a producer thread streams it
//     through a three-stage shared-memory ring with TMA (one SM takes in about 64 bytes per clock: the
//     64 KB of a transition are most of a step), four warps round it to nearest tf32 in place, and a
//     separate warp issues the MMAs;
//   - D = S^T T_j^T lands in one of two TMEM accumulators in two 64-column halves; two epilogue
//     warpgroups (thread = one state column, warpgroup = one half of the state rows) add S_j^T -- read
//     from global memory into registers while the MMAs run -- round, and store the result as the next
//     step's A operand; after the last chunk they write S0.
// The step is a chain MMA -> epilogue -> MMA.  It is shortened by splitting the contraction: the half of the
// new S^T that the first warpgroup writes holds the K-steps 0..7 of the next product, so the issuer starts
// those (both output halves) as soon as that warpgroup is done, while the second warpgroup still works, and
// issues K-steps 8..15 when it is done too -- output half 0 first, so that its epilogue starts while half 1
// is still on the tensor core.
// The tensor cores drop the low 13 mantissa bits of fp32 operands, which would shrink every product
// a little and add up along the chain, so S is rounded to nearest tf32 when it is stored as an
// operand, and every T_j is rounded to nearest in place in its stage before its MMAs.
// Every wait on an mbarrier is bounded; a wait that runs out marks the workspace status word.
#include <type_traits>

#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kD = 128;                      // d_k = d_v = MMA M = MMA N (two halves of 64)
constexpr int kTStageBytes = kD * kD * 4;    // one transition: 4 K-blocks of [128 rows x 128 B]
constexpr int kStages = 3;                   // transitions in the shared-memory ring
constexpr int kEpiThreads = 256;             // two epilogue warpgroups
constexpr int kRoundThreads = 128;           // warps that round the transitions
constexpr int kThreads = kEpiThreads + kRoundThreads + 64;   // + MMA warp + TMA warp
constexpr int kSmemBytes = kStages * kTStageBytes + 1024;
constexpr uint32_t kTmemCols = 512;          // D buffers: 0..127 and 128..255, A buffers: 256..383 and 384..511

// fp32 -> nearest tf32 (ties away from zero, as cvt.rna.tf32.f32 rounds), in integer arithmetic: the conversion
// instruction runs at a fraction of the integer rate, and one step rounds 32 K values per CTA.  Adding half a tf32 ulp
// to the magnitude and dropping the 13 low bits is that rounding (a carry out of the mantissa bumps the exponent, which
// is the right result; infinities and NaNs keep their class).
__device__ __forceinline__ uint32_t rn_tf32_bits(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }

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
init_gdn_exact_tensor_kernel(const __grid_constant__ InitArgs a, const __grid_constant__ CUtensorMap mapT) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // fullT: TMA transactions; roundT: the rounding warps are done with the stage; freeT: the MMAs of the step have read it;
    // e_ready[h]: warpgroup h has stored its half of the new operand; mma[h]: output half h of the step is complete
    __shared__ uint64_t bar_fullT[kStages], bar_roundT[kStages], bar_freeT[kStages], bar_eready[2], bar_mma[2];
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
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_fullT[s], 1); mbar_init(&bar_roundT[s], kRoundThreads); mbar_init(&bar_freeT[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&bar_eready[s], kEpiThreads / 2); mbar_init(&bar_mma[s], 1); }
        mbar_fence_init();
    }
    constexpr int kMmaWarp = (kEpiThreads + kRoundThreads) / 32, kTmaWarp = kMmaWarp + 1;
    if (warp == kMmaWarp) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tacc = tmem_base;
    auto prow = [&](int j) { return (a.id(k0 + j) * a.H + h) * kD; };   // first pool row of chunk j of this request, this head

    if (warp == kTmaWarp) {
        // ------------------------------------------------ TMA producer: transitions only
        if (lane == 0) {
            tma_prefetch_desc(&mapT);
            auto load_T = [&](int j) {
                const int st = stage_of(j);
                mbar_expect_tx(&bar_fullT[st], kTStageBytes);
                for (int kb = 0; kb < 4; ++kb) tma_load_2d(sm + st * kTStageBytes + kb * kD * 128, &mapT, kb * 32, prow(j), &bar_fullT[st]);
            };
            for (int j = 1; j < K && j <= kStages; ++j) load_T(j);
            for (int j = 1; j + kStages < K; ++j) {
                if (dead) break;   // a wait ran out: nothing more is issued
                // T_{j+kStages} takes over the stage of T_j as soon as the MMAs of step j are done
                mbar_wait(&bar_freeT[stage_of(j)], phase_of(j), &dead, a.status);
                load_T(j + kStages);
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(kFmtTF32, false, false, kD, 64);
            const uint64_t desc_hi = umma_desc(0, 0, 1024) & 0xFFFFFFFF00000000ull;
            for (int j = 1; j < K; ++j) {
                if (dead) break;   // a wait ran out: nothing more is issued
                const uint32_t lo0 = (smem_u32(sm + stage_of(j) * kTStageBytes) & 0x3FFFFu) >> 4;
                const uint32_t abuf = tacc + 256 + 128 * ((j - 1) & 1);
                const uint32_t dbuf = tacc + 128 * (j & 1);
                auto issue = [&](int nh, int kbeg) {
                    // rows 64*nh .. 64*nh+63 of T_j are the N extent of output half nh; K-steps kbeg .. kbeg+7
#pragma unroll
                    for (int k = kbeg; k < kbeg + 8; ++k) {
                        const uint32_t off = ((k >> 2) * (kD * 128) + nh * (64 * 128) + (k & 3) * 32) >> 4;
                        umma_tf32_ts(dbuf + 64 * nh, abuf + 8 * k, desc_hi | (lo0 + off), idesc, k > 0);
                    }
                };
                // rows 0..63 of S^T after step j-1 (the first warpgroup's half) are K-steps 0..7 of this product
                mbar_wait(&bar_roundT[stage_of(j)], phase_of(j), &dead, a.status);
                mbar_wait(&bar_eready[0], (j - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
                issue(0, 0);
                issue(1, 0);
                mbar_wait(&bar_eready[1], (j - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
                issue(0, 8);
                umma_commit(&bar_mma[0]);
                issue(1, 8);
                umma_commit(&bar_mma[1]);
                umma_commit(&bar_freeT[stage_of(j)]);
            }
        }
    } else if (warp >= kEpiThreads / 32) {
        // ------------------------------------------------ rounding warps: every transition to nearest tf32, in place
        const int x = tid - kEpiThreads;
        for (int j = 1; j < K; ++j) {
            const int st = stage_of(j);
            mbar_wait(&bar_fullT[st], phase_of(j), &dead, a.status);
            uint4 *t4 = reinterpret_cast<uint4 *>(sm + st * kTStageBytes);
#pragma unroll 8
            for (int q = 0; q < kTStageBytes / 16 / kRoundThreads; ++q) {
                uint4 v = t4[q * kRoundThreads + x];
                v.x = rn_tf32_bits(__uint_as_float(v.x)); v.y = rn_tf32_bits(__uint_as_float(v.y));
                v.z = rn_tf32_bits(__uint_as_float(v.z)); v.w = rn_tf32_bits(__uint_as_float(v.w));
                t4[q * kRoundThreads + x] = v;
            }
            fence_async_smem();
            mbar_arrive(&bar_roundT[st]);
        }
    } else {
        // ------------------------------------------------ epilogue: thread = state column c, warpgroup = half of the rows
        const int half = warp >> 2;                 // rows 64*half .. 64*half+63
        const int c = tid & 127;                    // state column = TMEM lane
        const int i0 = 64 * half;
        const uint32_t lane_base = tacc + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        using PoolT = typename std::conditional<SBF16, __nv_bfloat16, float>::type;
        const PoolT *pool = static_cast<const PoolT *>(a.states);
        // this thread's 64 values of chunk j's cached state (column c, rows i0..i0+63): a warp reads whole 128-byte
        // (fp32) or 64-byte (bf16) row pieces; issued before the wait for the MMAs, which hides their latency
        float sv[64];
        auto fetch_S = [&](int j) {
            const PoolT *src = pool + (static_cast<size_t>(prow(j)) + i0) * kD + c;
#pragma unroll
            for (int i = 0; i < 64; ++i) sv[i] = to_f32<PoolT>(src[static_cast<size_t>(i) * kD]);
        };
        // the rows of the chunk after next, pulled into L2 (64 rows of 512 or 256 bytes per warpgroup)
        auto prefetch_S = [&](int j) {
            if (j >= K) return;
            const char *src = reinterpret_cast<const char *>(pool + (static_cast<size_t>(prow(j)) + i0) * kD);
            constexpr int bytes = 64 * kD * static_cast<int>(sizeof(PoolT));
            for (int o = (tid & 127) * 128; o < bytes; o += 128 * 128) prefetch_l2(src + o);
        };
        prefetch_S(1);
        for (int j = 0; j < K; ++j) {
            prefetch_S(j + 2);
            fetch_S(j);
            if (j > 0) {
                mbar_wait(&bar_mma[half], (j - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
            }
            const uint32_t dbuf = lane_base + 128 * (j & 1) + i0;
            const uint32_t abuf = lane_base + 256 + 128 * (j & 1) + i0;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[32];
                if (j > 0) {
                    tmem_ld32(dbuf + 32 * q, rr);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) sv[32 * q + i] += __uint_as_float(rr[i]);
                }   // j == 0 hands the first chunk through untouched
                if (j < K - 1) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) rr[i] = rn_tf32_bits(sv[32 * q + i]);
                    tmem_st32(abuf + 32 * q, rr);
                }
            }
            if (j == K - 1) {
                if (!dead) {   // a wait ran out: the status word says so, S0 is left alone
#pragma unroll
                    for (int i = 0; i < 64; ++i) __stcs(out + static_cast<size_t>(i0 + i) * kD + c, sv[i]);
                }
            } else {
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(&bar_eready[half]);
            }
        }
    }
    grace_after_timeout(&dead);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tacc, kTmemCols);
}

}  // namespace

bool init_gdn_exact_tensor_supported(const InitArgs &a, bool) {
    return a.d_k == kD && a.d_v == kD && a.n_chunks >= 1 &&
           static_cast<long long>(a.n_chunks) * a.H * kD < (1ll << 31);
}

cudaError_t launch_init_gdn_exact_tensor(const InitArgs &a, bool pool_bf16, cudaStream_t s) {
    CUtensorMap mapT;
    const uint64_t rows = static_cast<uint64_t>(a.n_chunks) * a.H * kD;
    if (!make_tensor_map_2d(&mapT, a.transitions, 4, kD, rows, kD * 4, 32, kD, true)) return cudaErrorInvalidValue;
    cudaError_t e;
    if (pool_bf16) {
        e = cudaFuncSetAttribute(init_gdn_exact_tensor_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_gdn_exact_tensor_kernel<true><<<dim3(a.H, a.n_req), kThreads, kSmemBytes, s>>>(a, mapT);
    } else {
        e = cudaFuncSetAttribute(init_gdn_exact_tensor_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        init_gdn_exact_tensor_kernel<false><<<dim3(a.H, a.n_req), kThreads, kSmemBytes, s>>>(a, mapT);
    }
    return cudaGetLastError();
}

}  // namespace lkv
