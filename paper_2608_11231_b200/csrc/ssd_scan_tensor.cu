// Chunkwise Mamba-2 (SSD) scan on the 5th-generation tensor cores (Eq. 1 with Eq. 2), for
// headdim P = 64, d_state N = 128 and bf16 x/B/C/y.  One CTA owns one (sequence, head) and walks
// the sequence in blocks of 128 tokens with the N x P state carried on chip (fp32 in tensor memory,
// a bf16 copy in shared memory as an MMA operand).  With l the running sum of dt * A_h inside the
// block and S the incoming state, per block:
//   (a) G      = C B^T                                   [128 x 128], K = N                 tcgen05
//       G'_ti  = G_ti e^{l_t - l_i} dt_i  (i <= t), 0 otherwise -> bf16 operand in TMEM     epilogue warps
//   (b) Yintra = G' X                                    [128 x 64],  K = 128 tokens         tcgen05 (A from TMEM)
//   (c) Yinter = C S                                     [128 x 64],  K = N                  tcgen05
//       y_t    = Yintra_t + e^{l_t} Yinter_t                                                 epilogue warps
//   (d) S     <- e^{l_Q} S + B^T X~,  X~_i = e^{l_Q - l_i} dt_i x_i   [128 x 64], K = tokens   tcgen05
//       (the state is pre-scaled in tensor memory, (d) accumulates onto it)                  state warps
// Only (c) and (d) depend on the previous block: (a) of the next block is issued as soon as the mask
// epilogue has drained G, so the epilogue warps never wait for the block-to-block chain
// (d) -> state copy -> (c), (d); the scaled X~ of the next block is prepared while (d) runs.
// A padded token has dt = 0.
// Warps 0-7 epilogue (thread = token row, warpgroup = column half), 8-11 state copy (the only SIMT
// work on the block-to-block chain), 12-15 per-block scalars and X~ (running ahead of the chain),
// 16 TMA, 17 MMA issue.  All waits on mbarriers are bounded.
#include <string.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kP = 64;     // headdim
constexpr int kN = 128;    // d_state
constexpr int kQ = 128;    // tokens per block
constexpr int kThreads = 576;

// shared-memory map (bytes, after 1024-byte alignment); every tile row is 128 bytes, 128-byte swizzle
constexpr int kXTile = kQ * 128;            // X [128 tokens x 64 p]
constexpr int kBTile = 2 * kQ * 128;        // B [B_kb0 | B_kb1], each [128 tokens x 64 n]
constexpr int kCTile = 2 * kQ * 128;        // C likewise
constexpr int kStageBytes = kXTile + kBTile + kCTile;   // 80 KB
constexpr int kOffX2 = 2 * kStageBytes;     // X~ [128 tokens x 64 p], double-buffered
constexpr int kOffHb = kOffX2 + 2 * kXTile; // bf16 state [128 n x 64 p]
constexpr int kOffSc = kOffHb + kN * 128;   // per-block scalars, three buffers
constexpr int kScFloats = 5 * kQ + 4;       // l2 = l log2(e), e^{l}, s = e^{l_Q - l} dt, f = e^{l_ref - l} dt, dt, flag
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxGroupRange = 100.f;     // log2 units: above this the per-group factors could overflow
constexpr int kSmemBytes = kOffSc + 3 * kScFloats * 4 + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

// tensor-memory map (columns)
constexpr uint32_t kTmG = 0;        // 128
constexpr uint32_t kTmYa = 128;     // Yintra, 2 x 64
constexpr uint32_t kTmYe = 256;     // Yinter, 2 x 64
constexpr uint32_t kTmH = 384;      // 64
constexpr uint32_t kTmGp = 448;     // G' as bf16 pairs: 128 K-elements in 64 columns
constexpr uint32_t kTmemCols = 512;

struct Bars {
    uint64_t full_bc[2], full_x[2];                    // TMA transactions
    uint64_t bc_free[2], ac_done, y_done, h_done[2];   // tcgen05.commit targets
    uint64_t mg_ready, yo_done[3], ys_ready[2];        // 256 epilogue threads
    uint64_t sc_ready[3], x2_ready[2], hb_ready;       // 128 threads (scalar warps; hb_ready: state warps)
};

__device__ __forceinline__ void named_bar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ uint32_t elect_one() {
    uint32_t e;
    asm volatile("{\n\t.reg .pred P1;\n\telect.sync _|P1, %1;\n\tselp.u32 %0, 1, 0, P1;\n\t}" : "=r"(e) : "r"(0xffffffffu));
    return e;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__global__ void __launch_bounds__(kThreads, 1)
ssd_scan_tensor_kernel(const __grid_constant__ SsdArgs a, const __grid_constant__ CUtensorMap mapX,
                       const __grid_constant__ CUtensorMap mapB, const __grid_constant__ CUtensorMap mapC,
                       const __grid_constant__ CUtensorMap mapY) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Bars bars;
    __shared__ uint32_t tmem_base;
    __shared__ volatile int dead;
    __shared__ float scan_carry[4];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, seq = a.cu[a.n_seq + 1 + blockIdx.y];   // launch order: longest sequence first
    const int grp = h / (a.H / a.G);
    const int t_begin = a.cu[seq], t_end = a.cu[seq + 1];
    const int nblk = (t_end - t_begin + kQ - 1) / kQ;
    const size_t sbase = (static_cast<size_t>(seq) * a.H + h) * kN * kP;

    if (nblk == 0) {  // empty sequence: hand the state through untouched
        if (a.S_T && a.S_T != a.S0)
            for (int e = tid; e < kN * kP; e += kThreads) store_state(a.S_T, a.st_bf16, sbase + e, a.S0 ? a.S0[sbase + e] : 0.f);
        return;
    }
    if (tid == 0) {
        dead = 0;
        uint64_t *b1 = &bars.full_bc[0];
        for (int i = 0; i < 10; ++i) mbar_init(b1 + i, 1);
        uint64_t *b256 = &bars.mg_ready;
        for (int i = 0; i < 6; ++i) mbar_init(b256 + i, 256);
        uint64_t *b128 = &bars.sc_ready[0];
        for (int i = 0; i < 6; ++i) mbar_init(b128 + i, 128);
        mbar_fence_init();
    }
    if (warp == 17) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    float *scal = reinterpret_cast<float *>(sm + kOffSc);

    if (warp == 16) {
        // ======================================================= TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&mapX);
            tma_prefetch_desc(&mapB);
            tma_prefetch_desc(&mapC);
            if (a.y) tma_prefetch_desc(&mapY);
            for (int b = 0; b < nblk + 2; ++b) {
                if (dead) break;   // a wait ran out: nothing more is issued
                const int st = b & 1;
                unsigned char *base = sm + st * kStageBytes;
                const int row = t_begin + b * kQ;
                // the two-stage ring cannot hide the DRAM latency of the tile loads: pull the tiles of block b+2 into L2 now
                if (b + 2 < nblk) {
                    tma_prefetch_l2_2d(&mapX, h * kP, row + 2 * kQ);
                    for (int kb = 0; kb < 2; ++kb) {
                        tma_prefetch_l2_2d(&mapB, grp * kN + kb * 64, row + 2 * kQ);
                        tma_prefetch_l2_2d(&mapC, grp * kN + kb * 64, row + 2 * kQ);
                    }
                }
                if (b < nblk) {
                    // B and C of block b-2 are free after its (d)
                    if (b >= 2) mbar_wait(&bars.bc_free[st], ((b - 2) >> 1) & 1, &dead, a.status);
                    mbar_expect_tx(&bars.full_bc[st], kBTile + kCTile);
                    for (int kb = 0; kb < 2; ++kb) {
                        tma_load_2d(base + kXTile + kb * kQ * 128, &mapB, grp * kN + kb * 64, row, &bars.full_bc[st]);
                        tma_load_2d(base + kXTile + kBTile + kb * kQ * 128, &mapC, grp * kN + kb * 64, row, &bars.full_bc[st]);
                    }
                }
                if (b >= 2) {
                    // the X tile of block b-2 now stages its y tile (whole blocks only): store it, then reuse the tile
                    mbar_wait(&bars.ys_ready[st], ((b - 2) >> 1) & 1, &dead, a.status);
                    if (a.y && row - kQ <= t_end && !dead) {
                        tma_store_2d(&mapY, base, h * kP, row - 2 * kQ);
                        tma_store_commit();
                        tma_store_wait_read();
                    }
                }
                if (b < nblk) {
                    mbar_expect_tx(&bars.full_x[st], kXTile);
                    tma_load_2d(base, &mapX, h * kP, row, &bars.full_x[st]);
                }
            }
            tma_store_wait_all();
        }
    } else if (warp == 17) {
        // ======================================================= MMA issuer (one elected thread)
        if (elect_one()) {
            constexpr uint32_t idA = umma_idesc(kFmtBF16, false, false, 128, 128);   // (a): C, B both K-major
            constexpr uint32_t idC = umma_idesc(kFmtBF16, false, true, 128, 64);     // (c), (b): B operand MN-major
            constexpr uint32_t idD = umma_idesc(kFmtBF16, true, true, 128, 64);      // (d): both MN-major
            const uint64_t dHb = umma_desc(smem_u32(sm + kOffHb), 0, 1024);
            // (a) G = C B^T of block b (both operands K-major)
            auto issue_a = [&](int b) {
                const uint32_t sbase_u = smem_u32(sm + (b & 1) * kStageBytes);
                const uint64_t dBk = umma_desc(sbase_u + kXTile, 0, 1024);
                const uint64_t dCk = umma_desc(sbase_u + kXTile + kBTile, 0, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t off = ((k >> 2) * (kQ * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmG, dCk + off, dBk + off, idA, k > 0);
                }
                umma_commit(&bars.ac_done);
            };
            mbar_wait(&bars.full_bc[0], 0, &dead, a.status);
            tc_fence_after_sync();
            issue_a(0);
            for (int b = 0; b < nblk; ++b) {
                if (dead) break;   // a wait ran out: nothing more is issued
                const uint32_t par = b & 1;
                const uint32_t sbase_u = smem_u32(sm + (b & 1) * kStageBytes);
                const uint64_t dX = umma_desc(sbase_u, 0, 1024);
                const uint64_t dBm = umma_desc(sbase_u + kXTile, kQ * 128, 1024);          // B tile, MN-major view (n blocks 16 KB apart)
                const uint64_t dCk = umma_desc(sbase_u + kXTile + kBTile, 0, 1024);
                const uint64_t dX2 = umma_desc(smem_u32(sm + kOffX2 + (b & 1) * kXTile), 0, 1024);
                mbar_wait(&bars.hb_ready, par, &dead, a.status);
                if (b >= 2) mbar_wait(&bars.yo_done[(b - 2) % 3], ((b - 2) / 3) & 1, &dead, a.status);
                tc_fence_after_sync();
                // (c) Yinter = C S : A = C (K = n), B = bf16 state read MN-major (rows = n)
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16(tm + kTmYe + 64 * par, dCk + (((k >> 2) * (kQ * 128) + (k & 3) * 32) >> 4), dHb + ((k * 16 * 128) >> 4), idC, k > 0);
                // (d) S += B^T X~ : A = B tile read MN-major (rows = tokens), B = X~ read MN-major
                mbar_wait(&bars.x2_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16(tm + kTmH, dBm + ((k * 16 * 128) >> 4), dX2 + ((k * 16 * 128) >> 4), idD, true);
                umma_commit(&bars.h_done[b & 1]);
                umma_commit(&bars.bc_free[b & 1]);
                // (b) Yintra = G' X : A = G' from tensor memory (8 columns per K-step of 16 tokens), B = X read MN-major
                mbar_wait(&bars.mg_ready, par, &dead, a.status);
                mbar_wait(&bars.full_x[b & 1], (b >> 1) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16_ts(tm + kTmYa + 64 * par, tm + kTmGp + 8 * k, dX + ((k * 16 * 128) >> 4), idC, k > 0);
                umma_commit(&bars.y_done);
                // (a) of the next block: G has been drained by the mask epilogue of this one
                if (b + 1 < nblk) {
                    mbar_wait(&bars.full_bc[(b + 1) & 1], ((b + 1) >> 1) & 1, &dead, a.status);
                    tc_fence_after_sync();
                    issue_a(b + 1);
                }
            }
        }
    } else if (warp >= 12) {
        // ======================================================= scalar warpgroup: thread = token; per-block scalars and X~, ahead of the chain
        const int x = tid - 384;   // 0..127
        const float Ah = a.A[h];
        // dt of this thread's token in block b (0 beyond the sequence end); fetched one block before it is used
        auto fetch_dt = [&](int b) {
            const int t = t_begin + b * kQ + x;
            return (b < nblk && t < t_end) ? a.dt[static_cast<size_t>(t) * a.H + h] : 0.f;
        };
        float dt_next = fetch_dt(0);
        auto prepare_scalars = [&](int b) {
            float *dst = scal + (b % 3) * kScFloats;
            const float dtv = dt_next;
            dt_next = fetch_dt(b + 1);
            float run = dtv * Ah;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float up = __shfl_up_sync(0xffffffffu, run, o);
                if (lane >= o) run += up;
            }
            if (lane == 31) scan_carry[warp & 3] = run;
            named_bar_sync(1, 128);
            for (int w = 0; w < (warp & 3); ++w) run += scan_carry[w];
            const float l2 = run * kLog2e;
            dst[x] = l2;
            dst[kQ + x] = exp2f(l2);
            dst[4 * kQ + x] = dtv;
            named_bar_sync(1, 128);
            dst[2 * kQ + x] = exp2f(dst[kQ - 1] - l2) * dtv;
            // factor of column x relative to the first column of its group of 16 (>= 1 before dt)
            const float rng = dst[x & ~15] - l2;
            dst[3 * kQ + x] = exp2f(fminf(rng, 126.f)) * dtv;
            // the fast epilogue is exact only while no group spans more than kMaxGroupRange
            const unsigned bad = __ballot_sync(0xffffffffu, rng > kMaxGroupRange);
            if (lane == 0) scan_carry[warp & 3] = bad ? 1.f : 0.f;
            named_bar_sync(1, 128);
            if (x == 0) dst[5 * kQ] = scan_carry[0] + scan_carry[1] + scan_carry[2] + scan_carry[3];
            named_bar_sync(1, 128);
            mbar_arrive(&bars.sc_ready[b % 3]);
        };
        // X~ row of token x of block b: s_x * X[x][:]
        auto scaled_x = [&](int b) {
            const float *sc = scal + (b % 3) * kScFloats;
            mbar_wait(&bars.full_x[b & 1], (b >> 1) & 1, &dead, a.status);
            const unsigned char *xt = sm + (b & 1) * kStageBytes;
            unsigned char *x2 = sm + kOffX2 + (b & 1) * kXTile;
            const float s = sc[2 * kQ + x];
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                const uint32_t off = sw128_offset(x, c8);
                const uint4 v = *reinterpret_cast<const uint4 *>(xt + off);
                const uint32_t in[4] = {v.x, v.y, v.z, v.w};
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    w[e] = pack_bf16(__uint_as_float(in[e] << 16) * s, __uint_as_float(in[e] & 0xFFFF0000u) * s);
                *reinterpret_cast<uint4 *>(x2 + off) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            fence_async_smem();
            mbar_arrive(&bars.x2_ready[b & 1]);
        };
        for (int b = 0; b < nblk; ++b) {
            // the scalar buffer of block b is the one block b-3 used: its outputs must be written
            if (b >= 3) mbar_wait(&bars.yo_done[b % 3], ((b - 3) / 3) & 1, &dead, a.status);
            prepare_scalars(b);
            // the X~ buffer of block b was read by (d) of block b-2
            if (b >= 2) mbar_wait(&bars.h_done[b & 1], ((b - 2) >> 1) & 1, &dead, a.status);
            scaled_x(b);
        }
    } else if (warp >= 8) {
        // ======================================================= state warpgroup: thread = state row n
        const int x = tid - 256;   // 0..127
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // initial state: fp32 into tensor memory pre-scaled by e^{l_Q} of block 0, bf16 copy unscaled
        mbar_wait(&bars.sc_ready[0], 0, &dead, a.status);
        {
            const float gq = scal[kQ + kQ - 1];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[32], sc[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const float v = a.S0 ? a.S0[sbase + static_cast<size_t>(x) * kP + 32 * q + c] : 0.f;
                    rr[c] = __float_as_uint(v);
                    sc[c] = __float_as_uint(v * gq);
                }
                tmem_st32(lane_base + kTmH + 32 * q, sc);
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) w[e] = pack_bf16(__uint_as_float(rr[8 * c8 + 2 * e]), __uint_as_float(rr[8 * c8 + 2 * e + 1]));
                    *reinterpret_cast<uint4 *>(sm + kOffHb + sw128_offset(x, 4 * q + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            tmem_st_wait();
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.hb_ready);
        }
        for (int b = 0; b < nblk; ++b) {
            // state after (d): copy for the next block's (c), pre-scale for its (d); or S_T at the end
            const bool last = b + 1 == nblk;
            if (!last) mbar_wait(&bars.sc_ready[(b + 1) % 3], ((b + 1) / 3) & 1, &dead, a.status);
            const float gq = last ? 1.f : scal[((b + 1) % 3) * kScFloats + kQ + kQ - 1];
            mbar_wait(&bars.h_done[b & 1], (b >> 1) & 1, &dead, a.status);
            tc_fence_after_sync();
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[32];
                tmem_ld32(lane_base + kTmH + 32 * q, rr);
                tmem_ld_wait();
                if (last) {
                    if (a.S_T && !dead && a.st_bf16) {
                        __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(a.S_T) + sbase + static_cast<size_t>(x) * kP + 32 * q;
#pragma unroll
                        for (int c = 0; c < 32; c += 8)
                            *reinterpret_cast<uint4 *>(dst + c) =
                                make_uint4(pack_bf16(__uint_as_float(rr[c]), __uint_as_float(rr[c + 1])), pack_bf16(__uint_as_float(rr[c + 2]), __uint_as_float(rr[c + 3])),
                                           pack_bf16(__uint_as_float(rr[c + 4]), __uint_as_float(rr[c + 5])), pack_bf16(__uint_as_float(rr[c + 6]), __uint_as_float(rr[c + 7])));
                    } else if (a.S_T && !dead) {
#pragma unroll
                        for (int c = 0; c < 32; c += 4)
                            *reinterpret_cast<float4 *>(a.S_T + sbase + static_cast<size_t>(x) * kP + 32 * q + c) =
                                make_float4(__uint_as_float(rr[c]), __uint_as_float(rr[c + 1]), __uint_as_float(rr[c + 2]), __uint_as_float(rr[c + 3]));
                    }
                } else {
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) w[e] = pack_bf16(__uint_as_float(rr[8 * c8 + 2 * e]), __uint_as_float(rr[8 * c8 + 2 * e + 1]));
                        *reinterpret_cast<uint4 *>(sm + kOffHb + sw128_offset(x, 4 * q + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
#pragma unroll
                    for (int c = 0; c < 32; ++c) rr[c] = __float_as_uint(__uint_as_float(rr[c]) * gq);
                    tmem_st32(lane_base + kTmH + 32 * q, rr);
                }
            }
            if (!last) {
                tmem_st_wait();
                fence_async_smem();
                tc_fence_before_sync();
                mbar_arrive(&bars.hb_ready);
            }
        }
    } else {
        // ======================================================= epilogue warpgroups: thread = token row t, warpgroup = column half
        const int t = tid & 127;
        const int half = warp >> 2;
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(a.y);
        {
            // operand columns above the diagonal for every row of this warp are never written again: zero them once
            const uint32_t z[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
            for (int q = 0; q < 4; ++q)
                if (64 * half + 16 * q > 32 * (warp & 3) + 31) tmem_st8(lane_base + kTmGp + 32 * half + 8 * q, z);
            tmem_st_wait();
        }
        for (int b = 0; b < nblk; ++b) {
            const float *sc = scal + (b % 3) * kScFloats;
            mbar_wait(&bars.sc_ready[b % 3], (b / 3) & 1, &dead, a.status);
            mbar_wait(&bars.ac_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            // G' row t, columns i = 64*half .. 64*half+63 -> bf16 pairs in TMEM columns 32*half .. 32*half+31 of the operand.
            // ((b) of the previous block, which read that operand, completed before its y epilogue ran.)
            // e^{l_t - l_i} dt_i = 2^{l2_t - l2_ref} * f_i with ref the first column of i's group of 16: one
            // exponential per group instead of one per element (every factor is <= 1 where i <= t);
            // blocks whose decay is too violent for that take the per-element path.
            {
                const float lt = sc[t];
                const bool fast = sc[5 * kQ] == 0.f;
#pragma unroll 1
                for (int q = 0; q < 4; ++q) {
                    const int i0 = 64 * half + 16 * q;
                    if (i0 > 32 * (warp & 3) + 31) break;   // above the diagonal for every row of this warp: stays zero
                    uint32_t rr[16];
                    tmem_ld16(lane_base + kTmG + 64 * half + 16 * q, rr);
                    tmem_ld_wait();
                    uint32_t w[8];
                    if (fast) {
                        float aa;
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(aa) : "f"(fminf(lt - sc[i0], 0.f)));
                        if (i0 + 15 <= 32 * (warp & 3)) {
                            // the whole group lies below the diagonal for every row of this warp: no masking
#pragma unroll
                            for (int c = 0; c < 16; c += 4) {
                                const float4 f = *reinterpret_cast<const float4 *>(sc + 3 * kQ + i0 + c);
                                w[c / 2] = pack_bf16(__uint_as_float(rr[c]) * aa * f.x, __uint_as_float(rr[c + 1]) * aa * f.y);
                                w[c / 2 + 1] = pack_bf16(__uint_as_float(rr[c + 2]) * aa * f.z, __uint_as_float(rr[c + 3]) * aa * f.w);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; c += 4) {
                                const float4 f = *reinterpret_cast<const float4 *>(sc + 3 * kQ + i0 + c);
                                const float v0 = (i0 + c <= t) ? __uint_as_float(rr[c]) * aa * f.x : 0.f;
                                const float v1 = (i0 + c + 1 <= t) ? __uint_as_float(rr[c + 1]) * aa * f.y : 0.f;
                                const float v2 = (i0 + c + 2 <= t) ? __uint_as_float(rr[c + 2]) * aa * f.z : 0.f;
                                const float v3 = (i0 + c + 3 <= t) ? __uint_as_float(rr[c + 3]) * aa * f.w : 0.f;
                                w[c / 2] = pack_bf16(v0, v1);
                                w[c / 2 + 1] = pack_bf16(v2, v3);
                            }
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; c += 2) {
                            const float v0 = (i0 + c <= t) ? __uint_as_float(rr[c]) * exp2f(lt - sc[i0 + c]) * sc[4 * kQ + i0 + c] : 0.f;
                            const float v1 = (i0 + c + 1 <= t) ? __uint_as_float(rr[c + 1]) * exp2f(lt - sc[i0 + c + 1]) * sc[4 * kQ + i0 + c + 1] : 0.f;
                            w[c / 2] = pack_bf16(v0, v1);
                        }
                    }
                    tmem_st8(lane_base + kTmGp + 32 * half + 8 * q, w);
                }
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars.mg_ready);
            // y_t[p] = Yintra + e^{l_t} Yinter, p = 32*half .. 32*half+31
            mbar_wait(&bars.y_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            {
                uint32_t ya[32], ye[32];
                tmem_ld32(lane_base + kTmYa + 64 * (b & 1) + 32 * half, ya);
                tmem_ld32(lane_base + kTmYe + 64 * (b & 1) + 32 * half, ye);
                tmem_ld_wait();
                const float et = sc[kQ + t];
                const int row0 = t_begin + b * kQ;
                uint32_t w[16];
#pragma unroll
                for (int c = 0; c < 32; c += 2)
                    w[c / 2] = pack_bf16(__uint_as_float(ya[c]) + et * __uint_as_float(ye[c]),
                                         __uint_as_float(ya[c + 1]) + et * __uint_as_float(ye[c + 1]));
                if (!a.y) {
                    // no outputs wanted (final states only)
                } else if (row0 + kQ <= t_end) {
                    // whole block inside the sequence: stage the y tile in this block's X tile ((b) has read it) in
                    // the layout of the tensor map and let the TMA warp store it -- full 128-byte rows
                    // instead of 32 scattered 16-byte pieces per warp instruction
                    unsigned char *ys = sm + (b & 1) * kStageBytes;
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8)
                        *reinterpret_cast<uint4 *>(ys + sw128_offset(t, 4 * half + c8)) = make_uint4(w[4 * c8], w[4 * c8 + 1], w[4 * c8 + 2], w[4 * c8 + 3]);
                    fence_async_smem();
                } else {
                    const int tok = row0 + t;
                    if (tok < t_end && !dead) {
                        __nv_bfloat16 *dst = y + (static_cast<size_t>(tok) * a.H + h) * kP + 32 * half;
#pragma unroll
                        for (int c8 = 0; c8 < 4; ++c8)
                            *reinterpret_cast<uint4 *>(dst + 8 * c8) = make_uint4(w[4 * c8], w[4 * c8 + 1], w[4 * c8 + 2], w[4 * c8 + 3]);
                    }
                }
                mbar_arrive(&bars.ys_ready[b & 1]);
            }
            tc_fence_before_sync();
            mbar_arrive(&bars.yo_done[b % 3]);
        }
    }
    grace_after_timeout(&dead);
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 17) tmem_dealloc(tm, kTmemCols);
}

}  // namespace

bool ssd_scan_tensor_supported(const SsdArgs &a, bool io_bf16) {
    return io_bf16 && a.P == kP && a.N == kN;
}

cudaError_t launch_ssd_scan_tensor(const SsdArgs &a, cudaStream_t s) {
    CUtensorMap mapX, mapB, mapC, mapY;
    const uint64_t rows = static_cast<uint64_t>(a.T_total);
    const uint64_t x_inner = static_cast<uint64_t>(a.H) * kP, bc_inner = static_cast<uint64_t>(a.G) * kN;
    if (rows == 0) {
        // no token anywhere: every CTA hands its state through and never touches a tile (and a map of zero rows
        // cannot be encoded)
        memset(&mapX, 0, sizeof(mapX));
        mapB = mapC = mapY = mapX;
    } else if (!make_tensor_map_2d(&mapX, a.x, 2, x_inner, rows, x_inner * 2, 64, kQ, true) ||
        !make_tensor_map_2d(&mapB, a.B, 2, bc_inner, rows, bc_inner * 2, 64, kQ, true) ||
        !make_tensor_map_2d(&mapC, a.C, 2, bc_inner, rows, bc_inner * 2, 64, kQ, true) ||
        (a.y && !make_tensor_map_2d(&mapY, a.y, 2, x_inner, rows, x_inner * 2, 64, kQ, true)))
        return cudaErrorInvalidValue;
    if (!a.y) mapY = mapX;   // never used by the kernel then
    cudaError_t e = cudaFuncSetAttribute(ssd_scan_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    ssd_scan_tensor_kernel<<<dim3(a.H, a.n_seq), kThreads, kSmemBytes, s>>>(a, mapX, mapB, mapC, mapY);
    return cudaGetLastError();
}

}  // namespace lkv
