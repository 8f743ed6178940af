// Chunkwise Gated DeltaNet scan on the 5th-generation tensor cores (Eq. 1 with Eq. 3), for
// d_k = d_v = 128 and bf16 q/k/v/o.  One CTA owns one (sequence, value head) and walks the
// sequence in blocks of 64 tokens, carrying the state on chip.
//
// Everything is held transposed so that every tensor-core tile has M = d_v = 128 rows (all 128
// TMEM lanes): lane j owns state column j.  Per block, with cg the running sum of g,
// gam_t = e^{cg_t}, Gam_ti = e^{cg_t - cg_i}, w_i = e^{cg_C - cg_i} and S the incoming state:
//   (1) G    = [Q;K] K^T             rows 0..63: q_t.k_i, rows 64..127: k_t.k_i           tcgen05
//       P_ti = Gam_ti q_t.k_i (i <= t),  A_ti = beta_t Gam_ti k_t.k_i (i < t)             out warps
//       M    = (I + A)^{-1}          (UT transform: 16x16 diagonal blocks by substitution in fp32,
//                                     off-diagonal blocks by tf32 block products)         prep warps
//   (6) PM   = P M                                                                        tcgen05
//   (2) D1   = S^T [Q;K]^T           cols 0..63: (S^T q_t)_j, cols 64..127: (S^T k_t)_j    tcgen05
//       r_t  = beta_t (v_t - gam_t S^T k_t)                                               chain warps
//   (3) [U^T | (PU)^T] = R^T [M; PM]^T   u = M r solves the block's triangular system     tcgen05
//       o_t  = scale (gam_t S^T q_t + (P u)_t)                                            out warps
//   (5) S^T <- gam_C S^T + (U o w)^T K   fp32 state accumulated in TMEM (pre-scaled there) tcgen05
//       and a bf16 copy of S^T in shared memory is the A operand of (2) for the next block.
// The prep warps (cumulative decay, the inverse, the bf16 [M; PM] operand) and the mask epilogue of (1)
// work one block ahead of the chain, so (1), the inverse and (6) are off the block-to-block chain
// (2) -> r -> (3) -> U o w -> (5) -> state copy.
// A padded token (beyond the sequence end) has g = 0 and beta = 0: the identity step.
// Warps 0-7 chain (lane = state column, warpgroup = half of the tokens / state rows), 8-11 out,
// 12-15 prep (the inverse), 16 TMA loads and the store of the output tile, 17 MMA issue of the chain ((2), (3), (5)),
// 18 MMA issue of the prep side ((1), (6)), 19 per-block scalars
// (running up to three blocks ahead).  All waits on mbarriers are bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kD = 128;   // d_k = d_v
constexpr int kC = 64;    // tokens per block
constexpr int kThreads = 640;

// shared-memory map (bytes, after 1024-byte alignment)
constexpr int kQKStage = 4 * kC * 128;                 // [Q_kb0 | K_kb0 | Q_kb1 | K_kb1], each [64 rows x 128 B]
constexpr int kOffV = 2 * kQKStage;                    // V tile [64][128] bf16, row-major (single buffer)
constexpr int kOffSt = kOffV + kC * kD * 2;            // S^T bf16: [St_kb0 | St_kb1], each [128 rows x 128 B]
constexpr int kOffR = kOffSt + 2 * kD * 128;           // R^T bf16 [128 rows x 128 B]
constexpr int kOffUw = kOffR;                          // (U o w)^T bf16: written only after (3) has consumed R^T
constexpr int kOffMPM = kOffR + kD * 128;              // [M; PM] bf16 [128 rows x 128 B], double-buffered; once (3) has read it,
                                                       // the buffer stages the block's output tile [64 tokens][128] bf16 for the TMA store
constexpr int kOffP = kOffMPM + 2 * kD * 128;          // P bf16 [64 rows x 128 B] = rows 64..127 of the A operand of (6), whose rows
                                                       // 0..63 (the end of the [M; PM] buffers) are don't-care: PM lands in TMEM lanes 64..127
constexpr int kLd = 68;                                // row stride (floats) of the fp32 A and M matrices: rows 4 banks apart
constexpr int kOffA = kOffP + kC * 128;                // A fp32 [t][i], double-buffered
constexpr int kOffM = kOffA + 2 * kC * kLd * 4;        // M fp32 [t][i]
constexpr int kOffGb = kOffM + kC * kLd * 4;           // per-block scalars, four buffers (prepared two blocks ahead)
constexpr int kGbFloats = 5 * kC + 4;                  // cg2 = cg log2(e), beta, gam (e^{cg}), w (e^{cg_C - cg}), f (e^{cg_ref - cg}), flag
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxGroupRange = 100.f;                // log2 units: above this the per-group factors could overflow
constexpr int kSmemUsed = kOffGb + 4 * kGbFloats * 4;   // from the 1024-byte aligned base
static_assert(kSmemUsed + 1024 <= 227 * 1024, "shared memory budget");

// tensor-memory map (columns)
constexpr uint32_t kTmG = 0;      // 64
constexpr uint32_t kTmPM = 448;   // 64
constexpr uint32_t kTmD1 = 64;    // 128: QS | KS
constexpr uint32_t kTmUP = 192;   // 128: U | PU
constexpr uint32_t kTmS = 320;    // 128
constexpr uint32_t kTmemCols = 512;

struct Bars {
    // single-arrival barriers: TMA transactions and tcgen05.commit
    uint64_t full_qk[2], tiles_free_qk[2], full_v, g_done, pm_done, d1_done, up_done, ds_done, o_free[2];
    // 128-thread barriers (prep or out warpgroup)
    uint64_t m_ready[2], o_done[4], inv_done[2], o_staged[2];
    // 64-thread barriers (the two halves of the out warpgroup)
    uint64_t a_ready, p_ready, gb_ready[4], mpm_ready[2];
    // 256-thread barriers (both chain warpgroups)
    uint64_t v_free, r_ready, uw_ready, st_ready, chain_done[4];
};

__device__ __forceinline__ uint32_t to_tf32(float v) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return r;
}
// acc[16 x 8] += A[16 x 8] B[8 x 8] on the warp-level MMA; fragments as the PTX ISA lays them out
// (row = lane / 4 (+8), column = lane % 4 (+4) for A; k = lane % 4 (+4), n = lane / 4 for B; row = lane / 4 (+8),
// columns 2 (lane % 4), +1 for the accumulator).
__device__ __forceinline__ void mma_tf32_16x8x8(float (&acc)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One off-diagonal block (r = c + D, c) of M = (I + A)^{-1}, or NH = 1 half of it (8 columns from 8 nh0):
// X = sum_{m=c}^{r-1} A_rm M_mc, M_rc = -D_r X with D_r the inverted diagonal block.  tf32 operands rounded to
// nearest, fp32 accumulation.  Every MMA of a stage has its own accumulator, so they are all in flight together
// (the warp-level MMA has a long latency here); X passes through the unused block (c, r) above the diagonal to
// change from accumulator to operand layout.  A, M: fp32 [64][ld].
template <int NH, int D>
__device__ __forceinline__ void inv_offdiag(const float *Af, float *Mf, int c, int nh0, int gid, int tig) {
    constexpr int ld = kLd;
    const int r = c + D;
    float part[D][2][NH][4];
#pragma unroll
    for (int mm = 0; mm < D; ++mm) {
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
            const float *ap = Af + (16 * r + gid) * ld + 16 * (c + mm) + 8 * ks + tig;
            const uint32_t a0 = to_tf32(ap[0]), a1 = to_tf32(ap[8 * ld]), a2 = to_tf32(ap[4]), a3 = to_tf32(ap[8 * ld + 4]);
#pragma unroll
            for (int hh = 0; hh < NH; ++hh) {
                const float *bp = Mf + (16 * (c + mm) + 8 * ks + tig) * ld + 16 * c + 8 * (nh0 + hh) + gid;
#pragma unroll
                for (int i = 0; i < 4; ++i) part[mm][ks][hh][i] = 0.f;
                mma_tf32_16x8x8(part[mm][ks][hh], a0, a1, a2, a3, to_tf32(bp[0]), to_tf32(bp[4 * ld]));
            }
        }
    }
    float *xs = Mf + (16 * c) * ld + 16 * r + 8 * nh0;
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
        float x[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int mm = 0; mm < D; ++mm)
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)
#pragma unroll
                for (int i = 0; i < 4; ++i) x[i] += part[mm][ks][hh][i];
        *reinterpret_cast<float2 *>(xs + 8 * hh + gid * ld + 2 * tig) = make_float2(x[0], x[1]);
        *reinterpret_cast<float2 *>(xs + 8 * hh + (gid + 8) * ld + 2 * tig) = make_float2(x[2], x[3]);
    }
    __syncwarp();
    float out[2][NH][4];
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
        const float *dp = Mf + (16 * r + gid) * ld + 16 * r + 8 * ks + tig;
        const uint32_t a0 = to_tf32(dp[0]), a1 = to_tf32(dp[8 * ld]), a2 = to_tf32(dp[4]), a3 = to_tf32(dp[8 * ld + 4]);
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
            const float *xp = xs + 8 * hh + (8 * ks + tig) * ld + gid;
#pragma unroll
            for (int i = 0; i < 4; ++i) out[ks][hh][i] = 0.f;
            mma_tf32_16x8x8(out[ks][hh], a0, a1, a2, a3, to_tf32(xp[0]), to_tf32(xp[4 * ld]));
        }
    }
#pragma unroll
    for (int hh = 0; hh < NH; ++hh) {
        float *mp = Mf + (16 * r + gid) * ld + 16 * c + 8 * (nh0 + hh) + 2 * tig;
        *reinterpret_cast<float2 *>(mp) = make_float2(-(out[0][hh][0] + out[1][hh][0]), -(out[0][hh][1] + out[1][hh][1]));
        *reinterpret_cast<float2 *>(mp + 8 * ld) = make_float2(-(out[0][hh][2] + out[1][hh][2]), -(out[0][hh][3] + out[1][hh][3]));
    }
}
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
// 16 consecutive fp32 values -> bf16, written as 2 swizzled 16-byte chunks (chunk0, chunk0+1) of operand row `row`
__device__ __forceinline__ void store_row_chunks(unsigned char *tile, int row, int chunk0, const float (&v)[16]) {
#pragma unroll
    for (int c8 = 0; c8 < 2; ++c8) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = pack_bf16(v[8 * c8 + 2 * e], v[8 * c8 + 2 * e + 1]);
        *reinterpret_cast<uint4 *>(tile + sw128_offset(row, chunk0 + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__global__ void __launch_bounds__(kThreads, 1)
gdn_scan_tensor_kernel(const __grid_constant__ GdnArgs a, const __grid_constant__ CUtensorMap mapQ,
                       const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                       const __grid_constant__ CUtensorMap mapO) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Bars bars;
    __shared__ uint32_t tmem_base;
    __shared__ int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, seq = blockIdx.y;
    {
        // the launch asks for all the dynamic shared memory the device has left; make sure the aligned map fits
        uint32_t dyn;
        asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
        if (static_cast<uint32_t>(sm - smem_raw) + kSmemUsed > dyn) {
            if (tid == 0 && a.status) atomicExch(a.status, 1);
            return;
        }
    }
    const int hk = h / (a.H_v / a.H_k);
    const int t_begin = a.cu[seq], t_end = a.cu[seq + 1];
    const int nblk = (t_end - t_begin + kC - 1) / kC;
    const size_t sbase = (static_cast<size_t>(seq) * a.H_v + h) * kD * kD;

    if (nblk == 0) {  // empty sequence: hand the state through untouched
        if (a.S_T && (a.S_T != a.S0 || a.s0_identity))
            for (int e = tid; e < kD * kD; e += kThreads)
                a.S_T[sbase + e] = a.s0_identity ? (e / kD == e % kD ? 1.f : 0.f) : (a.S0 ? a.S0[sbase + e] : 0.f);
        return;
    }
    if (tid == 0) {
        dead = 0;
        uint64_t *b1 = &bars.full_qk[0];
        for (int i = 0; i < 12; ++i) mbar_init(b1 + i, 1);
        uint64_t *b128 = &bars.m_ready[0];
        for (int i = 0; i < 10; ++i) mbar_init(b128 + i, 128);
        uint64_t *b64 = &bars.a_ready;
        for (int i = 0; i < 8; ++i) mbar_init(b64 + i, (i >= 2 && i < 6) ? 32 : 64);   // gb_ready: the scalar warp
        uint64_t *b256 = &bars.v_free;
        for (int i = 0; i < 8; ++i) mbar_init(b256 + i, 256);
        mbar_fence_init();
    }
    if (warp == 17) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    float *gb = reinterpret_cast<float *>(sm + kOffGb);

    if (warp == 16) {
        // ======================================================= TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapK);
            if (a.v) tma_prefetch_desc(&mapV);
            if (a.o) tma_prefetch_desc(&mapO);
            // the output tile of block b (whole blocks only) leaves its staging buffer, the [M; PM] buffer of parity b
            auto store_o = [&](int b) {
                mbar_wait(&bars.o_staged[b & 1], (b >> 1) & 1, &dead, a.status);
                const int t0 = t_begin + b * kC;
                if (a.o && t0 + kC <= t_end && !dead) {
                    tma_store_2d(&mapO, sm + kOffMPM + (b & 1) * (kD * 128), h * kD, t0);
                    tma_store_commit();
                    tma_store_wait_read();
                }
                mbar_arrive(&bars.o_free[b & 1]);
            };
            for (int b = 0; b < nblk; ++b) {
                const int st = b & 1;
                const int row = t_begin + b * kC;
                // the two-stage ring cannot hide the DRAM latency of the tile loads: pull the tiles of block b+2 into L2 now
                if (b + 2 < nblk) {
                    for (int kb = 0; kb < 2; ++kb) {
                        tma_prefetch_l2_2d(&mapQ, hk * kD + kb * 64, row + 2 * kC);
                        tma_prefetch_l2_2d(&mapK, hk * kD + kb * 64, row + 2 * kC);
                    }
                    if (a.v) tma_prefetch_l2_2d(&mapV, h * kD, row + 2 * kC);
                }
                if (b >= 2) mbar_wait(&bars.tiles_free_qk[st], ((b - 2) >> 1) & 1, &dead, a.status);
                unsigned char *base = sm + st * kQKStage;
                mbar_expect_tx(&bars.full_qk[st], kQKStage);
                for (int kb = 0; kb < 2; ++kb) {
                    tma_load_2d(base + kb * 2 * kC * 128, &mapQ, hk * kD + kb * 64, row, &bars.full_qk[st]);
                    tma_load_2d(base + kb * 2 * kC * 128 + kC * 128, &mapK, hk * kD + kb * 64, row, &bars.full_qk[st]);
                }
                if (a.v) {   // without v (read as zeros) nothing is loaded and the chain does not wait for it
                    if (b >= 1) mbar_wait(&bars.v_free, (b - 1) & 1, &dead, a.status);
                    mbar_expect_tx(&bars.full_v, kC * kD * 2);
                    tma_load_2d(sm + kOffV, &mapV, h * kD, row, &bars.full_v);
                }
                // the output of block b-2 was staged about one block ago; the inverse of block b needs its buffer only later
                if (b >= 2) store_o(b - 2);
            }
            if (nblk >= 2) store_o(nblk - 2);
            store_o(nblk - 1);
            tma_store_wait_all();
        }
    } else if (warp == 19) {
        // ======================================================= scalar warp: lane = tokens 2 lane, 2 lane + 1 of the block
        auto fetch_gb = [&](int b, float2 &gv, float2 &bv) {
            const int t = t_begin + b * kC + 2 * lane;
            gv = make_float2(0.f, 0.f); bv = make_float2(0.f, 0.f);
            if (b < nblk && t < t_end) {
                gv.x = a.g[static_cast<size_t>(t) * a.H_v + h];
                bv.x = a.beta[static_cast<size_t>(t) * a.H_v + h];
            }
            if (b < nblk && t + 1 < t_end) {
                gv.y = a.g[static_cast<size_t>(t + 1) * a.H_v + h];
                bv.y = a.beta[static_cast<size_t>(t + 1) * a.H_v + h];
            }
        };
        float2 gv_next, bv_next;
        fetch_gb(0, gv_next, bv_next);
        for (int b = 0; b < nblk; ++b) {
            // the buffer of block b was last read by the chain and the output epilogue of block b-4
            if (b >= 4) {
                mbar_wait(&bars.chain_done[b & 3], ((b - 4) >> 2) & 1, &dead, a.status);
                mbar_wait(&bars.o_done[b & 3], ((b - 4) >> 2) & 1, &dead, a.status);
            }
            // ---- per-block scalars: cg (in log2 units), beta, gam = e^{cg}, w = e^{cg_C - cg}, group factors
            float *sc = gb + (b & 3) * kGbFloats;
            const float2 gv = gv_next, bv = bv_next;
            fetch_gb(b + 1, gv_next, bv_next);   // in flight while this block is prepared
            const float pair = gv.x + gv.y;
            float run = pair;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float up = __shfl_up_sync(0xffffffffu, run, o);
                if (lane >= o) run += up;
            }
            const float c0 = (run - gv.y) * kLog2e, c1 = run * kLog2e;
            const float last = __shfl_sync(0xffffffffu, c1, 31);
            // first column of each group of 16 tokens = first token of lanes 0, 8, 16, 24
            const float ref = __shfl_sync(0xffffffffu, c0, lane & ~7);
            const float r0 = ref - c0, r1 = ref - c1;
            const int t = 2 * lane;
            *reinterpret_cast<float2 *>(sc + t) = make_float2(c0, c1);
            *reinterpret_cast<float2 *>(sc + kC + t) = bv;
            *reinterpret_cast<float2 *>(sc + 2 * kC + t) = make_float2(exp2f(c0), exp2f(c1));
            *reinterpret_cast<float2 *>(sc + 3 * kC + t) = make_float2(exp2f(last - c0), exp2f(last - c1));
            // factor of a column relative to the first column of its group (>= 1)
            *reinterpret_cast<float2 *>(sc + 4 * kC + t) = make_float2(exp2f(fminf(r0, 126.f)), exp2f(fminf(r1, 126.f)));
            const unsigned bad = __ballot_sync(0xffffffffu, r0 > kMaxGroupRange || r1 > kMaxGroupRange);
            if (lane == 0) *reinterpret_cast<float2 *>(sc + 5 * kC) = make_float2(bad ? 1.f : 0.f, 0.f);
            mbar_arrive(&bars.gb_ready[b & 3]);
        }
    } else if (warp == 18) {
        // ======================================================= second MMA issuer: (1) and (6), the prep side
        if (elect_one()) {
            constexpr uint32_t idG = umma_idesc(kFmtBF16, false, false, 128, 64);    // (1)
            constexpr uint32_t idPM = umma_idesc(kFmtBF16, false, true, 128, 64);    // (6): B = M read MN-major
            const uint64_t dP = umma_desc(smem_u32(sm + kOffP - kC * 128), 0, 1024);
            const uint64_t dMPM0 = umma_desc(smem_u32(sm + kOffMPM), 0, 1024);
            auto issue_G = [&](int b) {
                const uint64_t dQK = umma_desc(smem_u32(sm + (b & 1) * kQKStage), 0, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t off = ((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmG, dQK + off, dQK + off + ((kC * 128) >> 4), idG, k > 0);
                }
                umma_commit(&bars.g_done);
            };
            mbar_wait(&bars.full_qk[0], 0, &dead, a.status);
            tc_fence_after_sync();
            issue_G(0);
            for (int b = 0; b < nblk; ++b) {
                const uint32_t par = b & 1;
                // (1) of the next block as soon as the mask epilogue of this one has drained the G columns
                if (b + 1 < nblk) {
                    mbar_wait(&bars.a_ready, par, &dead, a.status);
                    mbar_wait(&bars.p_ready, par, &dead, a.status);
                    mbar_wait(&bars.full_qk[(b + 1) & 1], ((b + 1) >> 1) & 1, &dead, a.status);
                    tc_fence_after_sync();
                    issue_G(b + 1);
                }
                // (6) of this block as soon as its inverse is there: PM = P M, A = P (K = i), B = M rows of [M; PM] read MN-major
                mbar_wait(&bars.m_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                mbar_wait(&bars.p_ready, par, &dead, a.status);
                // the accumulator of (6) must have been read for block b-1 (its PM rows are in the operand)
                if (b >= 1) mbar_wait(&bars.mpm_ready[(b - 1) & 1], ((b - 1) >> 1) & 1, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dM = dMPM0 + ((b & 1) * ((kD * 128) >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmPM, dP + 2 * k, dM + ((k * 16 * 128) >> 4), idPM, k > 0);
                umma_commit(&bars.pm_done);
            }
        }
    } else if (warp == 17) {
        // ======================================================= first MMA issuer: (2), (3), (5), the block-to-block chain
        if (elect_one()) {
            constexpr uint32_t idD1 = umma_idesc(kFmtBF16, false, false, 128, 128);  // (2), (3)
            constexpr uint32_t idDS = umma_idesc(kFmtBF16, false, true, 128, 128);   // (5): B = K tile read MN-major
            const uint64_t dSt = umma_desc(smem_u32(sm + kOffSt), 0, 1024);
            const uint64_t dR = umma_desc(smem_u32(sm + kOffR), 0, 1024);
            const uint64_t dUw = umma_desc(smem_u32(sm + kOffUw), 0, 1024);
            const uint64_t dMPM0 = umma_desc(smem_u32(sm + kOffMPM), 0, 1024);
            for (int b = 0; b < nblk; ++b) {
                const uint32_t par = b & 1;
                const uint64_t dQK = umma_desc(smem_u32(sm + (b & 1) * kQKStage), 0, 1024);
                // (2) needs the bf16 state copy of block b, the D1 / UP accumulators drained, and the Q / K tiles
                mbar_wait(&bars.st_ready, par, &dead, a.status);
                if (b > 0) mbar_wait(&bars.o_done[(b - 1) & 3], ((b - 1) >> 2) & 1, &dead, a.status);
                mbar_wait(&bars.full_qk[b & 1], (b >> 1) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t offA = ((k >> 2) * (kD * 128) + (k & 3) * 32) >> 4;
                    const uint64_t offB = ((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmD1, dSt + offA, dQK + offB, idD1, k > 0);
                }
                umma_commit(&bars.d1_done);
                // (3) [U | PU] = R^T [M; PM]^T
                mbar_wait(&bars.mpm_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                mbar_wait(&bars.r_ready, par, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dMPM = dMPM0 + ((b & 1) * ((kD * 128) >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmUP, dR + 2 * k, dMPM + 2 * k, idD1, k > 0);
                umma_commit(&bars.up_done);
                // (5) accumulates onto the pre-scaled state; B = K tile read MN-major (rows = tokens)
                mbar_wait(&bars.uw_ready, par, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dKmn = umma_desc(smem_u32(sm + (b & 1) * kQKStage + kC * 128), 2 * kC * 128, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmS, dUw + 2 * k, dKmn + ((k * 16 * 128) >> 4), idDS, true);
                umma_commit(&bars.ds_done);
                umma_commit(&bars.tiles_free_qk[b & 1]);
            }
        }
    } else if (warp >= 12) {
        // ======================================================= prep warpgroup: the inverse, ahead of the chain
        const int x = tid - 384;                 // 0..127
        float *Mf = reinterpret_cast<float *>(sm + kOffM);
        for (int b = 0; b < nblk; ++b) {
            // ---- P and A come from the out warpgroup (epilogue of (1))
            mbar_wait(&bars.a_ready, b & 1, &dead, a.status);
            named_bar_sync(1, 128);   // every thread is done with the fp32 M of the previous block
            const float *Af = reinterpret_cast<const float *>(sm + kOffA) + (b & 1) * (kC * kLd);
            // ---- M = (I + A)^{-1}.  Diagonal 16x16 blocks: thread (k, c) solves column c of block k by forward
            // substitution; each row of the block is fetched with four 16-byte loads ahead of its use.
            if (x < kC) {
                const int k = x >> 4, c = x & 15;
                const float *Ab = Af + (16 * k) * kLd + 16 * k;
                float xv[16];
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    float row[16];
#pragma unroll
                    for (int i4 = 0; i4 < 16; i4 += 4) {
                        if (i4 < t) {
                            const float4 v = *reinterpret_cast<const float4 *>(Ab + t * kLd + i4);
                            row[i4] = v.x; row[i4 + 1] = v.y; row[i4 + 2] = v.z; row[i4 + 3] = v.w;
                        }
                    }
                    float acc0 = (t == c) ? 1.f : 0.f, acc1 = 0.f;
#pragma unroll
                    for (int i = 0; i < t; ++i) {
                        if (i & 1) acc1 = fmaf(-row[i], xv[i], acc1);
                        else acc0 = fmaf(-row[i], xv[i], acc0);
                    }
                    xv[t] = (t >= c) ? acc0 + acc1 : 0.f;
                }
#pragma unroll
                for (int t = 0; t < 16; ++t) Mf[(16 * k + t) * kLd + 16 * k + c] = xv[t];
            }
            named_bar_sync(1, 128);
            // Off-diagonal blocks by distance d from the diagonal, M_rc = -D_r sum_{m=c}^{r-1} A_rm M_mc, on the
            // warp-level tensor-core MMA; one warp per block (d = 1) or half block (d = 2, 3).
            {
                const int wq = warp & 3, gid = lane >> 2, tig = lane & 3;
                if (wq < 3) inv_offdiag<2, 1>(Af, Mf, wq, 0, gid, tig);
                named_bar_sync(1, 128);
                inv_offdiag<1, 2>(Af, Mf, wq >> 1, wq & 1, gid, tig);
                named_bar_sync(1, 128);
                if (wq < 2) inv_offdiag<1, 3>(Af, Mf, 0, wq, gid, tig);
                named_bar_sync(1, 128);
            }
            // ---- M as bf16 operand rows 0..63 of [M; PM] (zeros above the block diagonal)
            // the [M; PM] buffer of this parity was read by (3) of block b-2 and then staged that block's output tile
            if (b >= 2) mbar_wait(&bars.o_free[b & 1], ((b - 2) >> 1) & 1, &dead, a.status);
            unsigned char *mpm = sm + kOffMPM + (b & 1) * (kD * 128);
            {
                // thread = (row t, half of the columns)
                const int t = x & 63, q0 = 2 * (x >> 6);
#pragma unroll
                for (int q = q0; q < q0 + 2; ++q) {
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; c += 4) {
                        const int i = 16 * q + c;
                        const float4 mv = (i >> 4) <= (t >> 4) ? *reinterpret_cast<const float4 *>(Mf + t * kLd + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                        v[c] = mv.x; v[c + 1] = mv.y; v[c + 2] = mv.z; v[c + 3] = mv.w;
                    }
                    store_row_chunks(mpm, t, 2 * q, v);
                }
            }
            fence_async_smem();
            mbar_arrive(&bars.m_ready[b & 1]);
            mbar_arrive(&bars.inv_done[b & 1]);
        }
    } else if (warp >= 8) {
        // ======================================================= out warpgroup: o_t[j] = scale (gam_t (S^T q_t)_j + (P u)_t[j]); lane = j
        const int j = tid - 256;
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(a.o);
        const size_t tstride = static_cast<size_t>(a.H_v) * kD;
        const int x = j;   // TMEM lane: 0..63 rows of Q K^T (-> P), 64..127 rows of K K^T (-> A)
        // epilogue of (1) for block b: P (bf16 operand of (6)) and A (fp32, input of the inverse)
        // PM rows of block b (lanes 64..127 of the (6) accumulator) -> rows 64..127 of [M; PM]; warps 10 and 11 only,
        // so that the P rows of the next block (warps 8 and 9) are worked on at the same time
        auto pm_rows = [&](int b) {
            mbar_wait(&bars.pm_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            unsigned char *mpm = sm + kOffMPM + (b & 1) * (kD * 128);
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                uint32_t rr[16];
                tmem_ld16(lane_base + kTmPM + 16 * q, rr);
                tmem_ld_wait();
                float v[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = __uint_as_float(rr[c]);
                store_row_chunks(mpm, x, 2 * q, v);
            }
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.mpm_ready[b & 1]);
        };
        auto g_epilogue = [&](int b) {
            const float *sc = gb + (b & 3) * kGbFloats;
            mbar_wait(&bars.gb_ready[b & 3], (b >> 2) & 1, &dead, a.status);
            float *Af = reinterpret_cast<float *>(sm + kOffA) + (b & 1) * (kC * kLd);
            bool pm_pending = x >= kC && b >= 1;
            if (x < kC) {
                // the P buffer is free once (6) of block b-1 has read it
                if (b >= 1) mbar_wait(&bars.pm_done, (b - 1) & 1, &dead, a.status);
            } else {
                // the A buffer of this parity is free once block b-2 has been inverted
                if (b >= 2) mbar_wait(&bars.inv_done[b & 1], ((b - 2) >> 1) & 1, &dead, a.status);
                // the result of (6) of block b-1 is on the chain's critical path: take it first if it is there already
                if (pm_pending && __all_sync(0xffffffffu, mbar_test_wait(&bars.pm_done, (b - 1) & 1))) {
                    pm_rows(b - 1);
                    pm_pending = false;
                }
            }
            mbar_wait(&bars.g_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            {
                // Gam_ti = 2^{cg2_t - cg2_ref} * f_i with ref the first column of i's group of 16: one exponential
                // per group (both factors' product is <= 1 where i <= t); violent decay takes the per-element path
                const int t = x & 63;
                const float cgt = sc[t];
                const float coef = (x < kC) ? 1.f : sc[kC + t];     // rows of P: 1, rows of A: beta_t
                const int lim = (x < kC) ? t : t - 1;               // P keeps the diagonal, A is strictly lower
                const bool fast = sc[5 * kC] + sc[5 * kC + 1] == 0.f;
                const int row_hi = (t & 32) + 31;   // last row (token) of this warp
#pragma unroll 1
                for (int q = 0; q < 4; ++q) {
                    const int i0 = 16 * q;
                    if (i0 > row_hi) break;   // above the diagonal for every row of this warp: zeroed once, never written
                    uint32_t rr[16];
                    tmem_ld16(lane_base + kTmG + 16 * q, rr);
                    tmem_ld_wait();
                    float v[16];
                    if (fast) {
                        float aa;
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(aa) : "f"(fminf(cgt - sc[i0], 0.f)));
                        aa *= coef;
                        if (i0 + 15 <= row_hi - 32) {
                            // below the diagonal for every row of this warp: no masking
#pragma unroll
                            for (int c = 0; c < 16; c += 4) {
                                const float4 f = *reinterpret_cast<const float4 *>(sc + 4 * kC + i0 + c);
                                v[c] = __uint_as_float(rr[c]) * aa * f.x;
                                v[c + 1] = __uint_as_float(rr[c + 1]) * aa * f.y;
                                v[c + 2] = __uint_as_float(rr[c + 2]) * aa * f.z;
                                v[c + 3] = __uint_as_float(rr[c + 3]) * aa * f.w;
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; c += 4) {
                                const float4 f = *reinterpret_cast<const float4 *>(sc + 4 * kC + i0 + c);
                                v[c] = (i0 + c <= lim) ? __uint_as_float(rr[c]) * aa * f.x : 0.f;
                                v[c + 1] = (i0 + c + 1 <= lim) ? __uint_as_float(rr[c + 1]) * aa * f.y : 0.f;
                                v[c + 2] = (i0 + c + 2 <= lim) ? __uint_as_float(rr[c + 2]) * aa * f.z : 0.f;
                                v[c + 3] = (i0 + c + 3 <= lim) ? __uint_as_float(rr[c + 3]) * aa * f.w : 0.f;
                            }
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            v[c] = (i0 + c <= lim) ? coef * exp2f(cgt - sc[i0 + c]) * __uint_as_float(rr[c]) : 0.f;
                    }
                    if (x < kC) {
                        store_row_chunks(sm + kOffP, t, 2 * q, v);
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; c += 4)
                            *reinterpret_cast<float4 *>(Af + t * kLd + 16 * q + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                    }
                }
            }
            tc_fence_before_sync();
            if (x < kC) {
                fence_async_smem();
                mbar_arrive(&bars.p_ready);
            } else {
                mbar_arrive(&bars.a_ready);
            }
            if (pm_pending) pm_rows(b - 1);
        };
        if ((x & 32) == 0) {
            // columns 32..63 of rows 0..31 lie above the diagonal in P and in both A buffers: zero them once
            const int t = x & 63;
            float z[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) z[c] = 0.f;
            for (int q = 2; q < 4; ++q) {
                if (x < kC) {
                    store_row_chunks(sm + kOffP, t, 2 * q, z);
                } else {
                    for (int bufi = 0; bufi < 2; ++bufi)
                        for (int c = 0; c < 16; c += 4)
                            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(sm + kOffA) + bufi * (kC * kLd) + t * kLd + 16 * q + c) =
                                make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        g_epilogue(0);
        for (int b = 0; b < nblk; ++b) {
            if (b + 1 < nblk) g_epilogue(b + 1);   // while the chain works on block b
            else if (x >= kC) pm_rows(b);
            const float *sc = gb + (b & 3) * kGbFloats;
            mbar_wait(&bars.d1_done, b & 1, &dead, a.status);
            mbar_wait(&bars.up_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            const int t0 = t_begin + b * kC;
            const int n = min(kC, t_end - t0);
            if (!a.o) {
                // no outputs wanted (final state only): nothing to drain
            } else if (n == kC) {
                // whole block: stage the tile [token][j] in the [M; PM] buffer of this block, which (3) has finished
                // reading (up_done); the store warp writes it out with TMA
                __nv_bfloat16 *os = reinterpret_cast<__nv_bfloat16 *>(sm + kOffMPM + (b & 1) * (kD * 128)) + j;
#pragma unroll 1
                for (int q = 0; q < 8; ++q) {
                    uint32_t qs[8], pu[8];
                    tmem_ld8(lane_base + kTmD1 + 8 * q, qs);
                    tmem_ld8(lane_base + kTmUP + kC + 8 * q, pu);
                    tmem_ld_wait();
                    const float4 g0 = *reinterpret_cast<const float4 *>(sc + 2 * kC + 8 * q);
                    const float4 g1 = *reinterpret_cast<const float4 *>(sc + 2 * kC + 8 * q + 4);
                    const float gm[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        os[(8 * q + c) * kD] = __float2bfloat16_rn(a.scale * fmaf(gm[c], __uint_as_float(qs[c]), __uint_as_float(pu[c])));
                }
                fence_async_smem();
            } else {
                __nv_bfloat16 *orow = o + (static_cast<size_t>(t0) * a.H_v + h) * kD + j;
#pragma unroll 1
                for (int q = 0; q < 8; ++q) {
                    uint32_t qs[8], pu[8];
                    tmem_ld8(lane_base + kTmD1 + 8 * q, qs);
                    tmem_ld8(lane_base + kTmUP + kC + 8 * q, pu);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int t = 8 * q + c;
                        const float val = a.scale * fmaf(sc[2 * kC + t], __uint_as_float(qs[c]), __uint_as_float(pu[c]));
                        if (t < n) orow[t * tstride] = __float2bfloat16_rn(val);
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bars.o_done[b & 3]);
            mbar_arrive(&bars.o_staged[b & 1]);
        }
    } else {
        // ======================================================= chain warpgroups: lane = state column j, `half` = token / row half
        const int j = tid & 127, half = warp >> 2;
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // initial state: S0[m][j], m = 64*half..+63 -> TMEM (fp32, pre-scaled by gam_C of block 0) and bf16 copy
        mbar_wait(&bars.gb_ready[0], 0, &dead, a.status);
        {
            const float gamC = gb[2 * kC + kC - 1];
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                float v[16];
                uint32_t rr[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int m = 64 * half + 16 * q + c;
                    v[c] = a.s0_identity ? (m == j ? 1.f : 0.f) : (a.S0 ? a.S0[sbase + static_cast<size_t>(m) * kD + j] : 0.f);
                    rr[c] = __float_as_uint(v[c] * gamC);
                }
                tmem_st16(lane_base + kTmS + 64 * half + 16 * q, rr);
                store_row_chunks(sm + kOffSt + half * (kD * 128), j, 2 * q, v);
            }
            tmem_st_wait();
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.st_ready);
        }
        for (int b = 0; b < nblk; ++b) {
            const uint32_t par = b & 1;
            const float *sc = gb + (b & 3) * kGbFloats;
            const __nv_bfloat16 *vt = reinterpret_cast<const __nv_bfloat16 *>(sm + kOffV);
            if (b > 0) mbar_wait(&bars.gb_ready[b & 3], (b >> 2) & 1, &dead, a.status);
            const bool has_v = a.v != nullptr;
            if (has_v) mbar_wait(&bars.full_v, par, &dead, a.status);
            mbar_wait(&bars.d1_done, par, &dead, a.status);
            tc_fence_after_sync();
            // r_t = beta_t (v_t[j] - gam_t (S^T k_t)_j), t = 32*half..+31 -> R^T row j
#pragma unroll 1
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[16];
                tmem_ld16(lane_base + kTmD1 + kC + 32 * half + 16 * q, rr);
                tmem_ld_wait();
                float v[16];
#pragma unroll
                for (int c = 0; c < 16; c += 4) {
                    const int t = 32 * half + 16 * q + c;
                    const float4 be = *reinterpret_cast<const float4 *>(sc + kC + t);
                    const float4 ga = *reinterpret_cast<const float4 *>(sc + 2 * kC + t);
                    const float v0 = has_v ? __bfloat162float(vt[t * kD + j]) : 0.f;
                    const float v1 = has_v ? __bfloat162float(vt[(t + 1) * kD + j]) : 0.f;
                    const float v2 = has_v ? __bfloat162float(vt[(t + 2) * kD + j]) : 0.f;
                    const float v3 = has_v ? __bfloat162float(vt[(t + 3) * kD + j]) : 0.f;
                    v[c] = be.x * (v0 - ga.x * __uint_as_float(rr[c]));
                    v[c + 1] = be.y * (v1 - ga.y * __uint_as_float(rr[c + 1]));
                    v[c + 2] = be.z * (v2 - ga.z * __uint_as_float(rr[c + 2]));
                    v[c + 3] = be.w * (v3 - ga.w * __uint_as_float(rr[c + 3]));
                }
                store_row_chunks(sm + kOffR, j, 4 * half + 2 * q, v);
            }
            mbar_arrive(&bars.v_free);
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.r_ready);
            // (U o w)^T row j, i = 32*half..+31
            mbar_wait(&bars.up_done, par, &dead, a.status);
            tc_fence_after_sync();
#pragma unroll 1
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[16];
                tmem_ld16(lane_base + kTmUP + 32 * half + 16 * q, rr);
                tmem_ld_wait();
                float v[16];
#pragma unroll
                for (int c = 0; c < 16; c += 4) {
                    const float4 w4 = *reinterpret_cast<const float4 *>(sc + 3 * kC + 32 * half + 16 * q + c);
                    v[c] = __uint_as_float(rr[c]) * w4.x;
                    v[c + 1] = __uint_as_float(rr[c + 1]) * w4.y;
                    v[c + 2] = __uint_as_float(rr[c + 2]) * w4.z;
                    v[c + 3] = __uint_as_float(rr[c + 3]) * w4.w;
                }
                store_row_chunks(sm + kOffUw, j, 4 * half + 2 * q, v);
            }
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.uw_ready);
            // new state rows m = 64*half..+63: bf16 copy for the next block and pre-scale by its gam_C, or S_T at the end
            mbar_wait(&bars.ds_done, par, &dead, a.status);
            tc_fence_after_sync();
            const bool last = b + 1 == nblk;
            float gamN = 1.f;
            if (!last) {
                mbar_wait(&bars.gb_ready[(b + 1) & 3], ((b + 1) >> 2) & 1, &dead, a.status);
                gamN = gb[((b + 1) & 3) * kGbFloats + 2 * kC + kC - 1];
            }
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                uint32_t rr[16];
                tmem_ld16(lane_base + kTmS + 64 * half + 16 * q, rr);
                tmem_ld_wait();
                if (last) {
                    if (a.S_T) {
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            a.S_T[sbase + static_cast<size_t>(64 * half + 16 * q + c) * kD + j] = __uint_as_float(rr[c]);
                    }
                } else {
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        v[c] = __uint_as_float(rr[c]);
                        rr[c] = __float_as_uint(v[c] * gamN);
                    }
                    tmem_st16(lane_base + kTmS + 64 * half + 16 * q, rr);
                    store_row_chunks(sm + kOffSt + half * (kD * 128), j, 2 * q, v);
                }
            }
            if (!last) {
                tmem_st_wait();
                fence_async_smem();
                tc_fence_before_sync();
                mbar_arrive(&bars.st_ready);
            }
            mbar_arrive(&bars.chain_done[b & 3]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 17) tmem_dealloc(tm, kTmemCols);
}

}  // namespace

bool gdn_scan_tensor_supported(const GdnArgs &a, bool io_bf16) {
    return io_bf16 && a.d_k == kD && a.d_v == kD;
}

cudaError_t launch_gdn_scan_tensor(const GdnArgs &a, cudaStream_t s) {
    CUtensorMap mapQ, mapK, mapV, mapO;
    const uint64_t rows = static_cast<uint64_t>(a.T_total);
    const uint64_t qk_inner = static_cast<uint64_t>(a.H_k) * kD, v_inner = static_cast<uint64_t>(a.H_v) * kD;
    if (!make_tensor_map_2d(&mapQ, a.q, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        !make_tensor_map_2d(&mapK, a.k, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        (a.v && !make_tensor_map_2d(&mapV, a.v, 2, v_inner, rows, v_inner * 2, kD, kC, false)) ||
        (a.o && !make_tensor_map_2d(&mapO, a.o, 2, v_inner, rows, v_inner * 2, kD, kC, false)))
        return cudaErrorInvalidValue;
    if (!a.v) mapV = mapK;   // never used by the kernel then
    if (!a.o) mapO = mapK;
    // dynamic shared memory: everything the device allows beside the kernel's static part (the map needs
    // kSmemUsed bytes from a 1024-byte aligned base; the kernel checks that it fits)
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, gdn_scan_tensor_kernel);
    if (e != cudaSuccess) return e;
    int dev = 0, optin = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess) return e;
    const int dyn = optin - static_cast<int>(fa.sharedSizeBytes);
    if (dyn < kSmemUsed) return cudaErrorInvalidConfiguration;
    e = cudaFuncSetAttribute(gdn_scan_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);
    if (e != cudaSuccess) return e;
    gdn_scan_tensor_kernel<<<dim3(a.H_v, a.n_seq), kThreads, dyn, s>>>(a, mapQ, mapK, mapV, mapO);
    return cudaGetLastError();
}

}  // namespace lkv
