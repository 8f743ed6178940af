// Chunkwise Gated DeltaNet scan on the 5th-generation tensor cores (Eq. 1 with Eq. 3), for
// d_k = d_v = 128 and bf16 q/k/v/o.  One CTA owns one (sequence, value head) and walks the
// sequence in blocks of 64 tokens, carrying the state on chip.
//
// Everything is held transposed so that every tensor-core tile has M = d_v = 128 rows (all 128
// TMEM lanes): thread / lane j owns state column j.  Per block, with cg the running sum of g,
// gam_t = e^{cg_t}, Gam_ti = e^{cg_t - cg_i} and S the incoming state:
//   (1) G   = [Q;K] K^T            rows 0..63: q_t.k_i,  rows 64..127: k_t.k_i          tcgen05, bf16
//       P_ti = Gam_ti q_t.k_i (i <= t),   A_ti = beta_t Gam_ti k_t.k_i (i < t)          aux warpgroup
//   (2) D1  = S^T [Q;K]^T          cols 0..63: (S^T q_t)_j,  cols 64..127: (S^T k_t)_j   tcgen05
//   (3) r_t = beta_t (v_t - gam_t S^T k_t);   u = (I + A)^{-1} r  by forward substitution, each
//       thread solving its own column j in fp32                                          chain warpgroup
//   (4) PU  = U^T P^T              (sum_{i<=t} P_ti u_i)_j                               tcgen05
//       o_t = scale (gam_t S^T q_t + PU_t)                                               aux warpgroup
//   (5) S^T <- gam_C S^T + (U o w)^T K,  w_i = e^{cg_C - cg_i}                            tcgen05, fp32 state
//       accumulated in TMEM (pre-scaled there by gam_C); a bf16 copy of S^T in shared memory is the
//       A operand of (2) for the next block.
// A padded token (beyond the sequence end) has g = 0 and beta = 0, which makes it the identity step.
// Warp roles: warps 0-3 chain (steps 3 and the state copy), warps 4-7 aux (G epilogue, state
// pre-scale, outputs), warp 8 MMA issue, warp 9 TMA.  All waits on mbarriers are bounded.
#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kD = 128;   // d_k = d_v
constexpr int kC = 64;    // tokens per block
constexpr int kThreads = 320;

// shared-memory map (bytes, after 1024-byte alignment)
constexpr int kQKStage = 4 * kC * 128;                 // [Q_kb0 | K_kb0 | Q_kb1 | K_kb1], each [64 rows x 128 B]
constexpr int kVStage = kC * kD * 2;                   // [64][128] bf16, row-major
constexpr int kStageBytes = kQKStage + kVStage;        // 48 KB
constexpr int kOffSt = 2 * kStageBytes;                // S^T bf16: [St_kb0 | St_kb1], each [128 rows x 128 B]
constexpr int kOffU = kOffSt + 2 * kD * 128;           // U^T bf16 [128 rows x 128 B]
constexpr int kOffUw = kOffU + kD * 128;               // (U o w)^T bf16
constexpr int kOffP = kOffUw + kD * 128;               // P bf16 [64 rows x 128 B], double-buffered
constexpr int kOffAt = kOffP + 2 * kC * 128;           // A transposed, fp32 [i][t], double-buffered
constexpr int kOffGb = kOffAt + 2 * kC * kC * 4;       // per-block scalars, double-buffered
constexpr int kGbFloats = 4 * kC;                      // cg, beta, gam (e^{cg}), w (e^{cg_C - cg})
constexpr int kSmemBytes = kOffGb + 2 * kGbFloats * 4 + 1024;

// tensor-memory map (columns)
constexpr uint32_t kTmG = 0;      // 64
constexpr uint32_t kTmD1 = 64;    // 128: QS | KS
constexpr uint32_t kTmPU = 192;   // 64
constexpr uint32_t kTmS = 256;    // 128
constexpr uint32_t kTmemCols = 512;

struct Bars {
    uint64_t full[2], tiles_free[2];
    uint64_t g_done, d1_done, pu_done, ds_done;     // tcgen05.commit targets
    uint64_t gb_ready[2], pa_ready[2], u_ready, s_scaled, st_ready, o_done;  // thread arrivals (128 each)
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
gdn_scan_tensor_kernel(const __grid_constant__ GdnArgs a, const __grid_constant__ CUtensorMap mapQ,
                       const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Bars bars;
    __shared__ uint32_t tmem_base;
    __shared__ int dead;
    __shared__ float scan_carry;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, seq = blockIdx.y;
    const int hk = h / (a.H_v / a.H_k);
    const int t_begin = a.cu[seq], t_end = a.cu[seq + 1];
    const int nblk = (t_end - t_begin + kC - 1) / kC;
    const size_t sbase = (static_cast<size_t>(seq) * a.H_v + h) * kD * kD;

    if (nblk == 0) {  // empty sequence: hand the state through untouched
        if (a.S_T && a.S_T != a.S0)
            for (int e = tid; e < kD * kD; e += kThreads) a.S_T[sbase + e] = a.S0 ? a.S0[sbase + e] : 0.f;
        return;
    }
    if (tid == 0) {
        dead = 0;
        uint64_t *b1 = &bars.full[0];
        for (int i = 0; i < 8; ++i) mbar_init(b1 + i, 1);
        uint64_t *b128 = &bars.gb_ready[0];
        for (int i = 0; i < 8; ++i) mbar_init(b128 + i, 128);
        mbar_fence_init();
    }
    if (warp == 8) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    float *gb = reinterpret_cast<float *>(sm + kOffGb);

    if (warp == 9) {
        // ======================================================= TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapK);
            tma_prefetch_desc(&mapV);
            for (int b = 0; b < nblk; ++b) {
                const int st = b & 1;
                if (b >= 2) mbar_wait(&bars.tiles_free[st], ((b - 2) >> 1) & 1, &dead, a.status);
                unsigned char *base = sm + st * kStageBytes;
                const int row = t_begin + b * kC;
                mbar_expect_tx(&bars.full[st], kStageBytes);
                for (int kb = 0; kb < 2; ++kb) {
                    tma_load_2d(base + kb * 2 * kC * 128, &mapQ, hk * kD + kb * 64, row, &bars.full[st]);
                    tma_load_2d(base + kb * 2 * kC * 128 + kC * 128, &mapK, hk * kD + kb * 64, row, &bars.full[st]);
                }
                tma_load_2d(base + kQKStage, &mapV, h * kD, row, &bars.full[st]);
            }
        }
    } else if (warp == 8) {
        // ======================================================= MMA issuer (one elected thread, tight code)
        if (elect_one()) {
            constexpr uint32_t idG = umma_idesc(kFmtBF16, false, false, 128, 64);
            constexpr uint32_t idD1 = umma_idesc(kFmtBF16, false, false, 128, 128);
            constexpr uint32_t idPU = umma_idesc(kFmtBF16, false, false, 128, 64);
            constexpr uint32_t idDS = umma_idesc(kFmtBF16, false, true, 128, 128);
            const uint64_t dSt = umma_desc(smem_u32(sm + kOffSt), 0, 1024);
            const uint64_t dU = umma_desc(smem_u32(sm + kOffU), 0, 1024);
            const uint64_t dUw = umma_desc(smem_u32(sm + kOffUw), 0, 1024);
            const uint64_t dP0 = umma_desc(smem_u32(sm + kOffP), 0, 1024);
            auto issue_G = [&](int b) {
                const uint64_t dQK = umma_desc(smem_u32(sm + (b & 1) * kStageBytes), 0, 1024);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t off = ((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmG, dQK + off, dQK + off + ((kC * 128) >> 4), idG, k > 0);
                }
                umma_commit(&bars.g_done);
            };
            mbar_wait(&bars.full[0], 0, &dead, a.status);
            tc_fence_after_sync();
            issue_G(0);
            for (int b = 0; b < nblk; ++b) {
                const uint32_t par = b & 1;
                const uint64_t dQK = umma_desc(smem_u32(sm + (b & 1) * kStageBytes), 0, 1024);
                // (2) needs the bf16 state copy of block b and the D1 / PU accumulators drained
                mbar_wait(&bars.st_ready, par, &dead, a.status);
                if (b > 0) mbar_wait(&bars.o_done, (b - 1) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t offA = ((k >> 2) * (kD * 128) + (k & 3) * 32) >> 4;
                    const uint64_t offB = ((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmD1, dSt + offA, dQK + offB, idD1, k > 0);
                }
                umma_commit(&bars.d1_done);
                // (1) of the next block right behind it: its epilogue runs while the chain solves block b
                if (b + 1 < nblk) {
                    mbar_wait(&bars.full[(b + 1) & 1], ((b + 1) >> 1) & 1, &dead, a.status);
                    mbar_wait(&bars.pa_ready[b & 1], (b >> 1) & 1, &dead, a.status);   // G of block b has been read
                    tc_fence_after_sync();
                    issue_G(b + 1);
                }
                // (4) needs U and P
                mbar_wait(&bars.u_ready, par, &dead, a.status);
                mbar_wait(&bars.pa_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dP = dP0 + ((b & 1) * ((kC * 128) >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmPU, dU + 2 * k, dP + 2 * k, idPU, k > 0);
                umma_commit(&bars.pu_done);
                // (5) accumulates onto the pre-scaled state; B = K tile read MN-major (rows = tokens)
                mbar_wait(&bars.s_scaled, par, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dKmn = umma_desc(smem_u32(sm + (b & 1) * kStageBytes + kC * 128), 2 * kC * 128, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmS, dUw + 2 * k, dKmn + ((k * 16 * 128) >> 4), idDS, true);
                umma_commit(&bars.ds_done);
                umma_commit(&bars.tiles_free[b & 1]);
            }
        }
    } else if (warp >= 4) {
        // ======================================================= aux warpgroup
        const int x = tid - 128;                 // 0..127 = TMEM lane
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // per-block scalars: cg, beta, gam = e^{cg}, w = e^{cg_C - cg}
        auto prepare_scalars = [&](int b) {
            float *dst = gb + (b & 1) * kGbFloats;
            const int t0 = t_begin + b * kC;
            float gv = 0.f, bv = 0.f;
            if (x < kC && t0 + x < t_end) {
                gv = a.g[static_cast<size_t>(t0 + x) * a.H_v + h];
                bv = a.beta[static_cast<size_t>(t0 + x) * a.H_v + h];
            }
            float run = gv;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float up = __shfl_up_sync(0xffffffffu, run, o);
                if (lane >= o) run += up;
            }
            if (x == 31) scan_carry = run;
            named_bar_sync(1, 128);
            if (x >= 32 && x < kC) run += scan_carry;
            if (x < kC) { dst[x] = run; dst[kC + x] = bv; dst[2 * kC + x] = __expf(run); }
            named_bar_sync(1, 128);
            if (x < kC) dst[3 * kC + x] = __expf(dst[kC - 1] - run);
            named_bar_sync(1, 128);
        };
        // epilogue of (1): rows 0..63 -> P (bf16 operand), rows 64..127 -> A transposed (fp32)
        auto g_epilogue = [&](int b) {
            const float *sc = gb + (b & 1) * kGbFloats;
            mbar_wait(&bars.g_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            const int t = x & 63;
            const float cgt = sc[t], bt = sc[kC + t];
            // the P / A buffers of parity b were last used by block b-2, whose outputs this warpgroup
            // has already written: nothing to wait for
            mbar_arrive(&bars.gb_ready[b & 1]);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[32];
                tmem_ld32(lane_base + kTmG + 32 * q, rr);
                tmem_ld_wait();
                if (x < kC) {
                    unsigned char *prow = sm + kOffP + (b & 1) * (kC * 128);
#pragma unroll
                    for (int c8 = 0; c8 < 4; ++c8) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int i0 = 32 * q + 8 * c8 + 2 * e;
                            const float p0 = (i0 <= t) ? __expf(cgt - sc[i0]) * __uint_as_float(rr[8 * c8 + 2 * e]) : 0.f;
                            const float p1 = (i0 + 1 <= t) ? __expf(cgt - sc[i0 + 1]) * __uint_as_float(rr[8 * c8 + 2 * e + 1]) : 0.f;
                            w[e] = pack_bf16(p0, p1);
                        }
                        *reinterpret_cast<uint4 *>(prow + sw128_offset(t, 4 * q + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                } else {
                    float *at = reinterpret_cast<float *>(sm + kOffAt) + (b & 1) * (kC * kC);
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const int i = 32 * q + c;
                        at[i * kC + t] = (i < t) ? bt * __expf(cgt - sc[i]) * __uint_as_float(rr[c]) : 0.f;
                    }
                }
            }
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.pa_ready[b & 1]);
        };
        prepare_scalars(0);
        g_epilogue(0);
        __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(a.o);
        for (int b = 0; b < nblk; ++b) {
            const float *sc = gb + (b & 1) * kGbFloats;
            // pre-scale the fp32 state by gam_C once the chain warpgroup has taken its bf16 copy
            mbar_wait(&bars.st_ready, b & 1, &dead, a.status);
            tc_fence_after_sync();
            const float gamC = sc[2 * kC + kC - 1];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t rr[32];
                tmem_ld32(lane_base + kTmS + 32 * q, rr);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; ++c) rr[c] = __float_as_uint(__uint_as_float(rr[c]) * gamC);
                tmem_st32(lane_base + kTmS + 32 * q, rr);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars.s_scaled);
            // the next block's scalars and G epilogue, while the chain solves block b
            if (b + 1 < nblk) {
                prepare_scalars(b + 1);
                g_epilogue(b + 1);
            }
            // outputs of block b: o_t[j] = scale (gam_t (S^T q_t)_j + PU_t[j]); lane = j
            mbar_wait(&bars.d1_done, b & 1, &dead, a.status);
            mbar_wait(&bars.pu_done, b & 1, &dead, a.status);
            tc_fence_after_sync();
            const int t0 = t_begin + b * kC;
            const int n = min(kC, t_end - t0);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t qs[32], pu[32];
                tmem_ld32(lane_base + kTmD1 + 32 * q, qs);
                tmem_ld32(lane_base + kTmPU + 32 * q, pu);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int t = 32 * q + c;
                    const float val = a.scale * (sc[2 * kC + t] * __uint_as_float(qs[c]) + __uint_as_float(pu[c]));
                    if (t < n) o[(static_cast<size_t>(t0 + t) * a.H_v + h) * kD + x] = __float2bfloat16_rn(val);
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bars.o_done);
        }
    } else {
        // ======================================================= chain warpgroup: thread j = state column j
        const int j = tid;
        const uint32_t lane_base = tm + (static_cast<uint32_t>(warp * 32) << 16);
        // bf16 copy of S^T row j into the K-major operand [St_kb0 | St_kb1]; `vals` = 32 consecutive m
        auto store_st_chunk = [&](int q, const uint32_t (&rr)[32]) {
            unsigned char *base = sm + kOffSt + (q >> 1) * (kD * 128);
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    w[e] = pack_bf16(__uint_as_float(rr[8 * c8 + 2 * e]), __uint_as_float(rr[8 * c8 + 2 * e + 1]));
                *reinterpret_cast<uint4 *>(base + sw128_offset(j, 4 * (q & 1) + c8)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        };
        // initial state: S0[m][j] -> TMEM (fp32) and shared memory (bf16)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t rr[32];
#pragma unroll
            for (int c = 0; c < 32; ++c)
                rr[c] = a.S0 ? __float_as_uint(a.S0[sbase + static_cast<size_t>(32 * q + c) * kD + j]) : 0u;
            tmem_st32(lane_base + kTmS + 32 * q, rr);
            store_st_chunk(q, rr);
        }
        tmem_st_wait();
        fence_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&bars.st_ready);

        for (int b = 0; b < nblk; ++b) {
            const uint32_t par = b & 1;
            const float *sc = gb + (b & 1) * kGbFloats;
            const __nv_bfloat16 *vt = reinterpret_cast<const __nv_bfloat16 *>(sm + (b & 1) * kStageBytes + kQKStage);
            mbar_wait(&bars.gb_ready[b & 1], (b >> 1) & 1, &dead, a.status);
            mbar_wait(&bars.full[b & 1], (b >> 1) & 1, &dead, a.status);
            mbar_wait(&bars.d1_done, par, &dead, a.status);
            tc_fence_after_sync();
            // (3) right-hand side r_t = beta_t (v_t[j] - gam_t (S^T k_t)_j)
            float u[kC];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                uint32_t rr[32];
                tmem_ld32(lane_base + kTmD1 + kC + 32 * q, rr);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int t = 32 * q + c;
                    u[t] = sc[kC + t] * (__bfloat162float(vt[t * kD + j]) - sc[2 * kC + t] * __uint_as_float(rr[c]));
                }
            }
            // forward substitution with the transposed coupling matrix: u_t -= A_ti u_i for t > i
            mbar_wait(&bars.pa_ready[b & 1], (b >> 1) & 1, &dead, a.status);
            const float *at = reinterpret_cast<const float *>(sm + kOffAt) + (b & 1) * (kC * kC);
#pragma unroll
            for (int i = 0; i < kC - 1; ++i) {
                const float ui = u[i];
#pragma unroll
                for (int t4 = (i + 1) & ~3; t4 < kC; t4 += 4) {
                    const float4 av = *reinterpret_cast<const float4 *>(at + i * kC + t4);
                    if (t4 + 0 > i) u[t4 + 0] = fmaf(-av.x, ui, u[t4 + 0]);
                    if (t4 + 1 > i) u[t4 + 1] = fmaf(-av.y, ui, u[t4 + 1]);
                    if (t4 + 2 > i) u[t4 + 2] = fmaf(-av.z, ui, u[t4 + 2]);
                    if (t4 + 3 > i) u[t4 + 3] = fmaf(-av.w, ui, u[t4 + 3]);
                }
            }
            // U^T and (U o w)^T rows as bf16 K-major operands
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                uint32_t w0[4], w1[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = 8 * c8 + 2 * e;
                    w0[e] = pack_bf16(u[i], u[i + 1]);
                    w1[e] = pack_bf16(u[i] * sc[3 * kC + i], u[i + 1] * sc[3 * kC + i + 1]);
                }
                *reinterpret_cast<uint4 *>(sm + kOffU + sw128_offset(j, c8)) = make_uint4(w0[0], w0[1], w0[2], w0[3]);
                *reinterpret_cast<uint4 *>(sm + kOffUw + sw128_offset(j, c8)) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
            }
            fence_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars.u_ready);
            // new state: fp32 stays in TMEM, bf16 copy for the next block (or S_T at the end)
            mbar_wait(&bars.ds_done, par, &dead, a.status);
            tc_fence_after_sync();
            const bool last = b + 1 == nblk;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t rr[32];
                tmem_ld32(lane_base + kTmS + 32 * q, rr);
                tmem_ld_wait();
                if (!last) store_st_chunk(q, rr);
                else if (a.S_T) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) a.S_T[sbase + static_cast<size_t>(32 * q + c) * kD + j] = __uint_as_float(rr[c]);
                }
            }
            if (!last) {
                fence_async_smem();
                tc_fence_before_sync();
                mbar_arrive(&bars.st_ready);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tm, kTmemCols);
}

}  // namespace

bool gdn_scan_tensor_supported(const GdnArgs &a, bool io_bf16) {
    return io_bf16 && a.d_k == kD && a.d_v == kD;
}

cudaError_t launch_gdn_scan_tensor(const GdnArgs &a, cudaStream_t s) {
    CUtensorMap mapQ, mapK, mapV;
    const uint64_t rows = static_cast<uint64_t>(a.T_total);
    const uint64_t qk_inner = static_cast<uint64_t>(a.H_k) * kD, v_inner = static_cast<uint64_t>(a.H_v) * kD;
    if (!make_tensor_map_2d(&mapQ, a.q, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        !make_tensor_map_2d(&mapK, a.k, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        !make_tensor_map_2d(&mapV, a.v, 2, v_inner, rows, v_inner * 2, kD, kC, false))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(gdn_scan_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    gdn_scan_tensor_kernel<<<dim3(a.H_v, a.n_seq), kThreads, kSmemBytes, s>>>(a, mapQ, mapK, mapV);
    return cudaGetLastError();
}

}  // namespace lkv
