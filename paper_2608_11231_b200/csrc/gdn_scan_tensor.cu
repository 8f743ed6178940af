// Chunkwise Gated DeltaNet scan on the 5th-generation tensor cores (Eq. 1 with Eq. 3), for
// d_k = d_v = 128 and bf16 q/k/v/o.  One CTA owns one (sequence, value head) and walks the
// sequence in blocks of 64 tokens, carrying the state on chip.
//
// Everything is held transposed so that every tensor-core tile has M = d_v = 128 rows (all 128
// TMEM lanes): lane j owns state column j.  Per block, with cg the running sum of g,
// gam_t = e^{cg_t}, Gam_ti = e^{cg_t - cg_i}, w_t = e^{cg_C - cg_t} and S the incoming state:
//   (1) G    = [Q;K] K^T             rows 0..63: q_t.k_i, rows 64..127: k_t.k_i           tcgen05
//       Ps_ti = scale Gam_ti q_t.k_i (i <= t),  A_ti = beta_t Gam_ti k_t.k_i (i < t)      mask warps
//       M    = (I + A)^{-1}          (UT transform, by doubling: 8x8 blocks by substitution and 8 -> 16 in
//                                     fp32, 16 -> 32 -> 64 by fp16 block products)         prep warps
//       X_mi = M_mi beta_i           bf16 operand of the block's triangular solve          prep warps
//  (3a) U^T  = V^T X^T               the part of the solve that does not depend on S       tcgen05
//  (2K) KS   = S^T K^T               (S^T k_t)_j                                          tcgen05 (A = bf16 S^T in TMEM)
//       Rk_t = -gam_t KS_t           -> bf16 pairs in place                                chain warps
//  (3b) U^T += Rk X^T                u = M r, r_t = beta_t (v_t - gam_t S^T k_t): the block's pseudo-values
//       Uw_t = w_t u_t and u_t       -> two bf16 operands in place                         chain warps
//   (5) S^T <- gam_C S^T + Uw^T K    fp32 state accumulated in TMEM (pre-scaled there)      tcgen05 (A from TMEM)
//       S^T -> bf16 pairs in TMEM for (2K)/(2Q) of the next block, pre-scale by its gam_C  chain warps
//  (2Q) O^T  = S^T Qs^T,  Qs_t = scale gam_t q_t (the Q tile is scaled in place once (1) has read it)
//   (7) O^T += u^T Ps^T              so that o_t = scale (gam_t S^T q_t + (P u)_t)          tcgen05 (A from TMEM)
// The block-to-block chain is (2K) -> Rk -> (3b) -> Uw -> (5) -> state copy: three tensor-memory
// to tensor-memory conversions, no shared memory and no proxy fence on it.  Everything else ((1), the
// mask epilogue, the inverse, (3a), the Q scaling) runs up to two blocks ahead of the chain; (2Q) and
// (7) hang off it.  A padded token (beyond the sequence end) has g = 0 and beta = 0: the identity step.
//
// Warps 0-7 chain (lane = state column, warpgroup = half of the tokens / state rows), 8-11 mask epilogue of (1)
// and the output tile of the block the chain has finished, 12-15 prep (the inverse, Q scaling), 16 TMA loads of V and the store of the output tile, 17 MMA issue of
// the chain, 18 TMA loads of Q and K and MMA issue of (1), 19 per-block scalars.  All waits on mbarriers
// are bounded.
//
// The hot loops are kept small on purpose (loops that are not unrolled, rare paths in functions that are not
// inlined): the twenty warps run seven different programs at once, and with the first, fully unrolled
// version of this kernel the SMs fetched a third of their instructions from the cache they share with
// their neighbours, which then ran at 80 % of its request rate and set the pace of the whole kernel.
#include <cuda_fp16.h>
#include <string.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace lkv {

namespace {

using namespace tc;

constexpr int kD = 128;   // d_k = d_v
constexpr int kC = 64;    // tokens per block
constexpr int kThreads = 640;

// shared-memory map (bytes, after 1024-byte alignment); operand tiles have 128-byte rows, 128-byte swizzle
constexpr int kQKStage = 4 * kC * 128;                 // [Q_kb0 | K_kb0 | Q_kb1 | K_kb1], each [64 tokens x 128 B]
constexpr int kQKStages = 3;                           // (1) and the mask epilogue run two blocks ahead of the chain
constexpr int kVStage = 2 * kC * 128;                  // [V_jb0 | V_jb1], each [64 tokens x 128 B]; once (3a) has read it, the
                                                       // stage holds the block's output tile [64 tokens][128] bf16 for the TMA store
constexpr int kOffV = kQKStages * kQKStage;            // two V stages
constexpr int kOffX = kOffV + 2 * kVStage;             // X bf16 [64 rows m x 128 B], double-buffered
constexpr int kOffP = kOffX + 2 * kC * 128;            // Ps bf16 [64 rows t x 128 B], three buffers
constexpr int kLd = 68;                                // row stride (floats) of the fp32 A and M matrices: rows 4 banks apart
constexpr int kOffA = kOffP + 3 * kC * 128;            // A fp32 [t][i], double-buffered
constexpr int kOffM = kOffA + 2 * kC * kLd * 4;        // M fp32 [t][i]
constexpr int kOffGb = kOffM + kC * kLd * 4;           // per-block scalars, four buffers
constexpr int kGbFloats = 5 * kC + 4;                  // cg2 = cg log2(e), beta, gam (e^{cg}), w (e^{cg_C - cg}), f (e^{cg_ref - cg}), flag
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kMaxGroupRange = 100.f;                // log2 units: above this the per-group factors could overflow
constexpr int kSmemUsed = kOffGb + 4 * kGbFloats * 4;  // from the 1024-byte aligned base
constexpr int kSmemBytes = kSmemUsed + 1024;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

// tensor-memory map (columns)
constexpr uint32_t kTmS = 0;      // 128: S^T fp32
constexpr uint32_t kTmSb = 128;   // 64: S^T as bf16 pairs (A operand of (2K), (2Q))
constexpr uint32_t kTmKS = 192;   // 64: KS fp32; Rk as bf16 pairs in place (tokens 0..31 in columns 0..15, 32..63 in 32..47)
constexpr uint32_t kTmU = 256;    // 64: U fp32; in place Uw as bf16 pairs (columns 0..15 and 32..47) and u (16..31 and 48..63)
constexpr uint32_t kTmO = 320;    // 2 x 64: O^T of the even / odd blocks
constexpr uint32_t kTmG = 448;    // 64
constexpr uint32_t kTmemCols = 512;

struct Bars {
    // single-arrival barriers: TMA transactions and tcgen05.commit
    uint64_t full_qk[3], tiles_free_qk[3], full_v[2], g_done[2], ks_done, u_done, ds_done, o_mma_done[4], p_free[3], x_free[2];
    // 128-thread barriers (prep or mask warpgroup)
    uint64_t m_ready[2], o_done[4], o_staged[2];
    // 64-thread barriers (the two halves of the mask warpgroup)
    uint64_t a_ready[2], p_ready[3];
    // 32-thread barriers (the scalar warp)
    uint64_t gb_ready[4];
    // 256-thread barriers (both chain warpgroups)
    uint64_t rk_ready, uw_ready, st_ready, chain_done[4], qs_ready[3];
};
constexpr int kBars1 = 22, kBars128 = 8, kBars64 = 5, kBars32 = 4, kBars256 = 10;
static_assert(sizeof(Bars) == 8 * (kBars1 + kBars128 + kBars64 + kBars32 + kBars256), "barrier table");

// A quarter row of the Q tile (token tid & 63, 16-byte chunks 4 * (part & 1) .. + 3 of K-block part >> 1, part = tid >> 6)
// multiplied in place by f.  Not inlined: the chain warps' registers are spoken for.
static __device__ __noinline__ void scale_q_quarter(unsigned char *stage, int tid, float f) {
    const int tq = tid & 63, part = tid >> 6;
    unsigned char *qt = stage + (part >> 1) * (2 * kC * 128) + tq * 128;
    const __nv_bfloat162 f2 = __float2bfloat162_rn(f);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint4 *p = reinterpret_cast<uint4 *>(qt + (((4 * (part & 1) + c) ^ (tq & 7)) << 4));
        uint4 v = *p;
        __nv_bfloat162 *e = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = __hmul2(e[i], f2);
        *p = v;
    }
}

// Warp-level tensor-core MMA on fp16 operands (11-bit significands like tf32, but 16 k-elements per
// instruction): acc[16 x 8] += A[16 x 16] B[16 x 8], fp32 accumulation.  Fragments as the PTX ISA lays them out.
// Every operand here is an entry of A or of an inverse of I + A: of order one or smaller, far inside the fp16 range.
__device__ __forceinline__ void mma_f16_16x8x16(float (&acc)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(acc[0]), "+f"(acc[1]), "+f"(acc[2]), "+f"(acc[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16_early(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}
// A operand: the 16 x 16 tile at p of a row-major fp32 matrix (row stride kLd); gid = lane / 4, tig = lane % 4
__device__ __forceinline__ void frag_a(uint32_t (&a)[4], const float *p, int gid, int tig) {
    const float2 v0 = *reinterpret_cast<const float2 *>(p + gid * kLd + 2 * tig);
    const float2 v1 = *reinterpret_cast<const float2 *>(p + (gid + 8) * kLd + 2 * tig);
    const float2 v2 = *reinterpret_cast<const float2 *>(p + gid * kLd + 2 * tig + 8);
    const float2 v3 = *reinterpret_cast<const float2 *>(p + (gid + 8) * kLd + 2 * tig + 8);
    a[0] = pack_f16(v0.x, v0.y); a[1] = pack_f16(v1.x, v1.y); a[2] = pack_f16(v2.x, v2.y); a[3] = pack_f16(v3.x, v3.y);
}
// B operand: the 16 (k) x 8 (n) tile at p of a row-major fp32 matrix B[k][n]
__device__ __forceinline__ void frag_b(uint32_t &b0, uint32_t &b1, const float *p, int gid, int tig) {
    b0 = pack_f16(p[(2 * tig) * kLd + gid], p[(2 * tig + 1) * kLd + gid]);
    b1 = pack_f16(p[(2 * tig + 8) * kLd + gid], p[(2 * tig + 9) * kLd + gid]);
}
// accumulator tile [16 x 8] -> p (row-major fp32), times sgn
__device__ __forceinline__ void store_acc(float *p, const float (&acc)[4], float sgn, int gid, int tig) {
    *reinterpret_cast<float2 *>(p + gid * kLd + 2 * tig) = make_float2(sgn * acc[0], sgn * acc[1]);
    *reinterpret_cast<float2 *>(p + (gid + 8) * kLd + 2 * tig) = make_float2(sgn * acc[2], sgn * acc[3]);
}

// Byte offset of element (row m, column i) of a bf16 operand tile with 128-byte rows and the 128-byte swizzle
__device__ __forceinline__ uint32_t x_offset(int m, int i) { return m * 128u + ((((uint32_t)i >> 3) ^ (m & 7u)) << 4) + (i & 7) * 2u; }
// Final entries of M also go, times beta of their column and rounded to bf16, into the operand X = M diag(beta) of the
// block's triangular solve: no second pass over M.  Accumulator tile [16 x 8] at (m0, i0):
__device__ __forceinline__ void store_acc_x(unsigned char *xb, const float *beta, int m0, int i0, const float (&acc)[4], float sgn,
                                            int gid, int tig) {
    const int i = i0 + 2 * tig;
    const float b0 = sgn * beta[i], b1 = sgn * beta[i + 1];
    *reinterpret_cast<uint32_t *>(xb + x_offset(m0 + gid, i)) = pack_bf16_early(acc[0] * b0, acc[1] * b1);
    *reinterpret_cast<uint32_t *>(xb + x_offset(m0 + gid + 8, i)) = pack_bf16_early(acc[2] * b0, acc[3] * b1);
}

// The inverse M = (I + A)^{-1} of the unit lower triangular 64x64 matrix of a block is built by doubling:
// 8x8 diagonal blocks by forward substitution, then three merges
//     inv [[L1, 0], [A21, L2]] = [[inv L1, 0], [-inv(L2) A21 inv(L1), inv L2]]
// from 8 to 16 (fp32 FMAs), 16 to 32 and 32 to 64 (warp-level tensor-core MMA, fp16 operands rounded to nearest,
// fp32 accumulation): four rounds of dependent MMAs per block, eight MMAs per warp in all.
// A, M: fp32 [64][kLd]; the part of M above the block diagonal serves as scratch.
//
// 16 -> 32: half (8 columns from 8 nh) of the 16x16 block (c + 1, c): X = A_rc M_cc, M_rc = -M_rr X; X passes
// through the unused block (c, r) above the diagonal to change from accumulator to operand layout.
__device__ __forceinline__ void inv_merge32(const float *Af, float *Mf, unsigned char *xb, const float *beta, int c, int nh, int gid, int tig) {
    const int r = c + 1;
    uint32_t a[4], b0, b1;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    frag_a(a, Af + (16 * r) * kLd + 16 * c, gid, tig);
    frag_b(b0, b1, Mf + (16 * c) * kLd + 16 * c + 8 * nh, gid, tig);
    mma_f16_16x8x16(acc, a, b0, b1);
    float *xs = Mf + (16 * c) * kLd + 16 * r + 8 * nh;
    store_acc(xs, acc, 1.f, gid, tig);
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = 0.f;
    frag_a(a, Mf + (16 * r) * kLd + 16 * r, gid, tig);
    frag_b(b0, b1, xs, gid, tig);
    mma_f16_16x8x16(acc, a, b0, b1);
    store_acc(Mf + (16 * r) * kLd + 16 * c + 8 * nh, acc, -1.f, gid, tig);
    store_acc_x(xb, beta, 16 * r, 16 * c + 8 * nh, acc, -1.f, gid, tig);
}
// 32 -> 64, first half: T = A21 inv(L1) with A21 = A[32.., 0..31], inv(L1) = M[0..31, 0..31] (lower triangular by 16x16
// blocks).  Warp (mt, nb) computes rows 16 mt .. +15, columns 16 nb .. +15 of T into the scratch M[0..31, 32..63].
__device__ __forceinline__ void inv_merge64_a(const float *Af, float *Mf, int mt, int nb, int gid, int tig) {
    float acc[2][2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nt][e][i] = 0.f;
#pragma unroll
    for (int kb = 0; kb < 2; ++kb) {
        if (kb >= nb) {   // rows of inv(L1) above its block diagonal are zero
            uint32_t a[4], b0, b1;
            frag_a(a, Af + (32 + 16 * mt) * kLd + 16 * kb, gid, tig);
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                frag_b(b0, b1, Mf + (16 * kb) * kLd + 16 * nb + 8 * nt, gid, tig);
                mma_f16_16x8x16(acc[nt][kb], a, b0, b1);
            }
        }
    }
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][0][i] += acc[nt][1][i];
        store_acc(Mf + (16 * mt) * kLd + 32 + 16 * nb + 8 * nt, acc[nt][0], 1.f, gid, tig);
    }
}
// 32 -> 64, second half: M[32.., 0..31] = -inv(L2) T with inv(L2) = M[32.., 32..] (lower triangular by blocks).
__device__ __forceinline__ void inv_merge64_b(float *Mf, unsigned char *xb, const float *beta, int mt, int nb, int gid, int tig) {
    float acc[2][2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nt][e][i] = 0.f;
#pragma unroll
    for (int kb = 0; kb < 2; ++kb) {
        if (kb <= mt) {   // columns of inv(L2) right of its block diagonal are zero
            uint32_t a[4], b0, b1;
            frag_a(a, Mf + (32 + 16 * mt) * kLd + 32 + 16 * kb, gid, tig);
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                frag_b(b0, b1, Mf + (16 * kb) * kLd + 32 + 16 * nb + 8 * nt, gid, tig);
                mma_f16_16x8x16(acc[nt][kb], a, b0, b1);
            }
        }
    }
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][0][i] += acc[nt][1][i];
        store_acc_x(xb, beta, 32 + 16 * mt, 16 * nb + 8 * nt, acc[nt][0], -1.f, gid, tig);   // nobody reads these entries of M again
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
// 16 fp32 values (as loaded from tensor memory) -> 8 columns of bf16 pairs, the even element in the low half
__device__ __forceinline__ void pack16(const float (&v)[16], uint32_t (&w)[8]) {
#pragma unroll
    for (int e = 0; e < 8; ++e) w[e] = pack_bf16(v[2 * e], v[2 * e + 1]);
}
// Mask of one group of 16 columns of one row of G, exact form for a block whose decay is too violent for the
// per-group factors: one exponential per element.  Rare, kept out of the hot loop as a whole (load from tensor
// memory, mask, store) so that no register array crosses the call.  to_ps: bf16 row of Ps, else fp32 row of A.
__device__ __noinline__ void mask_group_exact(uint32_t taddr, const float *sc, float cgt, float coef, int i0, int lim, bool to_ps,
                                              unsigned char *ps, float *arow, int t) {
    uint32_t rr[16];
    tmem_ld16(taddr, rr);
    tmem_ld_wait();
    float v[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) v[c] = (i0 + c <= lim) ? coef * exp2f(cgt - sc[i0 + c]) * __uint_as_float(rr[c]) : 0.f;
    if (to_ps) {
        store_row_chunks(ps, t, i0 >> 3, v);
    } else {
#pragma unroll
        for (int c = 0; c < 16; c += 4) *reinterpret_cast<float4 *>(arow + i0 + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
    }
}
// Rows of a ragged last block go straight to global memory: 16 tokens of one state column per call, read from
// tensor memory here.
__device__ __noinline__ void store_o_partial(uint32_t taddr, __nv_bfloat16 *orow, size_t tstride, int n_left) {
    uint32_t pu[16];
    tmem_ld16(taddr, pu);
    tmem_ld_wait();
#pragma unroll
    for (int c = 0; c < 16; ++c)
        if (c < n_left) orow[c * tstride] = __float2bfloat16_rn(__uint_as_float(pu[c]));
}

__global__ void __launch_bounds__(kThreads, 1)
gdn_scan_tensor_kernel(const __grid_constant__ GdnArgs a, const __grid_constant__ CUtensorMap mapQ,
                       const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                       const __grid_constant__ CUtensorMap mapO) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char *sm = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ Bars bars;
    __shared__ uint32_t tmem_base;
    __shared__ volatile int dead;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, seq = a.cu[a.n_ranges + 1 + blockIdx.y];   // launch order: longest sequence first
    const bool tr = seq >= a.tr_first;                                    // transition sequence
    const int rg = tr ? seq - a.tr_first + a.tr_src0 : seq;
    const bool s0_id = a.s0_identity || tr;
    const int hk = h / (a.H_v / a.H_k);
    const int t_begin = a.cu[rg], t_end = a.cu[rg + 1];
    const int nblk = (t_end - t_begin + kC - 1) / kC;
    const size_t sbase = (static_cast<size_t>(seq) * a.H_v + h) * kD * kD;
    const bool has_v = a.v != nullptr && !tr, has_o = a.o != nullptr && !tr;

    if (nblk == 0) {  // empty sequence: hand the state through untouched
        float *ST = (tr && a.tr_out) ? a.tr_out : a.S_T;   // final state of this sequence
        const size_t obase = (tr && a.tr_out) ? (static_cast<size_t>(seq - a.tr_first) * a.H_v + h) * kD * kD : sbase;
        if (ST && (ST != a.S0 || s0_id || a.S_add))
            for (int e = tid; e < kD * kD; e += kThreads)
                store_state(ST, a.st_bf16, obase + e,
                            (s0_id ? (e / kD == e % kD ? 1.f : 0.f) : (a.S0 ? a.S0[sbase + e] : 0.f)) +
                                (a.S_add ? a.S_add[sbase + e] : 0.f));
        return;
    }
    if (tid == 0) {
        dead = 0;
        uint64_t *bp = &bars.full_qk[0];
        for (int i = 0; i < kBars1; ++i) mbar_init(bp++, 1);
        for (int i = 0; i < kBars128; ++i) mbar_init(bp++, 128);
        for (int i = 0; i < kBars64; ++i) mbar_init(bp++, 64);
        for (int i = 0; i < kBars32; ++i) mbar_init(bp++, 32);
        for (int i = 0; i < kBars256; ++i) mbar_init(bp++, 256);
        mbar_fence_init();
    }
    if (warp == 17) tmem_alloc(&tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tm = tmem_base;
    float *gb = reinterpret_cast<float *>(sm + kOffGb);

    if (warp == 16) {
        // ======================================================= TMA producer of the V tiles and store of the output tiles
        if (lane == 0) {
            if (has_v) tma_prefetch_desc(&mapV);
            if (has_o) tma_prefetch_desc(&mapO);
#pragma unroll 1
            for (int b = 0; b < nblk + 2; ++b) {
                if (dead) break;   // a wait ran out: nothing more is issued
                const int st = b & 1;
                const int row = t_begin + b * kC;
                if (has_v && b + 2 < nblk)
                    for (int kb = 0; kb < 2; ++kb) tma_prefetch_l2_2d(&mapV, h * kD + kb * 64, row + 2 * kC);
                // the V stage of this parity has held the output tile of block b-2 (whole blocks only) since (3a) of
                // that block had read it: store the tile, then reuse the stage
                if (b >= 2) {
                    mbar_wait(&bars.o_staged[st], ((b - 2) >> 1) & 1, &dead, a.status);
                    if (has_o && row - kC <= t_end && !dead) {
                        for (int jb = 0; jb < 2; ++jb) tma_store_2d(&mapO, sm + kOffV + st * kVStage + jb * kC * 128, h * kD + jb * 64, row - 2 * kC);
                        tma_store_commit();
                        tma_store_wait_read();
                    }
                }
                if (has_v && b < nblk) {   // without v (read as zeros) nothing is loaded and (3a) is not issued
                    unsigned char *vb = sm + kOffV + st * kVStage;
                    mbar_expect_tx(&bars.full_v[st], kVStage);
                    for (int jb = 0; jb < 2; ++jb) tma_load_2d(vb + jb * kC * 128, &mapV, h * kD + jb * 64, row, &bars.full_v[st]);
                }
            }
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
#pragma unroll 1
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
            float run = gv.x + gv.y;
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
        // ======================================================= TMA loads of the Q and K tiles (three stages) and MMA issue of (1)
        if (elect_one()) {
            constexpr uint32_t idG = umma_idesc(kFmtBF16, false, false, 128, 64);
            tma_prefetch_desc(&mapQ);
            tma_prefetch_desc(&mapK);
#pragma unroll 1
            for (int b = 0; b < nblk; ++b) {
                if (dead) break;   // a wait ran out: nothing more is issued
                const int s3 = b % kQKStages;
                const int row = t_begin + b * kC;
                unsigned char *base = sm + s3 * kQKStage;
                // the tiles of block b go into the stage that (5) of block b-3 has released: two blocks before the
                // chain needs them.  The ring cannot hide the DRAM latency: the tiles of block b+3 are pulled into L2 now.
#pragma unroll 1
                for (int kb = 0; kb < 2; ++kb) {
                    if (b + kQKStages < nblk) {
                        tma_prefetch_l2_2d(&mapQ, hk * kD + kb * 64, row + kQKStages * kC);
                        tma_prefetch_l2_2d(&mapK, hk * kD + kb * 64, row + kQKStages * kC);
                    }
                }
                if (b >= kQKStages) mbar_wait(&bars.tiles_free_qk[s3], ((b - kQKStages) / kQKStages) & 1, &dead, a.status);
                mbar_expect_tx(&bars.full_qk[s3], kQKStage);
#pragma unroll 1
                for (int kb = 0; kb < 2; ++kb) {
                    tma_load_2d(base + kb * 2 * kC * 128, &mapQ, hk * kD + kb * 64, row, &bars.full_qk[s3]);
                    tma_load_2d(base + kb * 2 * kC * 128 + kC * 128, &mapK, hk * kD + kb * 64, row, &bars.full_qk[s3]);
                }
                // (1) of block b: the mask epilogue of block b-1 has drained the G columns
                if (b >= 1) {
                    mbar_wait(&bars.a_ready[(b - 1) & 1], ((b - 1) >> 1) & 1, &dead, a.status);
                    mbar_wait(&bars.p_ready[(b - 1) % 3], ((b - 1) / 3) & 1, &dead, a.status);
                }
                mbar_wait(&bars.full_qk[s3], (b / kQKStages) & 1, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dQK = umma_desc(smem_u32(base), 0, 1024);
#pragma unroll 1
                for (int k = 0; k < 8; ++k) {
                    const uint64_t off = ((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4;
                    umma_bf16(tm + kTmG, dQK + off, dQK + off + ((kC * 128) >> 4), idG, k > 0);
                }
                umma_commit(&bars.g_done[b & 1]);
            }
        }
    } else if (warp == 17) {
        // ======================================================= first MMA issuer: (2K), (3a), (3b), (2Q), (5), (7)
        if (elect_one()) {
            constexpr uint32_t idN64 = umma_idesc(kFmtBF16, false, false, 128, 64);    // (2K), (2Q), (3b), (7)
            constexpr uint32_t id3a = umma_idesc(kFmtBF16, true, false, 128, 64);      // A = V tile read MN-major
            constexpr uint32_t id5 = umma_idesc(kFmtBF16, false, true, 128, 128);      // B = K tile read MN-major
#pragma unroll 1
            for (int b = 0; b < nblk; ++b) {
                const uint32_t par = b & 1;
                const uint32_t qk = smem_u32(sm + (b % kQKStages) * kQKStage);
                const uint64_t dQ = umma_desc(qk, 0, 1024), dK = umma_desc(qk + kC * 128, 0, 1024);
                const uint64_t dX = umma_desc(smem_u32(sm + kOffX + (b & 1) * (kC * 128)), 0, 1024);
                // (2K) needs the bf16 state of block b and the K tile
                mbar_wait(&bars.st_ready, par, &dead, a.status);
                mbar_wait(&bars.full_qk[b % kQKStages], (b / kQKStages) & 1, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16_ts(tm + kTmKS, tm + kTmSb + 8 * k, dK + (((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4), idN64, k > 0);
                umma_commit(&bars.ks_done);
                // (3a) U = V^T X^T: needs the inverse of the block and the V tile (the U columns were read by (5) and (7)
                // of the previous block, issued before)
                mbar_wait(&bars.m_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                if (has_v) {
                    mbar_wait(&bars.full_v[b & 1], (b >> 1) & 1, &dead, a.status);
                    tc_fence_after_sync();
                    const uint64_t dV = umma_desc(smem_u32(sm + kOffV + (b & 1) * kVStage), kC * 128, 1024);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(tm + kTmU, dV + ((k * 16 * 128) >> 4), dX + 2 * k, id3a, k > 0);
                }
                // (3b) U += Rk X^T
                mbar_wait(&bars.rk_ready, par, &dead, a.status);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_bf16_ts(tm + kTmU, tm + kTmKS + 32 * (k >> 1) + 8 * (k & 1), dX + 2 * k, idN64, has_v || k > 0);
                umma_commit(&bars.u_done);
                umma_commit(&bars.x_free[b & 1]);
                // (2Q) O = S^T Qs^T while the chain warps work on U: it reads the bf16 state of this block (rewritten only after
                // (5)), the Q tile scaled by the chain warps, and O columns that were drained with the outputs of block b-2
                if (has_o) {
                    if (b >= 2) mbar_wait(&bars.o_done[(b - 2) & 3], ((b - 2) >> 2) & 1, &dead, a.status);
                    mbar_wait(&bars.qs_ready[b % kQKStages], (b / kQKStages) & 1, &dead, a.status);
                    tc_fence_after_sync();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        umma_bf16_ts(tm + kTmO + 64 * par, tm + kTmSb + 8 * k, dQ + (((k >> 2) * (2 * kC * 128) + (k & 3) * 32) >> 4), idN64, k > 0);
                }
                // (5) accumulates onto the pre-scaled state; B = K tile read MN-major (rows = tokens)
                mbar_wait(&bars.uw_ready, par, &dead, a.status);
                tc_fence_after_sync();
                const uint64_t dKmn = umma_desc(qk + kC * 128, 2 * kC * 128, 1024);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_bf16_ts(tm + kTmS, tm + kTmU + 32 * (k >> 1) + 8 * (k & 1), dKmn + ((k * 16 * 128) >> 4), id5, true);
                umma_commit(&bars.ds_done);
                umma_commit(&bars.tiles_free_qk[b % kQKStages]);
                // (7) O += u^T Ps^T
                if (has_o) {
                    mbar_wait(&bars.p_ready[b % 3], (b / 3) & 1, &dead, a.status);
                    tc_fence_after_sync();
                    const uint64_t dP = umma_desc(smem_u32(sm + kOffP + (b % 3) * (kC * 128)), 0, 1024);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        umma_bf16_ts(tm + kTmO + 64 * par, tm + kTmU + 32 * (k >> 1) + 16 + 8 * (k & 1), dP + 2 * k, idN64, true);
                    umma_commit(&bars.p_free[b % 3]);
                }
                umma_commit(&bars.o_mma_done[b & 3]);
            }
        }
    } else if (warp >= 12) {
        // ======================================================= prep warpgroup: the inverse and its operand, ahead of the chain
        const int x = tid - 384;                 // 0..127
        float *Mf = reinterpret_cast<float *>(sm + kOffM);
        // both X buffers start as zeros: only entries on or below the block diagonal are ever written
        for (int e = x; e < 2 * kC * 128 / 16; e += 128) reinterpret_cast<uint4 *>(sm + kOffX)[e] = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
        for (int b = 0; b < nblk; ++b) {
            const float *sc = gb + (b & 3) * kGbFloats;
            const float *beta = sc + kC;
            // ---- A comes from the mask warpgroup (epilogue of (1))
            mbar_wait(&bars.a_ready[b & 1], (b >> 1) & 1, &dead, a.status);
            // X = M diag(beta) (bf16) is written as the entries of M become final; the buffer of this parity was read by
            // (3b) of block b-2
            if (b >= 2) mbar_wait(&bars.x_free[b & 1], ((b - 2) >> 1) & 1, &dead, a.status);
            unsigned char *xb = sm + kOffX + (b & 1) * (kC * 128);
            named_bar_sync(1, 128);   // every thread is done with the fp32 M of the previous block
            const float *Af = reinterpret_cast<const float *>(sm + kOffA) + (b & 1) * (kC * kLd);
            // ---- M = (I + A)^{-1} by doubling.  Warp w owns the 16x16 diagonal block w up to the 8 -> 16 merge, so that the two
            // steps need no barrier between the warps.  8x8 diagonal blocks 2w, 2w+1: lane (kk, c) solves column c of block
            // 2w + kk by forward substitution (fp32).
            if (lane < 16) {
                const int k = 2 * (warp & 3) + (lane >> 3), c = lane & 7;
                const float *Ab = Af + (8 * k) * kLd + 8 * k;
                float xv[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    float row[8];
#pragma unroll
                    for (int i4 = 0; i4 < 8; i4 += 4) {
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
                for (int t = 0; t < 8; ++t) Mf[(8 * k + t) * kLd + 8 * k + c] = xv[t];
                const float bc = beta[8 * k + c];
#pragma unroll
                for (int t = 0; t < 8; ++t)
                    *reinterpret_cast<__nv_bfloat16 *>(xb + x_offset(8 * k + t, 8 * k + c)) = __float2bfloat16_rn(xv[t] * bc);
            }
            __syncwarp();
            // 8 -> 16 in fp32: thread = (16-block k = this warp, row i, column pair) of the 8x8 block below the diagonal;
            // T = A21 inv(L1) passes through the scratch M[0..31, 32..39]
            {
                const int k = x >> 5, i = (x >> 2) & 7, j0 = 2 * (x & 3);
                const float *a21 = Af + (16 * k + 8 + i) * kLd + 16 * k;
                const float *d1 = Mf + (16 * k) * kLd + 16 * k;
                float t0 = 0.f, t1 = 0.f;
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    const float av = a21[m];
                    t0 = fmaf(av, d1[m * kLd + j0], t0);        // zero where m < j: inv(L1) is lower triangular
                    t1 = fmaf(av, d1[m * kLd + j0 + 1], t1);
                }
                float *ts = Mf + (8 * k) * kLd + 32;
                *reinterpret_cast<float2 *>(ts + i * kLd + j0) = make_float2(t0, t1);
                __syncwarp();
                const float *d2 = Mf + (16 * k + 8 + i) * kLd + 16 * k + 8;
                float m0 = 0.f, m1 = 0.f;
#pragma unroll
                for (int m = 0; m < 8; ++m) {
                    const float dv = d2[m];                       // zero where m > i
                    m0 = fmaf(dv, ts[m * kLd + j0], m0);
                    m1 = fmaf(dv, ts[m * kLd + j0 + 1], m1);
                }
                *reinterpret_cast<float2 *>(Mf + (16 * k + 8 + i) * kLd + 16 * k + j0) = make_float2(-m0, -m1);
                *reinterpret_cast<uint32_t *>(xb + x_offset(16 * k + 8 + i, 16 * k + j0)) =
                    pack_bf16(-m0 * beta[16 * k + j0], -m1 * beta[16 * k + j0 + 1]);
                // the 8x8 block above the diagonal of the 16x16 block reads as part of the operands later: zero
                *reinterpret_cast<float2 *>(Mf + (16 * k + i) * kLd + 16 * k + 8 + j0) = make_float2(0.f, 0.f);
            }
            named_bar_sync(1, 128);
            {
                const int wq = warp & 3, gid = lane >> 2, tig = lane & 3;
                // 16 -> 32: blocks (1, 0) and (3, 2), one half block per warp
                inv_merge32(Af, Mf, xb, beta, 2 * (wq >> 1), wq & 1, gid, tig);
                named_bar_sync(1, 128);
                // 32 -> 64: one 16x16 block of the 32x32 result per warp
                inv_merge64_a(Af, Mf, wq >> 1, wq & 1, gid, tig);
                named_bar_sync(1, 128);
                inv_merge64_b(Mf, xb, beta, wq >> 1, wq & 1, gid, tig);
            }
            fence_async_smem();
            mbar_arrive(&bars.m_ready[b & 1]);
        }
    } else if (warp >= 8) {
        // ======================================================= mask warpgroup: epilogue of (1) and Q scaling, as far ahead of the
        // chain as the buffers allow
        const int x = tid - 256;   // TMEM lane: 0..63 rows of Q K^T (-> Ps), 64..127 rows of K K^T (-> A)
        const int t = x & 63;
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const int row_hi = (t & 32) + 31;   // last row (token) of this warp
        if ((x & 32) == 0) {
            // columns 32..63 of rows 0..31 lie above the diagonal in all Ps and A buffers: zero them once
            float z[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) z[c] = 0.f;
#pragma unroll 1
            for (int i = 0; i < 6; ++i) {
                const int q = 2 + (i & 1), bufi = i >> 1;
                if (x < kC) {
                    store_row_chunks(sm + kOffP + bufi * (kC * 128), t, 2 * q, z);
                } else if (bufi < 2) {
#pragma unroll
                    for (int c = 0; c < 16; c += 4)
                        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(sm + kOffA) + bufi * (kC * kLd) + t * kLd + 16 * q + c) =
                            make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        // outputs of block b: O^T (complete once (7) has run) -> bf16 tile [token][j], lane = j
        __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(a.o);
        const size_t tstride = static_cast<size_t>(a.H_v) * kD;
        auto o_epilogue = [&](int b) {
            mbar_wait(&bars.o_mma_done[b & 3], (b >> 2) & 1, &dead, a.status);
            tc_fence_after_sync();
            const int t0 = t_begin + b * kC;
            const int n = min(kC, t_end - t0);
            if (has_o && (n == kC || !dead)) {
                if (n != kC) {
                    // ragged last block: straight to global memory, 16 tokens of one state column per call
#pragma unroll 1
                    for (int q = 0; q < 4; ++q)
                        store_o_partial(lane_base + kTmO + 64 * (b & 1) + 16 * q, o + (static_cast<size_t>(t0 + 16 * q) * a.H_v + h) * kD + x,
                                        tstride, n - 16 * q);
                } else {
                    // whole block: stage the tile in the V stage of this block, which (3a) has finished reading, in the layout of
                    // the tensor map (two halves of 64 features, 128-byte rows, 128-byte swizzle); the store warp writes it out
                    // with TMA.  O^T leaves tensor memory in accumulator layout (thread = feature, register pair = two tokens) and
                    // is stored transposed, 16 features x 16 tokens per instruction.
                    unsigned char *os = sm + kOffV + (b & 1) * kVStage + (warp & 2 ? kC * 128 : 0);
                    const int m = lane >> 3, i = lane & 7;
#pragma unroll 1
                    for (int lh = 0; lh < 2; ++lh) {
                        uint32_t pu[32];
                        tmem_ld_16x256b_x8(lane_base + (static_cast<uint32_t>(16 * lh) << 16) + kTmO + 64 * (b & 1), pu);
                        tmem_ld_wait();
                        const int chunk = 4 * (warp & 1) + 2 * lh + (m & 1);   // 16-byte piece of the 128-byte row: 8 features
                        const uint32_t row_addr = smem_u32(os) + (8 * (m >> 1) + i) * 128 + ((chunk ^ i) << 4);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)   // tokens 16 kk .. 16 kk + 15
                            stmatrix_x4_trans(row_addr + 16 * kk * 128,
                                              pack_bf16(__uint_as_float(pu[8 * kk]), __uint_as_float(pu[8 * kk + 1])),
                                              pack_bf16(__uint_as_float(pu[8 * kk + 2]), __uint_as_float(pu[8 * kk + 3])),
                                              pack_bf16(__uint_as_float(pu[8 * kk + 4]), __uint_as_float(pu[8 * kk + 5])),
                                              pack_bf16(__uint_as_float(pu[8 * kk + 6]), __uint_as_float(pu[8 * kk + 7])));
                    }
                }
                fence_async_smem();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars.o_done[b & 3]);
            mbar_arrive(&bars.o_staged[b & 1]);
        };
#pragma unroll 1
        for (int b = 0; b < nblk + 3; ++b) {
            // the outputs lag the masks by three blocks: by then the chain has normally produced them
            if (b >= 3) o_epilogue(b - 3);
            if (b >= nblk) continue;
            const float *sc = gb + (b & 3) * kGbFloats;
            mbar_wait(&bars.gb_ready[b & 3], (b >> 2) & 1, &dead, a.status);
            float *Af = reinterpret_cast<float *>(sm + kOffA) + (b & 1) * (kC * kLd);
            unsigned char *ps = sm + kOffP + (b % 3) * (kC * 128);
            if (x < kC) {
                // the Ps buffer is free once (7) of block b-3 has read it
                if (b >= 3 && has_o) mbar_wait(&bars.p_free[b % 3], ((b - 3) / 3) & 1, &dead, a.status);
            } else {
                // the A buffer of this parity is free once block b-2 has been inverted
                if (b >= 2) mbar_wait(&bars.m_ready[b & 1], ((b - 2) >> 1) & 1, &dead, a.status);
            }
            mbar_wait(&bars.g_done[b & 1], (b >> 1) & 1, &dead, a.status);
            tc_fence_after_sync();
            if (x >= kC || has_o) {
                // Gam_ti = 2^{cg2_t - cg2_ref} * f_i with ref the first column of i's group of 16: one exponential
                // per group (both factors' product is <= 1 where i <= t); violent decay takes the per-element path
                const float cgt = sc[t];
                const float coef = (x < kC) ? a.scale : sc[kC + t];     // rows of Ps: the output scale, rows of A: beta_t
                const int lim = (x < kC) ? t : t - 1;                   // P keeps the diagonal, A is strictly lower
                const bool fast = sc[5 * kC] + sc[5 * kC + 1] == 0.f;
                const uint32_t tmg = lane_base + kTmG;
                // column groups above the diagonal for every row of this warp are never touched
#pragma unroll 1
                for (int q = 0; 16 * q <= row_hi; ++q) {
                    const int i0 = 16 * q;
                    if (!fast) {
                        mask_group_exact(tmg + i0, sc, cgt, coef, i0, lim, x < kC, ps, Af + t * kLd, t);
                        continue;
                    }
                    uint32_t rr[16];
                    tmem_ld16(tmg + i0, rr);
                    tmem_ld_wait();
                    float v[16];
                    float aa;
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(aa) : "f"(fminf(cgt - sc[i0], 0.f)));
                    aa *= coef;
                    if (i0 + 15 <= row_hi - 32) {
                        // below the diagonal for every row of this warp: no masking
#pragma unroll
                        for (int c = 0; c < 16; c += 4) {
                            const float4 f = *reinterpret_cast<const float4 *>(sc + 4 * kC + i0 + c);
                            const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(rr[c]), __uint_as_float(rr[c + 1])), __fmul2_rn(make_float2(aa, aa), make_float2(f.x, f.y)));
                            const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(rr[c + 2]), __uint_as_float(rr[c + 3])), __fmul2_rn(make_float2(aa, aa), make_float2(f.z, f.w)));
                            v[c] = p0.x; v[c + 1] = p0.y; v[c + 2] = p1.x; v[c + 3] = p1.y;
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; c += 4) {
                            const float4 f = *reinterpret_cast<const float4 *>(sc + 4 * kC + i0 + c);
                            const float2 p0 = __fmul2_rn(make_float2(__uint_as_float(rr[c]), __uint_as_float(rr[c + 1])), __fmul2_rn(make_float2(aa, aa), make_float2(f.x, f.y)));
                            const float2 p1 = __fmul2_rn(make_float2(__uint_as_float(rr[c + 2]), __uint_as_float(rr[c + 3])), __fmul2_rn(make_float2(aa, aa), make_float2(f.z, f.w)));
                            v[c] = (i0 + c <= lim) ? p0.x : 0.f;
                            v[c + 1] = (i0 + c + 1 <= lim) ? p0.y : 0.f;
                            v[c + 2] = (i0 + c + 2 <= lim) ? p1.x : 0.f;
                            v[c + 3] = (i0 + c + 3 <= lim) ? p1.y : 0.f;
                        }
                    }
                    if (x < kC) {
                        store_row_chunks(ps, t, 2 * q, v);
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; c += 4)
                            *reinterpret_cast<float4 *>(Af + t * kLd + i0 + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                    }
                }
            }
            tc_fence_before_sync();
            if (x < kC) {
                fence_async_smem();
                mbar_arrive(&bars.p_ready[b % 3]);
            } else {
                mbar_arrive(&bars.a_ready[b & 1]);
            }
        }
    } else {
        // ======================================================= chain warpgroups: lane = state column j, `half` = token / row half
        const int j = tid & 127, half = warp >> 2;
        const uint32_t lane_base = tm + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        // initial state: S0[m][j], m = 64*half..+63 -> TMEM (fp32, pre-scaled by gam_C of block 0) and bf16 pairs
        mbar_wait(&bars.gb_ready[0], 0, &dead, a.status);
        {
            const float gamC = gb[2 * kC + kC - 1];
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                float v[16];
                uint32_t rr[16], w[8];
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    const int m = 64 * half + 16 * q + c;
                    v[c] = s0_id ? (m == j ? 1.f : 0.f) : (a.S0 ? a.S0[sbase + static_cast<size_t>(m) * kD + j] : 0.f);
                    rr[c] = __float_as_uint(v[c] * gamC);
                }
                tmem_st16(lane_base + kTmS + 64 * half + 16 * q, rr);
                pack16(v, w);
                tmem_st8(lane_base + kTmSb + 32 * half + 8 * q, w);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars.st_ready);
        }
#pragma unroll 1
        for (int b = 0; b < nblk; ++b) {
            const uint32_t par = b & 1;
            const float *sc = gb + (b & 3) * kGbFloats;
            if (b > 0) mbar_wait(&bars.gb_ready[b & 3], (b >> 2) & 1, &dead, a.status);
            mbar_wait(&bars.ks_done, par, &dead, a.status);
            tc_fence_after_sync();
            // Rk_t[j] = -gam_t (S^T k_t)_j, t = 32*half..+31 -> bf16 pairs over the first half of this thread's own columns
            {
                uint32_t rr[2][16], w[2][8];
                tmem_ld16(lane_base + kTmKS + 32 * half, rr[0]);
                tmem_ld16(lane_base + kTmKS + 32 * half + 16, rr[1]);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; c += 4) {
                        const float4 ga = *reinterpret_cast<const float4 *>(sc + 2 * kC + 32 * half + 16 * q + c);
                        const float2 p0 = __fmul2_rn(make_float2(-ga.x, -ga.y), make_float2(__uint_as_float(rr[q][c]), __uint_as_float(rr[q][c + 1])));
                        const float2 p1 = __fmul2_rn(make_float2(-ga.z, -ga.w), make_float2(__uint_as_float(rr[q][c + 2]), __uint_as_float(rr[q][c + 3])));
                        v[c] = p0.x; v[c + 1] = p0.y; v[c + 2] = p1.x; v[c + 3] = p1.y;
                    }
                    pack16(v, w[q]);
                }
                tmem_st8(lane_base + kTmKS + 32 * half, w[0]);
                tmem_st8(lane_base + kTmKS + 32 * half + 8, w[1]);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars.rk_ready);
            // While (3b) is on its way: the Q tile of block b scaled in place by scale gam_t for (2Q).  (1) has read the tile
            // once the block's inverse is ready (the mask epilogue came before it); thread = (token, quarter of the row).
            if (has_o) {
                mbar_wait(&bars.m_ready[b & 1], (b >> 1) & 1, &dead, a.status);
                mbar_wait(&bars.full_qk[b % kQKStages], (b / kQKStages) & 1, &dead, a.status);   // this thread reads what the TMA wrote
                scale_q_quarter(sm + (b % kQKStages) * kQKStage, tid, a.scale * sc[2 * kC + (tid & 63)]);
                fence_async_smem();
                mbar_arrive(&bars.qs_ready[b % kQKStages]);
            }
            // u_t[j], tokens 32*half..+31 -> Uw = w o u as bf16 pairs over the first 16 of this thread's own 32 columns, u over the rest
            mbar_wait(&bars.u_done, par, &dead, a.status);
            tc_fence_after_sync();
            {
                uint32_t rr[2][16], w[2][8], u[2][8];
                tmem_ld16(lane_base + kTmU + 32 * half, rr[0]);
                tmem_ld16(lane_base + kTmU + 32 * half + 16, rr[1]);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    float v[16];
#pragma unroll
                    for (int c = 0; c < 16; c += 4) {
                        const float4 w4 = *reinterpret_cast<const float4 *>(sc + 3 * kC + 32 * half + 16 * q + c);
                        const float2 p0 = __fmul2_rn(make_float2(w4.x, w4.y), make_float2(__uint_as_float(rr[q][c]), __uint_as_float(rr[q][c + 1])));
                        const float2 p1 = __fmul2_rn(make_float2(w4.z, w4.w), make_float2(__uint_as_float(rr[q][c + 2]), __uint_as_float(rr[q][c + 3])));
                        v[c] = p0.x; v[c + 1] = p0.y; v[c + 2] = p1.x; v[c + 3] = p1.y;
                    }
                    pack16(v, w[q]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) u[q][e] = pack_bf16(__uint_as_float(rr[q][2 * e]), __uint_as_float(rr[q][2 * e + 1]));
                }
                tmem_st8(lane_base + kTmU + 32 * half, w[0]);
                tmem_st8(lane_base + kTmU + 32 * half + 8, w[1]);
                tmem_st8(lane_base + kTmU + 32 * half + 16, u[0]);
                tmem_st8(lane_base + kTmU + 32 * half + 24, u[1]);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars.uw_ready);
            // new state rows m = 64*half..+63: bf16 pairs for the next block and pre-scale by its gam_C, or S_T at the end
            const bool last = b + 1 == nblk;
            float gamN = 1.f;
            if (!last) {
                mbar_wait(&bars.gb_ready[(b + 1) & 3], ((b + 1) >> 2) & 1, &dead, a.status);
                gamN = gb[((b + 1) & 3) * kGbFloats + 2 * kC + kC - 1];
            }
            mbar_wait(&bars.ds_done, par, &dead, a.status);
            tc_fence_after_sync();
            if (last) {
                // where this sequence's final state goes: a transition sequence may have a buffer of its own
                const bool own = seq >= a.tr_first && a.tr_out != nullptr;
                float *ST = own ? a.tr_out : a.S_T;
                const size_t obase = own ? (static_cast<size_t>(seq - a.tr_first) * a.H_v + h) * kD * kD : sbase;
                if (ST && !dead) {
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) {
                        uint32_t rr[16];
                        tmem_ld16(lane_base + kTmS + 64 * half + 16 * q, rr);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const size_t e = static_cast<size_t>(64 * half + 16 * q + c) * kD + j;
                            store_state(ST, a.st_bf16, obase + e, __uint_as_float(rr[c]) + (a.S_add ? a.S_add[sbase + e] : 0.f));
                        }
                    }
                }
            } else {
                uint32_t rr[4][16];
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld16(lane_base + kTmS + 64 * half + 16 * q, rr[q]);
                tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t w[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(rr[q][2 * e]), __uint_as_float(rr[q][2 * e + 1]));
                    tmem_st8(lane_base + kTmSb + 32 * half + 8 * q, w);
                }
#pragma unroll
                for (int q = 0; q < 4; ++q) {
#pragma unroll
                    for (int c = 0; c < 16; c += 2) {
                        const float2 p = __fmul2_rn(make_float2(gamN, gamN), make_float2(__uint_as_float(rr[q][c]), __uint_as_float(rr[q][c + 1])));
                        rr[q][c] = __float_as_uint(p.x);
                        rr[q][c + 1] = __float_as_uint(p.y);
                    }
                    tmem_st16(lane_base + kTmS + 64 * half + 16 * q, rr[q]);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(&bars.st_ready);
            }
            mbar_arrive(&bars.chain_done[b & 3]);
        }
    }
    grace_after_timeout(&dead);
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
    if (rows == 0) {
        // no token anywhere: every CTA hands its state through and never touches a tile (and a map of zero rows
        // cannot be encoded)
        memset(&mapQ, 0, sizeof(mapQ));
        mapK = mapV = mapO = mapQ;
    } else if (!make_tensor_map_2d(&mapQ, a.q, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        !make_tensor_map_2d(&mapK, a.k, 2, qk_inner, rows, qk_inner * 2, 64, kC, true) ||
        (a.v && !make_tensor_map_2d(&mapV, a.v, 2, v_inner, rows, v_inner * 2, 64, kC, true)) ||
        (a.o && !make_tensor_map_2d(&mapO, a.o, 2, v_inner, rows, v_inner * 2, 64, kC, true)))
        return cudaErrorInvalidValue;
    if (!a.v) mapV = mapK;   // never used by the kernel then
    if (!a.o) mapO = mapK;
    cudaError_t e = cudaFuncSetAttribute(gdn_scan_tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    gdn_scan_tensor_kernel<<<dim3(a.H_v, a.n_seq), kThreads, kSmemBytes, s>>>(a, mapQ, mapK, mapV, mapO);
    return cudaGetLastError();
}

}  // namespace lkv
