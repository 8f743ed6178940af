// C-ABI entry points: argument validation, index marshalling and kernel selection.
// Everything that can be wrong with a call is found here, on the host, before a launch.
#include <string.h>

#include <algorithm>
#include <vector>

#include "common.cuh"

using namespace lkv;

namespace {

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool dtype_ok(int d) { return d == LKV_DTYPE_F32 || d == LKV_DTYPE_BF16; }
inline bool compute_ok(int c) { return c == LKV_COMPUTE_AUTO || c == LKV_COMPUTE_FP32 || c == LKV_COMPUTE_TENSOR; }

// Byte ranges [p, p + n) and [q, q + m) share at least one byte (empty or NULL ranges never do).
inline bool overlaps(const void *p, size_t n, const void *q, size_t m) {
    if (!p || !q || n == 0 || m == 0) return false;
    const uintptr_t a = reinterpret_cast<uintptr_t>(p), b = reinterpret_cast<uintptr_t>(q);
    return a < b + m && b < a + n;
}

size_t ws_bytes_for(int n_ints, int cap) {
    return kWsHeaderBytes + (n_ints > cap ? align_up(sizeof(int32_t) * static_cast<size_t>(n_ints), 256) : 0);
}

// Puts `ints` where the kernels will find them: inline in the parameter block when they
// fit, otherwise one small async copy into the workspace behind its header.
template <int CAP>
int place_indices(IndexBlock<CAP> &blk, const std::vector<int32_t> &ints, void *workspace, cudaStream_t s) {
    if (static_cast<int>(ints.size()) <= CAP) {
        blk.ptr = nullptr;
        if (!ints.empty()) memcpy(blk.v, ints.data(), sizeof(int32_t) * ints.size());
        return LKV_OK;
    }
    // The copy reads a host array that dies with this call: a stream capture would record the read, not do it.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) {
        cudaGetLastError();
        return LKV_ERR_CUDA;
    }
    if (cap != cudaStreamCaptureStatusNone) return LKV_ERR_UNSUPPORTED;
    int32_t *dst = reinterpret_cast<int32_t *>(static_cast<char *>(workspace) + kWsHeaderBytes);
    if (cudaMemcpyAsync(dst, ints.data(), sizeof(int32_t) * ints.size(), cudaMemcpyHostToDevice, s) != cudaSuccess) {
        cudaGetLastError();
        return LKV_ERR_CUDA;
    }
    blk.ptr = dst;
    return LKV_OK;
}

int check_init_desc(const lkv_init_desc *d) {
    if (!d) return LKV_ERR_NULL;
    if (d->family != LKV_FAMILY_MAMBA2 && d->family != LKV_FAMILY_GDN) return LKV_ERR_MODE;
    if (!dtype_ok(d->state_dtype) || !compute_ok(d->compute)) return LKV_ERR_MODE;
    if (d->H < 1 || d->d_k < 1 || d->d_v < 1 || d->n_chunks < 0) return LKV_ERR_DIM;
    return LKV_OK;
}

int init_impl(const void *states, const void *transitions, const int32_t *chunk_ids, const int32_t *cu_k,
              int n_req, int mode, const int32_t *sel_index, void *S0, const lkv_init_desc *d, void *stream) {
    int st = check_init_desc(d);
    if (st != LKV_OK) return st;
    if (mode != LKV_INIT_LAST && mode != LKV_INIT_INDEX && mode != LKV_INIT_EXACT) return LKV_ERR_MODE;
    if (n_req < 0) return LKV_ERR_DIM;
    if (!cu_k) return LKV_ERR_NULL;
    if (cu_k[0] != 0) return LKV_ERR_INDEX;
    int max_k = 0;
    for (int r = 0; r < n_req; ++r) {
        if (cu_k[r + 1] < cu_k[r]) return LKV_ERR_INDEX;
        max_k = cu_k[r + 1] - cu_k[r] > max_k ? cu_k[r + 1] - cu_k[r] : max_k;
    }
    const int total = cu_k[n_req];
    if (total > 0 && !chunk_ids) return LKV_ERR_NULL;
    for (int i = 0; i < total; ++i)
        if (chunk_ids[i] < 0 || chunk_ids[i] >= d->n_chunks) return LKV_ERR_INDEX;
    if (mode == LKV_INIT_INDEX) {
        if (n_req > 0 && !sel_index) return LKV_ERR_NULL;
        for (int r = 0; r < n_req; ++r) {
            const int K = cu_k[r + 1] - cu_k[r];
            if (K > 0 && (sel_index[r] < 0 || sel_index[r] >= K)) return LKV_ERR_INDEX;
        }
    }
    if (n_req == 0) return LKV_OK;
    if (!S0) return LKV_ERR_NULL;
    if (total > 0 && !states) return LKV_ERR_NULL;
    const bool exact = mode == LKV_INIT_EXACT && max_k >= 2;
    if (exact && !transitions) return LKV_ERR_NULL;
    if (!aligned16(S0) || !aligned16(states) || (exact && !aligned16(transitions))) return LKV_ERR_ALIGN;
    const bool pool_bf16 = d->state_dtype == LKV_DTYPE_BF16;
    {
        const size_t state_elems = static_cast<size_t>(d->H) * d->d_k * d->d_v;
        const size_t out_bytes = sizeof(float) * state_elems * n_req;
        const size_t pool_bytes = (pool_bf16 ? 2 : 4) * state_elems * d->n_chunks;
        const size_t tr_bytes = sizeof(float) * static_cast<size_t>(d->n_chunks) * d->H *
                                (d->family == LKV_FAMILY_GDN ? static_cast<size_t>(d->d_k) * d->d_k : 1);
        if (overlaps(S0, out_bytes, states, total > 0 ? pool_bytes : 0) || (exact && overlaps(S0, out_bytes, transitions, tr_bytes)))
            return LKV_ERR_OVERLAP;
    }
    if (d->d_v % (pool_bf16 ? 8 : 4) != 0) return LKV_ERR_UNSUPPORTED;

    const int n_ints = (n_req + 1) + (mode == LKV_INIT_INDEX ? n_req : 0) + total;
    if (!d->workspace || d->workspace_bytes < ws_bytes_for(n_ints, kInitIdxCap)) return LKV_ERR_WORKSPACE;
    if (!aligned16(d->workspace)) return LKV_ERR_ALIGN;

    InitArgs a;
    a.states = states;
    a.transitions = static_cast<const float *>(transitions);
    a.S0 = static_cast<float *>(S0);
    a.n_req = n_req;
    a.H = d->H;
    a.d_k = d->d_k;
    a.d_v = d->d_v;
    a.n_chunks = d->n_chunks;
    a.status = static_cast<int32_t *>(d->workspace);
    std::vector<int32_t> ints;
    ints.reserve(n_ints);
    ints.insert(ints.end(), cu_k, cu_k + n_req + 1);
    a.off_sel = -1;
    if (mode == LKV_INIT_INDEX) {
        a.off_sel = static_cast<int32_t>(ints.size());
        ints.insert(ints.end(), sel_index, sel_index + n_req);
    }
    a.off_ids = static_cast<int32_t>(ints.size());
    if (total > 0) ints.insert(ints.end(), chunk_ids, chunk_ids + total);

    // kernel choice (no launch has happened yet: an unsupported request leaves everything untouched)
    enum { kSingle, kMamba, kGdnFp32, kGdnTensor } which;
    if (!exact) {
        which = kSingle;  // LAST, INDEX, and EXACT with K <= 1 everywhere are plain copies
        a.off_sel = (mode == LKV_INIT_INDEX) ? a.off_sel : -1;
    } else if (d->family == LKV_FAMILY_MAMBA2) {
        which = kMamba;
    } else {
        const bool tensor_fits = init_gdn_exact_tensor_supported(a, pool_bf16);
        if (d->compute == LKV_COMPUTE_TENSOR && !tensor_fits) return LKV_ERR_UNSUPPORTED;
        which = (d->compute != LKV_COMPUTE_FP32 && tensor_fits) ? kGdnTensor : kGdnFp32;
        if (which == kGdnFp32 && (2 * d->d_k * 32 + 32 * (d->d_k + 1)) * sizeof(float) > 227 * 1024) return LKV_ERR_UNSUPPORTED;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = place_indices(a.idx, ints, d->workspace, s);
    if (st != LKV_OK) return st;
    cudaError_t e = cudaSuccess;
    switch (which) {
        case kSingle: e = launch_init_single(a, pool_bf16, s); break;
        case kMamba:
            e = init_mamba_stream_supported(a, pool_bf16) ? launch_init_mamba_exact_stream(a, pool_bf16, s)
                                                          : launch_init_mamba_exact(a, pool_bf16, s);
            break;
        case kGdnFp32: e = launch_init_gdn_exact_fp32(a, pool_bf16, s); break;
        case kGdnTensor: e = launch_init_gdn_exact_tensor(a, pool_bf16, s); break;
    }
    return e == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

// Shared checks of the two scan descriptors' sequence layout; fills `cu` with the
// offsets the kernels will use.
int check_seqs(int T_total, int n_seq, const int32_t *cu_seqlens, std::vector<int32_t> &cu) {
    if (T_total < 0 || n_seq < 0) return LKV_ERR_DIM;
    if (!cu_seqlens) {
        if (n_seq != 1) return LKV_ERR_NULL;
        cu = {0, T_total};
        return LKV_OK;
    }
    if (cu_seqlens[0] != 0 || cu_seqlens[n_seq] != T_total) return LKV_ERR_INDEX;
    for (int i = 0; i < n_seq; ++i)
        if (cu_seqlens[i + 1] < cu_seqlens[i]) return LKV_ERR_INDEX;
    cu.assign(cu_seqlens, cu_seqlens + n_seq + 1);
    return LKV_OK;
}

// Appends to cu[n_seq + 1] the launch order of the sequences: longest first (ties by index), so that the CTAs of the
// long sequences, which are scheduled in grid order, start first and the short ones fill the tail of the launch.
void append_launch_order(std::vector<int32_t> &cu, int n_seq) {
    std::vector<int32_t> order(n_seq);
    for (int i = 0; i < n_seq; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t x, int32_t y) { return cu[x + 1] - cu[x] > cu[y + 1] - cu[y]; });
    cu.insert(cu.end(), order.begin(), order.end());
}

}  // namespace

extern "C" {

int lkv_init_state(const void *states, const void *transitions, int K, int mode, void *S0,
                   const lkv_init_desc *d, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (K < 0) return LKV_ERR_DIM;
    std::vector<int32_t> ids;
    const int32_t *idp = d->chunk_ids;
    if (!idp) {
        ids.resize(K);
        for (int i = 0; i < K; ++i) ids[i] = i;
        idp = ids.data();
    }
    const int32_t cu_k[2] = {0, K};
    const int32_t sel[1] = {d->sel_index};
    return init_impl(states, transitions, idp, cu_k, 1, mode, sel, S0, d, stream);
}

int lkv_init_state_batched(const void *states, const void *transitions, const int32_t *chunk_ids,
                           const int32_t *cu_k, int n_req, int mode, const int32_t *sel_index, void *S0,
                           const lkv_init_desc *d, void *stream) {
    return init_impl(states, transitions, chunk_ids, cu_k, n_req, mode, sel_index, S0, d, stream);
}

// lkv_gdn_fwd, and with `transition` set the scan from S = I with v = 0 whose final state is the chunk transition
// what: 0 = scan, 1 = chunk transitions (start from S = I, v read as zeros), 2 = one step of the online fold (v read as
// zeros, S_add added to the final state), 3 = local states and transitions in one launch: d->n_seq = 2 m - 1 sequences,
// the first m of them scans over the m ranges of d->cu_seqlens (m + 1 entries), the other m - 1 the transitions of ranges
// 1 .. m-1 (the kernels' "transition sequences")
// 4 = local states and transitions of every sequence in one launch: d->n_seq = 2 m sequences over the m ranges of
// d->cu_seqlens, the last m of them transition sequences that write to tr_out
static int gdn_impl(const void *q, const void *k, const void *v, const float *g, const float *beta,
                    const float *S0, void *o, void *S_T, const lkv_gdn_desc *d, void *stream, int what,
                    const float *S_add = nullptr, float *tr_out = nullptr) {
    const bool transition = what == 1;
    if (!d) return LKV_ERR_NULL;
    if (!dtype_ok(d->io_dtype) || !compute_ok(d->compute) || !dtype_ok(d->state_dtype)) return LKV_ERR_MODE;
    const bool st_bf16 = d->state_dtype == LKV_DTYPE_BF16;
    if (st_bf16 && S_T && S_T == S0) return LKV_ERR_OVERLAP;   // an fp32 input cannot be a bf16 output
    if (d->H_k < 1 || d->H_v < 1 || d->d_k < 1 || d->d_v < 1 || d->H_v % d->H_k != 0) return LKV_ERR_DIM;
    std::vector<int32_t> cu;
    const int n_ranges = what == 3 ? (d->n_seq + 1) / 2 : what == 4 ? d->n_seq / 2 : d->n_seq;
    int st = check_seqs(d->T_total, n_ranges, d->cu_seqlens, cu);
    if (st != LKV_OK) return st;
    if (d->n_seq == 0) return LKV_OK;
    if ((transition || what >= 3) && d->d_k != d->d_v) return LKV_ERR_DIM;
    if (d->T_total > 0 && (!q || !k || !g || !beta)) return LKV_ERR_NULL;
    if (what == 0 && d->T_total > 0 && !v) return LKV_ERR_NULL;
    if (!o && !S_T) return LKV_ERR_NULL;   // nothing to compute
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) || !aligned16(S0) ||
        !aligned16(o) || !aligned16(S_T))
        return LKV_ERR_ALIGN;
    if (!d->workspace || d->workspace_bytes < ws_bytes_for(2 * d->n_seq + 1, kScanIdxCap)) return LKV_ERR_WORKSPACE;
    if (!aligned16(d->workspace)) return LKV_ERR_ALIGN;
    {
        // outputs may not overlap inputs (S_T == S0 exactly is the one allowed alias) nor each other
        const size_t es = d->io_dtype == LKV_DTYPE_BF16 ? 2 : 4, T = static_cast<size_t>(d->T_total);
        const size_t qk_b = es * T * d->H_k * d->d_k, v_b = es * T * d->H_v * d->d_v, gb_b = sizeof(float) * T * d->H_v;
        const size_t st_in = sizeof(float) * static_cast<size_t>(what == 4 ? n_ranges : d->n_seq) * d->H_v * d->d_k * d->d_v;
        const size_t st_b = st_bf16 ? st_in / 2 : st_in;
        const void *in[6] = {q, k, v, g, beta, S0};
        const size_t in_b[6] = {qk_b, qk_b, v ? v_b : 0, gb_b, gb_b, S0 ? st_in : 0};
        for (int i = 0; i < 6; ++i) {
            if (overlaps(o, o ? v_b : 0, in[i], in_b[i])) return LKV_ERR_OVERLAP;
            if (!(i == 5 && S_T == S0) && overlaps(S_T, S_T ? st_b : 0, in[i], in_b[i])) return LKV_ERR_OVERLAP;
        }
        if (overlaps(o, o ? v_b : 0, S_T, S_T ? st_b : 0)) return LKV_ERR_OVERLAP;
    }

    GdnArgs a;
    a.q = q; a.k = k; a.v = v; a.g = g; a.beta = beta; a.S0 = S0; a.o = o; a.S_T = static_cast<float *>(S_T);
    a.S_add = S_add; a.st_bf16 = st_bf16 ? 1 : 0;
    a.n_seq = d->n_seq; a.T_total = d->T_total; a.H_k = d->H_k; a.H_v = d->H_v; a.d_k = d->d_k; a.d_v = d->d_v;
    a.scale = d->scale != 0.f ? d->scale : 1.0f / sqrtf(static_cast<float>(d->d_k));
    a.s0_identity = transition ? 1 : 0;
    a.n_ranges = n_ranges; a.tr_first = n_ranges; a.tr_src0 = what == 3 ? 1 : 0; a.tr_out = tr_out;
    a.status = static_cast<int32_t *>(d->workspace);
    const bool io_bf16 = d->io_dtype == LKV_DTYPE_BF16;
    const bool tensor_fits = gdn_scan_tensor_supported(a, io_bf16);
    const bool fp32_fits = gdn_scan_fp32_supported(d->d_k, d->d_v);
    bool use_tensor;
    if (d->compute == LKV_COMPUTE_TENSOR) {
        if (!tensor_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = true;
    } else if (d->compute == LKV_COMPUTE_FP32) {
        if (!fp32_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = false;
    } else {
        if (!tensor_fits && !fp32_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = tensor_fits;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (what >= 3) {
        // launch order over all sequences, longest first; transition sequence j runs over range j - m + (1 or 0)
        std::vector<int32_t> order(d->n_seq);
        auto len = [&](int sq) { const int r = sq < n_ranges ? sq : sq - n_ranges + (what == 3 ? 1 : 0); return cu[r + 1] - cu[r]; };
        for (int i = 0; i < d->n_seq; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return len(x) > len(y); });
        cu.insert(cu.end(), order.begin(), order.end());
    } else {
        append_launch_order(cu, d->n_seq);
    }
    st = place_indices(a.cu, cu, d->workspace, s);
    if (st != LKV_OK) return st;
    const cudaError_t e = use_tensor ? launch_gdn_scan_tensor(a, s) : launch_gdn_scan_fp32(a, io_bf16, s);
    return e == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

int lkv_gdn_fwd(const void *q, const void *k, const void *v, const float *g, const float *beta,
                const float *S0, void *o, void *S_T, const lkv_gdn_desc *d, void *stream) {
    return gdn_impl(q, k, v, g, beta, S0, o, S_T, d, stream, 0);
}

int lkv_gdn_chunk_transition(const void *k, const float *g, const float *beta, float *transitions,
                             const lkv_gdn_desc *d, void *stream) {
    if (d && d->n_seq > 0 && !transitions) return LKV_ERR_NULL;
    // q is not needed for the state: the key tensor stands in for it (its read-outs are not written)
    if (d && d->state_dtype != LKV_DTYPE_F32) return LKV_ERR_MODE;   // transitions are fp32
    return gdn_impl(k, k, nullptr, g, beta, nullptr, nullptr, transitions, d, stream, 1);
}

int lkv_init_state_fold(const void *states, const void *k, const float *g, const float *beta,
                        const int32_t *cu_tokens, int K, void *S0, const lkv_init_desc *d, int H_k, int io_dtype,
                        void *stream) {
    int st = check_init_desc(d);
    if (st != LKV_OK) return st;
    if (d->family != LKV_FAMILY_GDN || !dtype_ok(io_dtype)) return LKV_ERR_MODE;
    if (d->state_dtype != LKV_DTYPE_F32) return LKV_ERR_UNSUPPORTED;   // the cached states are added in fp32
    if (K < 0 || H_k < 1 || d->H % H_k != 0 || d->d_k != d->d_v) return LKV_ERR_DIM;
    if (!states || !S0 || !cu_tokens) return LKV_ERR_NULL;
    if (K > 0 && !d->chunk_ids && K > d->n_chunks) return LKV_ERR_INDEX;
    if (cu_tokens[0] != 0) return LKV_ERR_INDEX;
    for (int c = 0; c < d->n_chunks; ++c)
        if (cu_tokens[c + 1] < cu_tokens[c]) return LKV_ERR_INDEX;
    std::vector<int32_t> ids(K);
    for (int j = 0; j < K; ++j) {
        ids[j] = d->chunk_ids ? d->chunk_ids[j] : j;
        if (ids[j] < 0 || ids[j] >= d->n_chunks) return LKV_ERR_INDEX;
    }
    if (K >= 2 && cu_tokens[d->n_chunks] > 0 && (!k || !g || !beta)) return LKV_ERR_NULL;
    // the first chunk's state (or the zero state) through the single-state path, then one scan per later chunk
    lkv_init_desc first = *d;
    first.sel_index = 0;
    st = lkv_init_state(states, nullptr, K, LKV_INIT_INDEX, S0, &first, stream);
    if (st != LKV_OK) return st;
    const size_t es = io_dtype == LKV_DTYPE_BF16 ? 2 : 4;
    const size_t state_elems = static_cast<size_t>(d->H) * d->d_k * d->d_v;
    for (int j = 1; j < K; ++j) {
        const int c = ids[j], t0 = cu_tokens[c], len = cu_tokens[c + 1] - t0;
        lkv_gdn_desc sd{};
        sd.T_total = len; sd.n_seq = 1; sd.cu_seqlens = nullptr; sd.H_k = H_k; sd.H_v = d->H; sd.d_k = d->d_k; sd.d_v = d->d_v;
        sd.io_dtype = io_dtype; sd.compute = d->compute; sd.scale = 0.f; sd.state_dtype = LKV_DTYPE_F32;
        sd.workspace = d->workspace; sd.workspace_bytes = d->workspace_bytes;
        const char *kc = static_cast<const char *>(k) + es * static_cast<size_t>(t0) * H_k * d->d_k;
        const float *gc = g ? g + static_cast<size_t>(t0) * d->H : nullptr;
        const float *bc = beta ? beta + static_cast<size_t>(t0) * d->H : nullptr;
        st = gdn_impl(kc, kc, nullptr, gc, bc, static_cast<const float *>(S0), nullptr, S0, &sd, stream, 2,
                      static_cast<const float *>(states) + static_cast<size_t>(c) * state_elems);
        if (st != LKV_OK) return st;
    }
    return LKV_OK;
}

// n_segments == 0: as many segments as keep both scanning passes within one round of CTAs on this GPU -- (2 n - 3) H_v and
// n H_v CTAs, one per SM -- and no segment shorter than 512 tokens
static int auto_segments(const lkv_gdn_desc *d) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        sms = 148;
    }
    int n = (sms / (d->H_v > 0 ? d->H_v : 1) + 3) / 2;
    if (n > d->T_total / 512) n = d->T_total / 512;
    return n < 1 ? 1 : n;
}

size_t lkv_gdn_segmented_scratch_bytes(const lkv_gdn_desc *d, int n_segments) {
    if (!d || n_segments < 0 || d->H_v < 1 || d->d_k < 1 || d->d_v < 1) return 0;
    if (n_segments == 0) n_segments = auto_segments(d);
    if (n_segments < 2) return 0;
    return sizeof(float) * static_cast<size_t>(4 * n_segments - 3) * d->H_v * d->d_k * d->d_v;
}

int lkv_gdn_fwd_segmented(const void *q, const void *k, const void *v, const float *g, const float *beta,
                          const float *S0, void *o, void *S_T, const lkv_gdn_desc *d, int n_segments,
                          void *scratch, size_t scratch_bytes, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (n_segments < 0) return LKV_ERR_DIM;
    if (n_segments == 0) {
        if (d->H_v < 1 || d->T_total < 0) return LKV_ERR_DIM;
        n_segments = auto_segments(d);
    }
    if (n_segments == 1) return lkv_gdn_fwd(q, k, v, g, beta, S0, o, S_T, d, stream);
    if (d->n_seq != 1 || d->state_dtype != LKV_DTYPE_F32) return LKV_ERR_UNSUPPORTED;   // one sequence, fp32 final state
    if (d->d_k != d->d_v) return LKV_ERR_DIM;                                            // transitions are d_k x d_k
    if (d->T_total < 0) return LKV_ERR_DIM;
    if (d->cu_seqlens && (d->cu_seqlens[0] != 0 || d->cu_seqlens[1] != d->T_total)) return LKV_ERR_INDEX;
    if (!scratch || scratch_bytes < lkv_gdn_segmented_scratch_bytes(d, n_segments)) return LKV_ERR_WORKSPACE;
    if (!aligned16(scratch)) return LKV_ERR_ALIGN;
    if (!o && !S_T) return LKV_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n_seg = n_segments, n_st = n_seg - 1;
    const size_t slot = static_cast<size_t>(d->H_v) * d->d_k * d->d_v;   // floats per state of all heads
    float *pool = static_cast<float *>(scratch);                        // S_local of segments 0 .. n_st-1, then T of 1 .. n_st-1
    float *trans = pool + (static_cast<size_t>(n_st) - 1) * slot;       // T of segment j at trans + j slots (slot 0 is never read)
    float *S_init = pool + (2 * static_cast<size_t>(n_st) - 1) * slot;  // [n_seg]
    float *S_fin = S_init + static_cast<size_t>(n_seg) * slot;          // [n_seg]; first the initial states of pass 1
    // segment boundaries on multiples of 64 tokens, so that every block of the segmented scan is a block of the plain one
    const int per = ((d->T_total + n_seg - 1) / n_seg + 63) / 64 * 64;
    std::vector<int32_t> bounds(n_seg + 1);
    for (int i = 0; i <= n_seg; ++i) bounds[i] = std::min<long long>(static_cast<long long>(i) * per, d->T_total);
    // ---- pass 1: local states of segments 0 .. n_st-1 (segment 0 from S0) and transitions of segments 1 .. n_st-1, one launch
    if (cudaMemsetAsync(S_fin, 0, sizeof(float) * slot * n_st, s) != cudaSuccess) return LKV_ERR_CUDA;
    if (S0 && cudaMemcpyAsync(S_fin, S0, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LKV_ERR_CUDA;
    lkv_gdn_desc d1 = *d;
    d1.n_seq = 2 * n_st - 1;
    d1.T_total = bounds[n_st];
    d1.cu_seqlens = bounds.data();
    int st = gdn_impl(q, k, v, g, beta, S_fin, nullptr, pool, &d1, stream, 3);
    if (st != LKV_OK) return st;
    // ---- pass 2: the state each segment starts from, by exact composition (Eq. 6) over the segments before it
    if (S0) {
        if (cudaMemcpyAsync(S_init, S0, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LKV_ERR_CUDA;
    } else if (cudaMemsetAsync(S_init, 0, sizeof(float) * slot, s) != cudaSuccess) {
        return LKV_ERR_CUDA;
    }
    {
        std::vector<int32_t> ids, cu_k(n_st + 1, 0);
        for (int r = 0; r < n_st; ++r) {
            for (int j = 0; j <= r; ++j) ids.push_back(j);
            cu_k[r + 1] = static_cast<int32_t>(ids.size());
        }
        lkv_init_desc di{};
        di.family = LKV_FAMILY_GDN; di.H = d->H_v; di.d_k = d->d_k; di.d_v = d->d_v; di.n_chunks = n_st;
        di.state_dtype = LKV_DTYPE_F32; di.sel_index = 0; di.compute = d->compute; di.chunk_ids = nullptr;
        di.workspace = d->workspace; di.workspace_bytes = d->workspace_bytes;
        st = lkv_init_state_batched(pool, trans, ids.data(), cu_k.data(), n_st, LKV_INIT_EXACT, nullptr, S_init + slot, &di, stream);
        if (st != LKV_OK) return st;
    }
    // ---- pass 3: every segment scanned from its initial state, all at once
    lkv_gdn_desc d3 = *d;
    d3.n_seq = n_seg;
    d3.cu_seqlens = bounds.data();
    st = gdn_impl(q, k, v, g, beta, S_init, o, S_fin, &d3, stream, 0);
    if (st != LKV_OK) return st;
    if (S_T && cudaMemcpyAsync(S_T, S_fin + static_cast<size_t>(n_seg - 1) * slot, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return LKV_ERR_CUDA;
    return LKV_OK;
}

int lkv_stage_chunks(const void *host_states, const void *host_transitions, const int32_t *chunk_ids, int n_ids,
                     void *dev_states, void *dev_transitions, int capacity, int32_t *staged_ids, int32_t *n_staged,
                     const lkv_init_desc *d, void *stream) {
    int st = check_init_desc(d);
    if (st != LKV_OK) return st;
    if (n_ids < 0 || capacity < 0) return LKV_ERR_DIM;
    if (!n_staged) return LKV_ERR_NULL;
    *n_staged = 0;
    if (n_ids == 0) return LKV_OK;
    if (!host_states || !dev_states || !chunk_ids || !staged_ids) return LKV_ERR_NULL;
    if ((host_transitions == nullptr) != (dev_transitions == nullptr)) return LKV_ERR_NULL;   // both pools or neither
    if (!aligned16(dev_states) || !aligned16(dev_transitions)) return LKV_ERR_ALIGN;
    // slots in order of first appearance; everything is checked before the first copy is queued
    std::vector<int32_t> slot_of(d->n_chunks, -1), order;
    for (int i = 0; i < n_ids; ++i) {
        const int32_t c = chunk_ids[i];
        if (c < 0 || c >= d->n_chunks) return LKV_ERR_INDEX;
        if (slot_of[c] < 0) {
            slot_of[c] = static_cast<int32_t>(order.size());
            order.push_back(c);
        }
    }
    if (static_cast<long long>(order.size()) > capacity) return LKV_ERR_WORKSPACE;
    const size_t es = d->state_dtype == LKV_DTYPE_BF16 ? 2 : 4;
    const size_t state_b = es * static_cast<size_t>(d->H) * d->d_k * d->d_v;
    const size_t trans_b = sizeof(float) * static_cast<size_t>(d->H) * (d->family == LKV_FAMILY_GDN ? static_cast<size_t>(d->d_k) * d->d_k : 1);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (size_t k = 0; k < order.size(); ++k) {
        const size_t c = static_cast<size_t>(order[k]);
        if (cudaMemcpyAsync(static_cast<char *>(dev_states) + k * state_b, static_cast<const char *>(host_states) + c * state_b,
                            state_b, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            (host_transitions &&
             cudaMemcpyAsync(static_cast<char *>(dev_transitions) + k * trans_b, static_cast<const char *>(host_transitions) + c * trans_b,
                             trans_b, cudaMemcpyHostToDevice, s) != cudaSuccess)) {
            cudaGetLastError();
            return LKV_ERR_CUDA;
        }
    }
    for (int i = 0; i < n_ids; ++i) staged_ids[i] = slot_of[chunk_ids[i]];
    *n_staged = static_cast<int32_t>(order.size());
    return LKV_OK;
}

int lkv_gdn_chunk_artifacts(const void *k, const void *v, const float *g, const float *beta, float *states,
                            float *transitions, const lkv_gdn_desc *d, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (d->state_dtype != LKV_DTYPE_F32) return LKV_ERR_MODE;
    if (d->n_seq > 0 && (!states || !transitions)) return LKV_ERR_NULL;
    if (d->n_seq < 0 || d->n_seq > (1 << 29)) return LKV_ERR_DIM;
    if (!aligned16(transitions)) return LKV_ERR_ALIGN;
    {
        const size_t st_b = sizeof(float) * static_cast<size_t>(d->n_seq > 0 ? d->n_seq : 0) * d->H_v * d->d_k * d->d_v;
        if (overlaps(states, st_b, transitions, st_b)) return LKV_ERR_OVERLAP;
    }
    lkv_gdn_desc d2 = *d;
    d2.n_seq = 2 * d->n_seq;   // every chunk twice: once as a scan from the empty state, once as a transition sequence
    // q is not needed for the states: the key tensor stands in for it (its read-outs are not written)
    return gdn_impl(k, k, v, g, beta, nullptr, nullptr, states, &d2, stream, 4, nullptr, transitions);
}

int lkv_mamba_chunk_logdecay(const float *dt, const float *A, float *logdecay, const lkv_ssd_desc *d, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (d->H < 1) return LKV_ERR_DIM;
    std::vector<int32_t> cu;
    int st = check_seqs(d->T_total, d->n_seq, d->cu_seqlens, cu);
    if (st != LKV_OK) return st;
    if (d->n_seq == 0) return LKV_OK;
    if (!A || !logdecay || (d->T_total > 0 && !dt)) return LKV_ERR_NULL;
    if (!aligned16(dt) || !aligned16(A) || !aligned16(logdecay)) return LKV_ERR_ALIGN;
    if (!d->workspace || d->workspace_bytes < ws_bytes_for(d->n_seq + 1, kScanIdxCap)) return LKV_ERR_WORKSPACE;
    if (!aligned16(d->workspace)) return LKV_ERR_ALIGN;
    SsdArgs a{};
    a.dt = dt; a.A = A; a.n_seq = d->n_seq; a.T_total = d->T_total; a.H = d->H; a.P = d->P; a.N = d->N; a.G = d->G;
    a.status = static_cast<int32_t *>(d->workspace);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = place_indices(a.cu, cu, d->workspace, s);
    if (st != LKV_OK) return st;
    return launch_mamba_logdecay(a, logdecay, s) == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

size_t lkv_state_rel_error_workspace_bytes(int n_states, size_t state_elems) {
    if (n_states < 0 || state_elems == 0) return 0;
    return align_up(sizeof(float) * 2 * static_cast<size_t>(n_states) * state_err_parts(state_elems) + 16, 256);
}

int lkv_state_rel_error(const float *S_init, const float *S_ref, float *rel_err, int n_states, size_t state_elems,
                        void *workspace, size_t workspace_bytes, void *stream) {
    if (n_states < 0 || state_elems == 0 || state_elems % 4 != 0 || n_states > 65535) return LKV_ERR_DIM;
    if (n_states == 0) return LKV_OK;
    if (!S_init || !S_ref || !rel_err) return LKV_ERR_NULL;
    if (!aligned16(S_init) || !aligned16(S_ref) || !aligned16(workspace)) return LKV_ERR_ALIGN;
    if (!workspace || workspace_bytes < lkv_state_rel_error_workspace_bytes(n_states, state_elems)) return LKV_ERR_WORKSPACE;
    const cudaError_t e = launch_state_rel_error(S_init, S_ref, rel_err, n_states, state_elems,
                                                 static_cast<float *>(workspace), static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

int lkv_ssd_fwd(const void *x, const float *dt, const float *A, const void *B, const void *C,
                const float *S0, void *y, void *S_T, const lkv_ssd_desc *d, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (!dtype_ok(d->io_dtype) || !compute_ok(d->compute) || !dtype_ok(d->state_dtype)) return LKV_ERR_MODE;
    const bool st_bf16 = d->state_dtype == LKV_DTYPE_BF16;
    if (st_bf16 && S_T && S_T == S0) return LKV_ERR_OVERLAP;   // an fp32 input cannot be a bf16 output
    if (d->H < 1 || d->P < 1 || d->N < 1 || d->G < 1 || d->H % d->G != 0) return LKV_ERR_DIM;
    std::vector<int32_t> cu;
    int st = check_seqs(d->T_total, d->n_seq, d->cu_seqlens, cu);
    if (st != LKV_OK) return st;
    if (d->n_seq == 0) return LKV_OK;
    if (!A) return LKV_ERR_NULL;
    if (d->T_total > 0 && (!x || !dt || !B || !C)) return LKV_ERR_NULL;
    if (!y && !S_T) return LKV_ERR_NULL;   // nothing to compute
    if (!aligned16(x) || !aligned16(dt) || !aligned16(A) || !aligned16(B) || !aligned16(C) || !aligned16(S0) ||
        !aligned16(y) || !aligned16(S_T))
        return LKV_ERR_ALIGN;
    if (!d->workspace || d->workspace_bytes < ws_bytes_for(2 * d->n_seq + 1, kScanIdxCap)) return LKV_ERR_WORKSPACE;
    if (!aligned16(d->workspace)) return LKV_ERR_ALIGN;
    {
        // outputs may not overlap inputs (S_T == S0 exactly is the one allowed alias) nor each other
        const size_t es = d->io_dtype == LKV_DTYPE_BF16 ? 2 : 4, T = static_cast<size_t>(d->T_total);
        const size_t x_b = es * T * d->H * d->P, bc_b = es * T * d->G * d->N, dt_b = sizeof(float) * T * d->H;
        const size_t st_in = sizeof(float) * static_cast<size_t>(d->n_seq) * d->H * d->N * d->P;
        const size_t st_b = st_bf16 ? st_in / 2 : st_in;
        const void *in[6] = {x, dt, A, B, C, S0};
        const size_t in_b[6] = {x_b, dt_b, sizeof(float) * d->H, bc_b, bc_b, S0 ? st_in : 0};
        for (int i = 0; i < 6; ++i) {
            if (overlaps(y, y ? x_b : 0, in[i], in_b[i])) return LKV_ERR_OVERLAP;
            if (!(i == 5 && S_T == S0) && overlaps(S_T, S_T ? st_b : 0, in[i], in_b[i])) return LKV_ERR_OVERLAP;
        }
        if (overlaps(y, y ? x_b : 0, S_T, S_T ? st_b : 0)) return LKV_ERR_OVERLAP;
    }

    SsdArgs a;
    a.x = x; a.dt = dt; a.A = A; a.B = B; a.C = C; a.S0 = S0; a.y = y; a.S_T = static_cast<float *>(S_T);
    a.st_bf16 = st_bf16 ? 1 : 0;
    a.n_seq = d->n_seq; a.T_total = d->T_total; a.H = d->H; a.P = d->P; a.N = d->N; a.G = d->G;
    a.status = static_cast<int32_t *>(d->workspace);
    const bool io_bf16 = d->io_dtype == LKV_DTYPE_BF16;
    const bool tensor_fits = ssd_scan_tensor_supported(a, io_bf16);
    const bool fp32_fits = ssd_scan_fp32_supported(d->N, d->P);
    bool use_tensor;
    if (d->compute == LKV_COMPUTE_TENSOR) {
        if (!tensor_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = true;
    } else if (d->compute == LKV_COMPUTE_FP32) {
        if (!fp32_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = false;
    } else {
        if (!tensor_fits && !fp32_fits) return LKV_ERR_UNSUPPORTED;
        use_tensor = tensor_fits;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    append_launch_order(cu, d->n_seq);
    st = place_indices(a.cu, cu, d->workspace, s);
    if (st != LKV_OK) return st;
    const cudaError_t e = use_tensor ? launch_ssd_scan_tensor(a, s) : launch_ssd_scan_fp32(a, io_bf16, s);
    return e == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

size_t lkv_workspace_bytes(int which, const void *desc, int n_units, int n_index) {
    if (!desc || n_units < 0 || n_index < 0) return 0;
    switch (which) {
        case LKV_WS_INIT: return ws_bytes_for(2 * n_units + 1 + n_index, kInitIdxCap);
        case LKV_WS_GDN:
        case LKV_WS_SSD: return ws_bytes_for(2 * n_units + 1, kScanIdxCap);
        default: return 0;
    }
}

int lkv_device_status(const void *workspace, void *stream) {
    if (!workspace) return LKV_ERR_NULL;
    int32_t word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return LKV_ERR_CUDA;
    }
    return word == 0 ? LKV_OK : LKV_ERR_DEVICE_TIMEOUT;
}

int lkv_selftest_bounded_wait(int poll_limit, void *workspace, void *stream) {
    if (!workspace) return LKV_ERR_NULL;
    if (poll_limit < 1 || poll_limit > (1 << 20)) return LKV_ERR_DIM;
    if (!aligned16(workspace)) return LKV_ERR_ALIGN;
    return launch_selftest_bounded_wait(static_cast<uint32_t>(poll_limit), static_cast<int32_t *>(workspace),
                                        static_cast<cudaStream_t>(stream)) == cudaSuccess ? LKV_OK : LKV_ERR_CUDA;
}

const char *lkv_status_string(int status) {
    switch (status) {
        case LKV_OK: return "ok";
        case LKV_ERR_NULL: return "a required pointer is NULL";
        case LKV_ERR_DIM: return "bad dimension";
        case LKV_ERR_MODE: return "unknown mode, family, dtype or compute value";
        case LKV_ERR_INDEX: return "index out of range or offsets not monotone";
        case LKV_ERR_ALIGN: return "pointer not 16-byte aligned";
        case LKV_ERR_UNSUPPORTED: return "no kernel for this shape or dtype";
        case LKV_ERR_WORKSPACE: return "workspace missing or too small";
        case LKV_ERR_CUDA: return "CUDA runtime call failed";
        case LKV_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case LKV_ERR_OVERLAP: return "an output buffer overlaps an input or another output";
        default: return "unknown status";
    }
}

int lkv_version(void) { return LKV_VERSION; }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Batched state initialisation for callers that cannot allocate device memory and therefore
// have no workspace to pass (an engine whose allocator is closed on the request path, a
// plugin running inside another component's memory budget).  The scratch is this fixed array,
// part of the library image on every GPU that loads it.
//
// In host code the name `g_static_scratch` is only a handle for the runtime, NOT a device
// address: the address a kernel may use has to be asked for with cudaGetSymbolAddress, once
// per device and with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[LKV_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void *g_static_scratch_addr[kMaxDevices];  // per device, filled on the first call there

// Device address of the static scratch on the current device (nullptr on failure).
void *static_scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return nullptr;
    }
    void *p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return nullptr;
        }
        __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);
    }
    return p;
}
}  // namespace

// Status word of the static scratch on the current device: read, and cleared if it was set (nobody else can).
extern "C" int lkv_device_status_static(void *stream) {
    void *scratch = static_scratch_for_current_device();
    if (!scratch) return LKV_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return LKV_ERR_CUDA;
    }
    if (word == 0) return LKV_OK;
    if (cudaMemsetAsync(scratch, 0, sizeof(word), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return LKV_ERR_CUDA;
    }
    return LKV_ERR_DEVICE_TIMEOUT;
}

extern "C" int lkv_init_state_batched_static(const void *states, const void *transitions, const int32_t *chunk_ids,
                                             const int32_t *cu_k, int n_req, int mode, const int32_t *sel_index,
                                             void *S0, const lkv_init_desc *d, void *stream) {
    if (!d) return LKV_ERR_NULL;
    if (n_req < 0) return LKV_ERR_DIM;
    if (!cu_k) return LKV_ERR_NULL;
    // size check first: beyond the fixed array there is nowhere to put the index list
    const long long n_ints = 2LL * n_req + 1 + (cu_k[n_req] > 0 ? cu_k[n_req] : 0);
    if (n_ints > LKV_STATIC_MAX_INDEX) return LKV_ERR_WORKSPACE;
    void *scratch = static_scratch_for_current_device();
    if (!scratch) return LKV_ERR_CUDA;
    lkv_init_desc local = *d;
    local.workspace = scratch;
    local.workspace_bytes = LKV_STATIC_SCRATCH_BYTES;
    return init_impl(states, transitions, chunk_ids, cu_k, n_req, mode, sel_index, S0, &local, stream);
}
