// libmars: streaming top-2 over logits rows fused with the MARS verification tail.
//
// One kernel per call.  A thread block owns one slice of one logits row (a whole row when
// the batch has enough rows to fill the GPU, 1/S of a row otherwise) and streams it once
// from HBM with 16-byte loads.  Each thread keeps an exact top-2 (values and token ids) in
// registers, but touches it only for the few batches that can still change the answer:
//
//   - a batch of U (8, or 4 in the high-occupancy variant) 16-byte vectors per thread is first reduced to its maximum with packed
//     bf16x2 (or fp32) max instructions -- about one instruction per two bf16 elements;
//   - the batch is skipped unless its maximum beats the thread's own runner-up AND is not
//     below T2, a lower bound on the slice's runner-up value that the whole block shares
//     through shared memory (order-preserving integer encoding, atomicMax);
//   - the bound is bootstrapped from the first batch: each warp publishes the top-2 of its
//     lanes' batch maxima, so that no thread pays the exact path for its whole first batch;
//     the first batch's loads are issued before the block's set-up barrier.
//
// Why skipping is exact: threads visit their elements in increasing token id, so an element
// equal to the thread's runner-up loses the id tie-break; and an element below a value that
// two other elements of the slice reach cannot be in the slice's top-2.
//
// Finished slices meet in global memory: the block writes its 16-byte record, bumps the
// sequence's arrival counter, and the block that arrives last (nobody waits, nobody spins)
// merges the records of the sequence and runs the verification tail of mars_common.cuh.
#include "mars_top2_stream.cuh"

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "mars.h"

namespace mars {

struct Params {
    const void *logits;
    long long ld;
    int V;
    int N;
    int S;   // slices per row
    int L;   // elements per slice (multiple of 16)
    Rec *partial;        // [R*S]
    unsigned *counters;  // [B]
    Rec *shard_out;      // non-null: emit merged per-row records [B*N] instead of verifying
    int id_offset;       // ... with this offset added to the token ids (vocabulary shard)
    int early;           // MARS_LOGITS_READY: stream the logits before waiting for the predecessor
    int stage_partials;  // last block copies the sequence's N*S records to shared memory first
    int tail_smem_off;   // byte offset of that staging area in dynamic shared memory
    TailArgs tail;
};

template <int DT, int U, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) verify_kernel(const Params p)
{
    typedef Elem<DT> E;
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    __shared__ unsigned sT[2];
    __shared__ Rec s_warp[kThreads / 32];
    __shared__ int s_last;

    // The next call on this stream may be scheduled while this one drains.  This call itself
    // waits for its predecessor right here unless the caller vouched that the logits do not come
    // from it (MARS_LOGITS_READY); then the wait moves to the point where the workspace is first
    // touched.
    pdl_launch_dependents();
    if (!p.early) pdl_wait();
    const int tid = threadIdx.x;
    const long long blk = blockIdx.x;
    const long long row = blk / p.S;
    const int slice = (int)(blk - row * p.S);
    const int b = (int)(row / p.N);

    const int lo = slice * p.L;
    const int hi = min(p.V, lo + p.L);
    const char *rowp = (const char *)p.logits + (size_t)row * (size_t)p.ld * E::kBytes;

    // [lo, hi) = head scalars | 16-byte vectors | tail scalars
    const uintptr_t a0 = (uintptr_t)(rowp + (size_t)lo * E::kBytes);
    int nhead = (int)(((16 - (a0 & 15)) & 15) / E::kBytes);
    nhead = min(nhead, max(hi - lo, 0));
    const int vlo = lo + nhead;
    const int nvec = max(hi - vlo, 0) / E::kVec;
    const int tlo = vlo + nvec * E::kVec;
    const int ntail = max(hi - tlo, 0);
    const uint4 *vbase = (const uint4 *)(rowp + (size_t)vlo * E::kBytes);

    constexpr int kBatchVecs = kThreads * U;
    const int nfull = nvec / kBatchVecs;
    uint4 v[U];
    typename E::packed_t q[U];

    // ---- batch 0: issue its loads first, so that the set-up below overlaps their latency ----
    float bm = (nfull > 0) ? load_batch<DT, U, false>(vbase, tid, nvec, v, q)
                           : load_batch<DT, U, true>(vbase, tid, nvec, v, q);
    if (tid == 0) { sT[0] = enc(-INFINITY); sT[1] = enc(-INFINITY); }
    __syncthreads();

    Rec s = empty_rec();
    if (tid < nhead) insert<false>(s, E::scalar(rowp, lo + tid), lo + tid, sT);

    // Bootstrap the shared bound from the batch maxima: every warp publishes the top-2 of its
    // lanes' maxima (distinct elements) and goes on without waiting for the other warps; it
    // sees at least its own contribution.
    {
        float a1 = (bm == bm) ? bm : -INFINITY, a2 = -INFINITY;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            float b1 = __shfl_xor_sync(0xffffffffu, a1, m), b2 = __shfl_xor_sync(0xffffffffu, a2, m);
            a2 = fmaxf(fminf(a1, b1), fmaxf(a2, b2));
            a1 = fmaxf(a1, b1);
        }
        if ((tid & 31) == 0) { publish(sT, a1); publish(sT, a2); }
        __syncwarp();
    }
    float T2 = dec(*(volatile unsigned *)&sT[1]);
    process_batch<DT, U, false>(v, q, bm, T2, vlo + tid * E::kVec, s, sT);

    // ---- steady state ----
    for (int bi = 1; bi < nfull; ++bi) {
        bm = load_batch<DT, U, false>(vbase, bi * kBatchVecs + tid, nvec, v, q);
        T2 = dec(*(volatile unsigned *)&sT[1]);
        process_batch<DT, U, true>(v, q, bm, T2, vlo + (bi * kBatchVecs + tid) * E::kVec, s, sT);
    }
    if (nfull > 0 && nfull * kBatchVecs < nvec) {
        bm = load_batch<DT, U, true>(vbase, nfull * kBatchVecs + tid, nvec, v, q);
        T2 = dec(*(volatile unsigned *)&sT[1]);
        process_batch<DT, U, true>(v, q, bm, T2, vlo + (nfull * kBatchVecs + tid) * E::kVec, s, sT);
    }
    if (tid < ntail) insert<false>(s, E::scalar(rowp, tlo + tid), tlo + tid, sT);

    // ---- block merge under the full total order ----
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) s = merge(s, shfl_xor_rec(s, m));
    if ((tid & 31) == 0) s_warp[tid >> 5] = s;
    // Everything up to here only read this call's logits.  Workspace and outputs may still be in
    // use by the previous call on the stream: wait for it to finish before touching them.
    pdl_wait();
    __syncthreads();
    if (tid == 0) {
        Rec r = s_warp[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) r = merge(r, s_warp[w]);
        p.partial[blk] = r;
        __threadfence();
        unsigned ticket = atomicAdd(&p.counters[b], 1u);
        s_last = (ticket == (unsigned)(p.N * p.S - 1)) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;

    // ---- last block of the sequence: merge slices, verify, emit ----
    __threadfence();
    const int S = p.S;
    const Rec *seq_partial = p.partial + (size_t)b * p.N * S;
    unsigned char *tail_smem = smem_dyn;
    const Rec *src = seq_partial;
    if (p.stage_partials) {
        // Bring all N*S records in with independent coalesced loads (one memory latency
        // instead of S dependent ones per row), then merge out of shared memory.
        Rec *s_part = reinterpret_cast<Rec *>(smem_dyn + p.tail_smem_off);
        for (int f = tid; f < p.N * S; f += kThreads) {
            int4 w = __ldcg(reinterpret_cast<const int4 *>(seq_partial + f));
            *reinterpret_cast<int4 *>(s_part + f) = w;
        }
        __syncthreads();
        src = s_part;
    }
    const bool staged = p.stage_partials != 0;
    auto merged_row = [&](int i) {
        Rec acc = empty_rec();
        for (int k = 0; k < S; ++k) {
            const int4 *q = reinterpret_cast<const int4 *>(src + (size_t)i * S + k);
            int4 w = staged ? *q : __ldcg(q);
            Rec r;
            r.z1 = __int_as_float(w.x); r.id1 = w.y; r.z2 = __int_as_float(w.z); r.id2 = w.w;
            acc = merge(acc, r);
        }
        return acc;
    };
    if (p.shard_out) {
        // vocabulary shard: hand the rows' records (global token ids, still unfinished) on
        for (int i = tid; i < p.N; i += kThreads) {
            Rec r = merged_row(i);
            if (r.id1 != kNoId) r.id1 += p.id_offset;
            if (r.id2 != kNoId) r.id2 += p.id_offset;
            p.shard_out[(size_t)b * p.N + i] = r;
        }
    } else {
        verify_tail(p.tail, b, tail_smem, [&](int i) { return finish_record(merged_row(i)); });
    }
    if (tid == 0) p.counters[b] = 0;
}

// ------------------------------------------------------------------------- host side

static size_t counters_bytes(int B) { return ((size_t)B * sizeof(unsigned) + 255) / 256 * 256; }

static bool sizes_supported(int B, int N, int V, int dt)
{
    if (B < 1 || N < 1 || V < 2) return false;
    if (dt != MARS_BF16 && dt != MARS_FP32) return false;
    if (N > MARS_MAX_NODES) return false;
    if (V > (1 << 30)) return false;
    if ((long long)B * N > (1ll << 40)) return false;
    return true;
}

static mars_status_t run(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *tok,
                         const int32_t *parent, int chain, int B, int N, int V, float theta,
                         uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                         int32_t *path_nodes, int32_t *out_len, int Dcap, int32_t *seq_status,
                         const mars_debug_out_t *dbg, void *workspace, size_t workspace_bytes,
                         void *cuda_stream, Rec *shard_out = nullptr, int id_offset = 0)
{
    if (B < 1 || N < 1 || V < 2 || !logits) return MARS_ERR_INVALID_ARG;
    if (ld < V || Dcap < 0 || theta != theta) return MARS_ERR_INVALID_ARG;
    if (!shard_out) {
        if (!accept_len || !out_tokens || !out_len) return MARS_ERR_INVALID_ARG;
        if (!chain && (!tok || !parent)) return MARS_ERR_INVALID_ARG;
        if (chain && N > 1 && !tok) return MARS_ERR_INVALID_ARG;
    }
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_COUNTERS_ZERO | MARS_RULE_MARGIN |
                  MARS_RULE_PROB_RATIO | MARS_LOGITS_READY))
        return MARS_ERR_UNSUPPORTED;
    if ((flags & MARS_RULE_MARGIN) && (flags & MARS_RULE_PROB_RATIO)) return MARS_ERR_INVALID_ARG;
    rule_threshold(&theta, &flags);
    if (!sizes_supported(B, N, V, (int)dt)) return MARS_ERR_UNSUPPORTED;
    const int es = dt == MARS_BF16 ? 2 : 4;
    if ((uintptr_t)logits % es) return MARS_ERR_INVALID_ARG;
    const long long R = (long long)B * N;
    const Split sp = choose_split(R, V, (int)dt);
    if (R * sp.S > 0x7fffffffll) return MARS_ERR_UNSUPPORTED;
    const size_t need = counters_bytes(B) + (size_t)R * sp.S * sizeof(Rec);
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return MARS_ERR_WORKSPACE;

    Params p;
    p.logits = logits; p.ld = ld; p.V = V; p.N = N; p.S = sp.S; p.L = sp.L;
    p.counters = (unsigned *)workspace;
    p.partial = (Rec *)((char *)workspace + counters_bytes(B));
    p.shard_out = shard_out; p.id_offset = id_offset;
    p.early = (flags & MARS_LOGITS_READY) ? 1 : 0;
    p.tail.tok = tok; p.tail.parent = parent;
    p.tail.accept_len = accept_len; p.tail.out_tokens = out_tokens; p.tail.path_nodes = path_nodes;
    p.tail.out_len = out_len; p.tail.seq_status = seq_status;
    p.tail.dbg_val = dbg ? dbg->top2_val : nullptr;
    p.tail.dbg_id = dbg ? dbg->top2_id : nullptr;
    p.tail.dbg_flags = dbg ? dbg->node_flags : nullptr;
    p.tail.N = N; p.tail.Dcap = Dcap; p.tail.theta = theta; p.tail.flags = flags; p.tail.chain = chain;

    cudaStream_t st = (cudaStream_t)cuda_stream;
    // Arrival counters start at zero.  Every sequence's last block puts its counter back to
    // zero, so a caller that knows the counters are clean may skip the memset node.
    if (!(flags & MARS_COUNTERS_ZERO) &&
        cudaMemsetAsync(p.counters, 0, (size_t)B * sizeof(unsigned), st) != cudaSuccess)
        return MARS_ERR_CUDA;
    const unsigned grid = (unsigned)(R * sp.S);
    // dynamic shared memory: the tail's arrays, then (if it fits in 48 KB) room for N*S records
    const size_t tail_bytes = (tail_smem_bytes(N) + 15) / 16 * 16;
    const size_t stage_bytes = (size_t)N * sp.S * sizeof(Rec);
    p.stage_partials = (sp.S > 1 && tail_bytes + stage_bytes <= 48 * 1024) ? 1 : 0;
    p.tail_smem_off = (int)tail_bytes;
    const size_t smem = tail_bytes + (p.stage_partials ? stage_bytes : 0);
    cudaError_t le;
    const bool overlap = hook(kHookNoOverlap) == 0;
    // The variant with 4 vectors per batch and 8 blocks per SM: large batches; also whenever a
    // batch just overflows one wave of the 4-blocks-per-SM variant (592 rows) but fits one of
    // this one, and for short rows (up to 128 KB: a block lives for a few batches only, and twice
    // the resident blocks hide twice the start-up and merge phases).
    const bool dense = dt == MARS_BF16 && sp.S == 1 &&
                       (R >= kDenseMinRows ||
                        (R > kTargetBlocks && ((long long)V * 2 <= 128 * 1024 || R <= kTargetBlocks * 3 / 2)));
    if (dense)
        le = launch_pdl(overlap, verify_kernel<MARS_BF16, kUDense, 8>, dim3(grid), dim3(kThreads), smem, st, p);
    else if (dt == MARS_BF16)
        le = launch_pdl(overlap, verify_kernel<MARS_BF16, kU, 4>, dim3(grid), dim3(kThreads), smem, st, p);
    else
        le = launch_pdl(overlap, verify_kernel<MARS_FP32, kU, 4>, dim3(grid), dim3(kThreads), smem, st, p);
    if (le != cudaSuccess) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    return MARS_OK;
}

}  // namespace mars

extern "C" {

size_t mars_workspace_bytes(int B, int N, int V, mars_dtype_t dt)
{
    if (!mars::sizes_supported(B, N, V, (int)dt)) return 0;
    const long long R = (long long)B * N;
    const mars::Split sp = mars::choose_split(R, V, (int)dt);
    return mars::counters_bytes(B) + (size_t)R * sp.S * sizeof(mars::Rec);
}

mars_status_t mars_verify_chain(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *draft,
                                int B, int K, int V, float theta, uint32_t flags, int32_t *accept_len,
                                int32_t *out_tokens, int32_t *out_len, int32_t *seq_status,
                                const mars_debug_out_t *dbg, void *workspace, size_t workspace_bytes,
                                void *cuda_stream)
{
    if (flags & MARS_SHARED_PARENT) return MARS_ERR_INVALID_ARG;
    return mars::run(logits, ld, dt, draft, nullptr, 1, B, K, V, theta, flags, accept_len, out_tokens,
                     nullptr, out_len, K - 1, seq_status, dbg, workspace, workspace_bytes, cuda_stream);
}

mars_status_t mars_verify_tree(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *tok,
                               const int32_t *parent, int B, int N, int V, float theta, uint32_t flags,
                               int32_t *accept_len, int32_t *out_tokens, int32_t *path_nodes,
                               int32_t *out_len, int Dcap, int32_t *seq_status,
                               const mars_debug_out_t *dbg, void *workspace, size_t workspace_bytes,
                               void *cuda_stream)
{
    return mars::run(logits, ld, dt, tok, parent, 0, B, N, V, theta, flags, accept_len, out_tokens,
                     path_nodes, out_len, Dcap, seq_status, dbg, workspace, workspace_bytes, cuda_stream);
}

// ---- host-buffer form: copies in, verification, copies out, all on the caller's stream --------

namespace mars {
struct HostStaging {       // byte offsets into the device staging buffer, each 256-byte aligned
    size_t logits, tok, parent, accept_len, out_tokens, path_nodes, out_len, seq_status, workspace, total;
    size_t logits_bytes, tok_bytes, parent_bytes, per_seq_bytes, path_bytes, workspace_bytes;
};

static bool host_staging_layout(int B, int N, int V, int dt, long long ld, int Dcap, bool shared_parent,
                                HostStaging *h)
{
    if (!sizes_supported(B, N, V, dt) || ld < V || Dcap < 0 || Dcap > MARS_MAX_NODES) return false;
    const size_t es = dt == MARS_BF16 ? 2 : 4;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    h->logits_bytes = (size_t)B * N * (size_t)ld * es;
    h->tok_bytes = (size_t)B * N * sizeof(int32_t);
    h->parent_bytes = shared_parent ? (size_t)N * sizeof(int32_t) : h->tok_bytes;
    h->per_seq_bytes = (size_t)B * sizeof(int32_t);
    h->path_bytes = (size_t)B * (Dcap + 1) * sizeof(int32_t);
    const Split sp = choose_split((long long)B * N, V, dt);
    h->workspace_bytes = counters_bytes(B) + (size_t)B * N * sp.S * sizeof(Rec);
    size_t o = 0;
    h->logits = o; o += up(h->logits_bytes);
    h->tok = o; o += up(h->tok_bytes);
    h->parent = o; o += up(h->tok_bytes);            // room for per-sequence parents either way
    h->accept_len = o; o += up(h->per_seq_bytes);
    h->out_tokens = o; o += up(h->path_bytes);
    h->path_nodes = o; o += up(h->path_bytes);
    h->out_len = o; o += up(h->per_seq_bytes);
    h->seq_status = o; o += up(h->per_seq_bytes);
    h->workspace = o; o += up(h->workspace_bytes);
    h->total = o;
    return true;
}
}  // namespace mars

size_t mars_verify_tree_host_staging_bytes(int B, int N, int V, mars_dtype_t dt, int64_t ld, int Dcap)
{
    mars::HostStaging h;
    return mars::host_staging_layout(B, N, V, (int)dt, ld, Dcap, false, &h) ? h.total : 0;
}

mars_status_t mars_verify_tree_host(const void *logits_host, int64_t ld, mars_dtype_t dt, const int32_t *tok_host,
                                    const int32_t *parent_host, int B, int N, int V, float theta, uint32_t flags,
                                    int32_t *accept_len_host, int32_t *out_tokens_host, int32_t *path_nodes_host,
                                    int32_t *out_len_host, int Dcap, int32_t *seq_status_host, void *staging,
                                    size_t staging_bytes, void *cuda_stream)
{
    if (!logits_host || !tok_host || !parent_host || !accept_len_host || !out_tokens_host || !out_len_host)
        return MARS_ERR_INVALID_ARG;
    if (B < 1 || N < 1 || V < 2 || ld < V || Dcap < 0 || theta != theta) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_RULE_MARGIN | MARS_RULE_PROB_RATIO))
        return MARS_ERR_UNSUPPORTED;
    mars::HostStaging h;
    if (!mars::host_staging_layout(B, N, V, (int)dt, ld, Dcap, (flags & MARS_SHARED_PARENT) != 0, &h))
        return MARS_ERR_UNSUPPORTED;
    if (!staging || ((uintptr_t)staging & 255) || staging_bytes < h.total) return MARS_ERR_WORKSPACE;
    char *d = (char *)staging;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(d + h.logits, logits_host, h.logits_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(d + h.tok, tok_host, h.tok_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(d + h.parent, parent_host, h.parent_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return MARS_ERR_CUDA;
    }
    // the staging buffer's workspace is not known to be clean: the counters are cleared on the stream
    const mars_status_t rs = mars::run(d + h.logits, ld, dt, (const int32_t *)(d + h.tok), (const int32_t *)(d + h.parent), 0,
                                       B, N, V, theta, flags, (int32_t *)(d + h.accept_len), (int32_t *)(d + h.out_tokens),
                                       (int32_t *)(d + h.path_nodes), (int32_t *)(d + h.out_len), Dcap,
                                       (int32_t *)(d + h.seq_status), nullptr, d + h.workspace, h.workspace_bytes, st);
    if (rs != MARS_OK) return rs;
    bool ok = cudaMemcpyAsync(accept_len_host, d + h.accept_len, h.per_seq_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out_tokens_host, d + h.out_tokens, h.path_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(out_len_host, d + h.out_len, h.per_seq_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (path_nodes_host)
        ok = ok && cudaMemcpyAsync(path_nodes_host, d + h.path_nodes, h.path_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (seq_status_host)
        ok = ok && cudaMemcpyAsync(seq_status_host, d + h.seq_status, h.per_seq_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return MARS_ERR_CUDA; }
    return MARS_OK;
}

// ---- verification without any caller-provided or allocated scratch -------------------------
//
// Scratch for mars_verify_tree_static lives in this fixed device array.  Every GPU that loads
// the library keeps these bytes until the process exits.  In host code the name
// `g_static_scratch` is only a handle for the runtime, not a device address: the address
// that kernels can use is obtained once per device with cudaGetSymbolAddress.
#define MARS_STATIC_SCRATCH_BYTES (1u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[MARS_STATIC_SCRATCH_BYTES];

namespace mars {
constexpr int kMaxDevices = 64;
static std::mutex g_static_mu;
static void *g_static_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on first use).
static mars_status_t static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MARS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MARS_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return MARS_OK;
}
}  // namespace mars

size_t mars_static_scratch_bytes(void) { return MARS_STATIC_SCRATCH_BYTES; }

mars_status_t mars_verify_tree_static(const void *logits, int64_t ld, mars_dtype_t dt, const int32_t *tok,
                                      const int32_t *parent, int B, int N, int V, float theta,
                                      uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                                      int32_t *path_nodes, int32_t *out_len, int Dcap,
                                      int32_t *seq_status, const mars_debug_out_t *dbg, void *cuda_stream)
{
    // sizes first: nothing is looked up or launched for a batch that cannot fit
    const size_t need = mars_workspace_bytes(B, N, V, dt);
    if (need == 0) return (B < 1 || N < 1 || V < 2) ? MARS_ERR_INVALID_ARG : MARS_ERR_UNSUPPORTED;
    if (need > MARS_STATIC_SCRATCH_BYTES) return MARS_ERR_STATIC_CAPACITY;
    void *scratch = nullptr;
    const mars_status_t st = mars::static_scratch(&scratch);
    if (st != MARS_OK) return st;
    // The arrival counters at the front of the scratch must start at zero; run() clears them
    // on the stream before the kernel.  Everything else in the array is overwritten before
    // it is read, so the previous call's leftovers are harmless.  MARS_COUNTERS_ZERO is a
    // promise about a workspace that the caller owns; nobody can make it about this array
    // (its counter region grows with B and may hold an earlier call's records), so the bit is
    // dropped and the counters are always cleared.
    flags &= ~MARS_COUNTERS_ZERO;
    return mars::run(logits, ld, dt, tok, parent, 0, B, N, V, theta, flags, accept_len, out_tokens,
                     path_nodes, out_len, Dcap, seq_status, dbg, scratch, MARS_STATIC_SCRATCH_BYTES,
                     cuda_stream);
}

mars_status_t mars_top2_shard(const void *logits, int64_t ld, mars_dtype_t dt, int B, int N, int V_local,
                              int32_t id_offset, void *records, uint32_t flags, void *workspace,
                              size_t workspace_bytes, void *cuda_stream)
{
    if (!records || ((uintptr_t)records & 15) || id_offset < 0) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_COUNTERS_ZERO | MARS_LOGITS_READY)) return MARS_ERR_UNSUPPORTED;
    return mars::run(logits, ld, dt, nullptr, nullptr, 0, B, N, V_local, 0.0f, flags, nullptr, nullptr,
                     nullptr, nullptr, 0, nullptr, nullptr, workspace, workspace_bytes, cuda_stream,
                     (mars::Rec *)records, id_offset);
}

const char *mars_status_string(mars_status_t s)
{
    switch (s) {
    case MARS_ERR_STATIC_CAPACITY: return "batch needs more scratch than the built-in static array holds";
    case MARS_OK: return "ok";
    case MARS_ERR_INVALID_ARG: return "invalid argument";
    case MARS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MARS_ERR_UNSUPPORTED: return "unsupported size, dtype or flag";
    case MARS_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
    }
}

}  // extern "C"
