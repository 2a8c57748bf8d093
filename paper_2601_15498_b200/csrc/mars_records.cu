// libmars: verification from per-row top-2 records (vocabulary-parallel logits).
//
// When the LM head is sharded over the vocabulary (tensor parallelism), every GPU holds only a
// column range of each logits row.  mars_top2_shard (mars_verify.cu) reduces a shard to one
// 16-byte record per row with global token ids; the ranks exchange those records (one
// all-gather of 16 B x rows per rank, received into local memory), and this kernel merges the
// G records of every row -- the merge operator is associative and commutative under the total
// order, so the result is bit-identical to a single-GPU scan -- and runs the same verification
// tail as the other entry points.
#include "mars_common.cuh"

#include "mars.h"

namespace mars {

__global__ void __launch_bounds__(128) records_tail_kernel(const Rec *records, long long rows, int G,
                                                           const TailArgs t)
{
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    const int b = blockIdx.x;
    const Rec *base = records + (size_t)b * t.N;
    verify_tail(t, b, smem_dyn, [&](int i) {
        Rec acc = empty_rec();
        for (int g = 0; g < G; ++g) acc = merge(acc, base[(size_t)g * rows + i]);
        return finish_record(acc);
    });
}

}  // namespace mars

extern "C" mars_status_t mars_verify_records(const void *records, int G, const int32_t *tok,
                                             const int32_t *parent, int B, int N, float theta,
                                             uint32_t flags, int32_t *accept_len, int32_t *out_tokens,
                                             int32_t *path_nodes, int32_t *out_len, int Dcap,
                                             int32_t *seq_status, const mars_debug_out_t *dbg,
                                             void *cuda_stream)
{
    using namespace mars;
    if (!records || ((uintptr_t)records & 15) || !tok || !parent || !accept_len || !out_tokens || !out_len)
        return MARS_ERR_INVALID_ARG;
    if (G < 1 || B < 1 || N < 1 || Dcap < 0 || theta != theta) return MARS_ERR_INVALID_ARG;
    if (flags & ~(MARS_SIGN_LITERAL | MARS_SHARED_PARENT | MARS_RULE_MARGIN | MARS_RULE_PROB_RATIO))
        return MARS_ERR_UNSUPPORTED;
    if ((flags & MARS_RULE_MARGIN) && (flags & MARS_RULE_PROB_RATIO)) return MARS_ERR_INVALID_ARG;
    rule_threshold(&theta, &flags);
    if (N > MARS_MAX_NODES || G > 4096) return MARS_ERR_UNSUPPORTED;
    TailArgs t;
    t.tok = tok; t.parent = parent; t.accept_len = accept_len; t.out_tokens = out_tokens;
    t.path_nodes = path_nodes; t.out_len = out_len; t.seq_status = seq_status;
    t.dbg_val = dbg ? dbg->top2_val : nullptr;
    t.dbg_id = dbg ? dbg->top2_id : nullptr;
    t.dbg_flags = dbg ? dbg->node_flags : nullptr;
    t.N = N; t.Dcap = Dcap; t.theta = theta; t.flags = flags; t.chain = 0;
    records_tail_kernel<<<B, 128, tail_smem_bytes(N), (cudaStream_t)cuda_stream>>>(
        (const Rec *)records, (long long)B * N, G, t);
    return cudaGetLastError() == cudaSuccess ? MARS_OK : MARS_ERR_CUDA;
}
