// Host-visible interface of the tensor-core tree attention (attention_tc.cu).
#pragma once

#include "common.cuh"

namespace llmcad {

size_t attention_tc_workspace_bytes(int n_heads, int n_sms);

// Hand-over counters of an attention launch inside a pass (common.cuh, "completion counters"): the kernel waits
// until *dep_ctr has reached dep_target instead of for its grid dependency, and every CTA adds one to *done_ctr
// when its rows of the output are written; the launcher reports how many arrivals that makes.
struct AttnSync {
    const uint32_t *dep_ctr;
    uint32_t dep_target;
    uint32_t *done_ctr;
    uint64_t wait_limit_ns;
    mutable uint32_t arrivals;
};

// q, o: [n][H][128] bf16; k, v: [H][kv_stride][128] bf16; anc: [n][4] ancestor-or-self bit rows.
// comp != 0: q and o each consist of a hi and a lo plane, the lo plane kLoRows rows ([H][128] each)
// after the hi plane, and kv_lo holds the bf16 remainders of the tree nodes' keys and values,
// [2][H][kLoRows][128] (K then V, row = query index).
// n_tree > 0: the queries are only the tree nodes q_first .. q_first + n - 1 (anc holds the rows of
// all n_tree nodes), the keys the prefix and all n_tree tree nodes; 0 means n_tree = n, q_first = 0.
cudaError_t launch_attention_tc(const void *q, const void *k, const void *v, int n_heads, int hd, int kv_stride, int P,
                                int n, const uint32_t *anc, void *o, float *ws, uint32_t *counters, int n_sms,
                                int32_t *status, cudaStream_t st, int *launched, unsigned long long *trace = nullptr, int comp = 0,
                                const void *kv_lo = nullptr, int n_tree = 0, int q_first = 0, const AttnSync *sync = nullptr);

// The same operation on the tcgen05 tensor cores (attention_t5.cu), for larger trees; arguments as above.
cudaError_t launch_attention_t5(const void *q, const void *k, const void *v, int n_heads, int hd, int kv_stride, int P,
                                int n, const uint32_t *anc, void *o, int n_sms, int32_t *status, cudaStream_t st,
                                int *launched, unsigned long long *trace = nullptr, int comp = 0, const void *kv_lo = nullptr,
                                int n_tree = 0, int q_first = 0, uint64_t wait_limit_ns = kDefaultWaitLimitNs,
                                const AttnSync *sync = nullptr);

// Which of the two serves a tree of n query rows by default: the tcgen05 kernel above 32 rows (measured on
// B200 in whole passes of the 7B shape: 1-3 % of the pass faster at 33-64 nodes, 4-8 % at 96-128; at 32 nodes
// and below, where only one of its four softmax warps has rows to work on, 1-2 % slower).
// LLMCAD_ATTN_T5_MIN_N moves the switch (tuning aid, read once; 0 = never).
bool attention_prefers_t5(int n);

}  // namespace llmcad
