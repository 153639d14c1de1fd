// placeholder until the tensor-core kernel lands: route to the scalar kernel
#include "common.cuh"
namespace hpd {
int launch_attn_tc(const AttnArgs& a)
{
    SimtArgs s{};
    s.g = a.g; s.max_rows = a.max_rows; s.n_splits = 1; s.n_active = a.n_active; s.q = a.q;
    s.k1 = a.prefix_k; s.v1 = a.prefix_v; s.doc_id = a.doc_id; s.doc_kv_start = a.doc_kv_start;
    s.doc_prefix_len = a.doc_prefix_len; s.k2 = a.suffix_k; s.v2 = a.suffix_v; s.suffix_off = a.suffix_off;
    s.suffix_len = a.suffix_len; s.suffix_extra = a.suffix_extra; s.o = a.o; s.lse = a.lse; s.stream = a.stream;
    return launch_attn_simt(s);
}
}
