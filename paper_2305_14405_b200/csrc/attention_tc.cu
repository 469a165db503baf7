// placeholder until the tensor-core attention kernel lands
#include "nm_common.cuh"
bool nm_attention_tc_supported(const nm_attn_desc*) { return false; }
nm_status nm_launch_attention_tc(nm_ctx*, const nm_attn_desc*, cudaStream_t) { return NM_ERR_UNSUPPORTED; }
