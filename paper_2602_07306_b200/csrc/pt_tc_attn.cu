// Attention kernels of the bf16 path (first version routes through the plain per-row kernel).
#include "pt_tc.h"
namespace pt {
pt_status launch_flash_prefill(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    launch_simt_attn_bf16(k, q, k.m->QD, pool_l, o);
    return PT_OK;
}
pt_status launch_decode_attn(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    launch_simt_attn_bf16(k, q, k.m->QD, pool_l, o);
    return PT_OK;
}
}
