// placeholder until the tensor-core path lands
#include "pt_internal.h"
namespace pt {
pt_status tc_build_weight_maps(pt_model*) { return PT_OK; }
pt_status tc_forward(Call&) { set_error("bf16 tensor-core path not built yet"); return PT_ERR_UNSUPPORTED; }
}
