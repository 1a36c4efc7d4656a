#include "common.cuh"
bool fax_gemm_tc_supported(const FaxGemm&) { return false; }
fax_status fax_gemm_tc(fax_ctx*, const FaxGemm&) { return FAX_ERR_UNSUPPORTED_SHAPE; }
