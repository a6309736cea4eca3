#include "common.cuh"
size_t rs_probe_workspace_bytes(const rs_problem*) { return 0; }
size_t rs_indices_workspace_bytes(const rs_problem*, const rs_candidate*, int) { return 0; }
extern "C" int rs_probe(const rs_problem*, const void*, const void*, const void*, float*, float*, float*, float*, float*, float*, float*, void*, size_t, int32_t*, void*) { return RS_ERR_INVALID_ARG; }
extern "C" int rs_build_indices(const rs_problem*, const rs_candidate*, int, const float*, const float*, const float*, const float*, const float*, const int32_t*, const rs_index_set*, rs_cand_stats*, void*, size_t, int32_t*, void*) { return RS_ERR_INVALID_ARG; }
extern "C" int rs_route(const rs_problem*, const rs_candidate*, int, const rs_cand_stats*, const int64_t*, const float*, const rs_route_params*, int32_t*, rs_route_report*, int32_t*, void*) { return RS_ERR_INVALID_ARG; }
extern "C" int rs_certificate(int, int, const float*, const float*, const int32_t*, int, const float*, const float*, float, float*, float*, float*, float*, float*, int32_t*, void*) { return RS_ERR_INVALID_ARG; }
