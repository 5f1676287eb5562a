// placeholder: tensor-core kernels
#include "sc_internal.cuh"
namespace sc {
bool tc_shape_supported(int64_t, int64_t, int) { return false; }
size_t tc_tmaps_bytes(int) { return 0; }
sc_status tc_init() { return SC_OK; }
sc_status tc_encode_class(sc_plan*, ShapeClass&, bool, bool) { return SC_OK; }
sc_status tc_launch_project(sc_plan*, ShapeClass&, const int*, int) { return SC_ERR_INVALID_ARG; }
sc_status tc_launch_epilogue(sc_plan*, ShapeClass&, const int*, int, const StepScalars&) { return SC_ERR_INVALID_ARG; }
}
