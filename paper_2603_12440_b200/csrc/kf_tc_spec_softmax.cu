// tcgen05 linear kernel with the row-norm fixed at compile time (softmax) and one instantiation per
// activation: see kf_tc_kernel.cuh.  Split over translation units so that they build in parallel.
#include "kf_tc_kernel.cuh"

namespace kf {

kf_status tc_launch_spec_softmax(int act, const TcLaunchArgs& a) {
    return tc_launch_norm<KF_NORM_SOFTMAX>(act, a.grid, a.st, *a.tmX, *a.tmW, *a.tmY, *static_cast<const TcParams*>(a.params));
}

}  // namespace kf
