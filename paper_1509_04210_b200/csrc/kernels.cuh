// Launch interface between the host side of the parameter server and its sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace rudra {

constexpr int kMaxGroup = 128;   // RUDRA_MAX_GROUP
constexpr int kMaxDsts = 128;    // RUDRA_MAX_DSTS

enum GradType : int { kF32 = 0, kBF16 = 1 };
enum Optim : int { kMomentumSgd = 0, kAdagrad = 1 };

// Everything one fused sumGradients + applyUpdate launch needs.  Passed by value as a
// __grid_constant__ kernel parameter: the per-gradient pointers and step sizes form a small
// table in the constant bank, read with uniform addresses, so an update costs one launch and no
// other stream operation.
struct UpdateParams {
  const void* grad[kMaxGroup];   // c gradient vectors, arrival order
  float* dst[kMaxDsts];          // ndst learner buffers that receive the new weights
  float scale[kMaxGroup];        // s_l (momentum SGD) or s_l / sum(s) (AdaGrad)
  float* theta;
  float* state;                  // velocity (momentum SGD) or sum of squared gradients (AdaGrad)
  uint64_t n;                    // number of weights
  uint32_t c;
  uint32_t ndst;
  float momentum;
  float awd;                     // momentum SGD: sum(s) * weight_decay
  float abar;                    // AdaGrad: sum(s), the group's learning rate
  float wd;                      // AdaGrad: weight decay
  float eps;                     // AdaGrad: denominator floor
  uint32_t reverse;              // sweep the vector from the end (alternates launch to launch)
};

struct SnapshotParams {
  float* dst[kMaxDsts];
  const float* src;
  uint64_t n;
  uint32_t ndst;
  uint32_t reverse;
};

// Enqueue one fused update (and ndst snapshot writes) on stream.  Returns the CUDA status of the launch.
cudaError_t launch_update(const UpdateParams& p, GradType gtype, Optim optim, cudaStream_t stream);

// Enqueue one 1 -> ndst copy of the weights.
cudaError_t launch_snapshot(const SnapshotParams& p, cudaStream_t stream);

}  // namespace rudra
