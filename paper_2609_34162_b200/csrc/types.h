// Plain types shared by the host code and the kernels of libslidedp.
#pragma once

#include <stdint.h>

namespace slidedp {

constexpr int kMaxRanks = 16;

struct GradPtrs {
  const uint16_t* p[kMaxRanks];
};

// Everything the update needs that does not depend on the element, prepared on the host
// in double from the double-typed hyper-parameters.
struct UpdateConsts {
  double beta1, beta2;
  double omb1, omb2;        // 1 - beta1, 1 - beta2 (exact in double for beta in [0.5, 1))
  double rsqrt_bc2;         // 1 / sqrt(1 - beta2^t)
  double eps;
  double neg_lr_over_bc1;   // -lr / (1 - beta1^t)
  double decay;             // 1 - lr * weight_decay
  float inv_R;              // (float)inv_R
};

}  // namespace slidedp
