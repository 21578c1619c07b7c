// Tensor-core (tcgen05 / TMEM / TMA) attention over the paged store.  Placeholder host object
// until the kernel lands: reports "not enabled" so that the SIMT kernel serves every dtype.
#pragma once
#include <string>

#include "common.cuh"

namespace scalekv {

struct AttendTc {
  bool init(int, int, void *, void *, long long, int, std::string &) { return true; }
  bool enabled() const { return false; }
  bool launch(const LayerView &, const TensorView &, const TensorView &, float *, int, int, float, cudaStream_t, std::string &) {
    return false;
  }
};

}  // namespace scalekv
