// Status bits that kernels OR into the context's device status word; the host reads them in
// lpc_sync_status().
#pragma once
namespace lpc {
constexpr unsigned int DEV_NONFINITE = 1u;  // a NaN or Inf reached the quantizer
constexpr unsigned int DEV_TIMEOUT = 2u;    // a bounded wait on an mbarrier ran out
}  // namespace lpc
