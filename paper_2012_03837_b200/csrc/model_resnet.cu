// ResNet family (App. B.3): not built yet in this file; lp_create reports LP_ERR_UNSUPPORTED.
#include <stdexcept>

#include "runtime.h"

namespace lp {
void build_resnet(Handle&) { throw std::runtime_error("unsupported: the RESNET family is not implemented yet"); }
}  // namespace lp
