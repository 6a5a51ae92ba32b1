// Workspace layout of elm_attend (byte offsets into the caller's workspace).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include "../../include/elm.h"

namespace elm {

struct AttendLayout {
    size_t Kc;    // [problems][n_core][d] gathered keys, input dtype
    size_t Vc;    // [problems][n_core][d] gathered values, input dtype
    size_t bias;  // [problems][n_core] log2 of the weights, fp32
    size_t total;
};
AttendLayout attend_layout(const elm_params *p, int32_t n_core);

}  // namespace elm
