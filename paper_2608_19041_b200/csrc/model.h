// Host-side model construction: blob parsing and the create-time precomputation that the
// paper's compressed inference performs once per model (radial table, pair cache, Gaunt
// couplings).  Plain C++, double precision.
#pragma once

#include <string>
#include <vector>

#include <cuda_fp16.h>

#include "common.cuh"

namespace umd {

struct HostModel {
    Dims d;
    double rc = 0, dx = 0;
    std::vector<float> table;      // [n_rows][3][CP]: c0, c1, packed (c2, c3) (see tab_pack)
    std::vector<float> pairmod;    // [T*T][2+R][C0]
    std::vector<float> X0, W1p, W2p, A1, A2, mu, inv_sigma;
    std::vector<std::vector<float>> theta, thetaT, bias;   // per hidden layer
    // half-precision splits of w_scale[t] * theta[t] (and of the transposes) for the tensor-core GEMM
    std::vector<std::vector<__half>> theta_hi, theta_lo, thetaT_hi, thetaT_lo;
    std::vector<float> w_scale;    // per layer, a power of two
    float grad_scale = 1.0f;       // power of two for the back-propagated gradients
    std::vector<float> type_bias;  // [T][F]: b_1 plus the first layer's image of the centre's calibrated initial features
    std::vector<float> w_head, e_ref;
    float b_head = 0;
    GauntSparse g123, g233;
    std::vector<GauntSparseBig> g4;   // (1,3,4), (2,2,4), (2,4,4), (3,3,4), (4,4,4) when L = 4
};

// Fills `d` widths for (C0, L, R); false when the triple is unsupported.
bool derive_dims(int C0, int L, int R, Dims* d);

// Returns UMLMD_OK or an error code with `err` set.
int build_host_model(const void* blob, size_t bytes, double table_dx_override, HostModel* out,
                     std::string* err);

}  // namespace umd
