// placeholder until the MLP families are wired in
#include "ops.cuh"
namespace betty {
betty_status mlpfam_validate(const betty_level*) { return BETTY_ERR_UNSUPPORTED; }
size_t mlpfam_workspace(const betty_level*) { return 0; }
betty_status mlpfam_grad(Ctx&, const betty_level*, const betty_level*, float*) { return BETTY_ERR_UNSUPPORTED; }
betty_status mlpfam_hvp_begin(Ctx&, const betty_level*, MlpHvpCache**) { return BETTY_ERR_UNSUPPORTED; }
betty_status mlpfam_hvp(Ctx&, const betty_level*, MlpHvpCache*, const float*, float*) { return BETTY_ERR_UNSUPPORTED; }
betty_status mlpfam_mixed(Ctx&, const betty_level*, MlpHvpCache*, const betty_level*, const float*, float*) { return BETTY_ERR_UNSUPPORTED; }
betty_status mlpfam_lower_step(Ctx&, const betty_level*, int) { return BETTY_ERR_UNSUPPORTED; }
betty_status mlpfam_fd(Ctx&, const betty_level*, const betty_level*, const float*, const float*, float, float, float*, bool) { return BETTY_ERR_UNSUPPORTED; }
}
