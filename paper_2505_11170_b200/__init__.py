"""B200 (sm_100a) implementation of the weight-sampling pass of Gaussian weight sampling.

``binding`` mirrors the C ABI of ``include/gws.h`` one to one (argument marshalling only);
``synthetic`` draws seeded inputs shaped like the paper's workloads.  There is no CPU fallback:
every call goes to the CUDA library and raises if it cannot be loaded.
"""
from . import synthetic  # noqa: F401
from .binding import (GwsError, Desc, MultiPlan, bitwidth, bitwidth_grad, bitwidth_loss, bitwidth_multi, bitwidth_grad_multi, layer_seed, group_absmax, kernel_class, launch_count, set_launch_overlap, load_library, n_groups,  # noqa: F401
                      noise, noise_alu_probe, issue_probe, issue_probe_mix, sample_fwd_compare, noise_compare, NOISE_UNIFORM_BF16, NOISE_BOX_MULLER, philox_words, gemm_fused, sample_bwd, sample_fwd, sample_fwd_mx, mx_layout, mx_quantize, MX_FP8_E4M3, MX_FP6_E3M2, MX_FP8_E3M4, sample_fwd_scaled, scale_from_absmax, sample_fwd_multi_static, sample_step_host, status_string)
