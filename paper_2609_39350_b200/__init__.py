"""B200-native planner hot path of HAPMoE: a thin ctypes binding over libhap.so.

Every step of the path (layer costs, candidate decode, pipeline dynamic program, argmin)
runs in the CUDA kernels of the library; this package only marshals arguments.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library is missing
or no CUDA device is present, the calls raise.
"""
from .binding import (HapError, HapProblem, hap_problem_create, hap_enumerate, hap_get_pconfs, hap_decode,  # noqa: F401
                      hap_eval_layer_costs, hap_eval_layer_costs_f64, hap_pipeline_dp, hap_pipeline_dp_f64, hap_search_best,
                      hap_search_range_f64,
                      hap_search_range, hap_argmin, hap_argmin_static, hap_joint_bottleneck, hap_count_cells, hap_get_timings, hap_launches_per_pass, hap_eval_appendix_b, hap_simulate_1f1b, hap_release_cached_memory, hap_self_check, hap_problem_save, hap_problem_load, hap_problem_dims, hap_problem_destroy, load_library, EXPORTS, INF, COEF,
                      NCOEF, MAX_PP, OPT_NO_MAPTAB, OPT_REFINE, OPT_EXACT, OPT_UNIFORM, OPT_NO_TRIE, OPT_NO_FUSE, OPT_COUNT_SPLITS,
                      OPT_HETERO_DISPATCH)
