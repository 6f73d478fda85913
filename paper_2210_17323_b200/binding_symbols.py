"""Names the C-ABI library exports (every symbol include/gptq_b200.h declares).  No CUDA needed to import."""
EXPORTS = (
    "gptq_status_string", "gptq_launch_count", "gptq_debug_wait_test",
    "gptq_hessian_workspace_bytes", "gptq_hessian_accumulate", "gptq_hessian_accumulate_upper", "gptq_hessian_symmetrize",
    "gptq_prepare_hinv_workspace_bytes", "gptq_prepare_hinv", "gptq_prepare_hinv_static", "gptq_prepare_factor",
    "gptq_quantize_workspace_bytes", "gptq_quantize_layer", "gptq_quantize_layer_factor", "gptq_set_stage3_variant",
    "gptq_solve_layer_host_workspace_bytes", "gptq_solve_layer_host",
    "gptq_solve_layer_host_grids_workspace_bytes", "gptq_solve_layer_host_grids",
    "gptq_rtn_layer", "gptq_dequantize", "gptq_matvec",
)
