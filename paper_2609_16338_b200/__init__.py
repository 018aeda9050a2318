"""BITCOS ternary GEMV for NVIDIA B200 (sm_100a).

A thin Python binding (argument marshalling only) over the C ABI declared in
``include/bitcos.h`` and implemented by ``csrc/`` as hand-written CUDA kernels plus C++ host
packers.  PyTorch is used for device memory and streams only.  There is no CPU fallback:
if ``libbitcos.so`` is missing, importing :mod:`paper_2609_16338_b200.binding` symbols that
need it raises.
"""
from .binding import (  # noqa: F401
    BitcosError,
    DeviceBitcos,
    DeviceExperts,
    DevicePlain,
    PackedBitcos,
    bit2_gemv,
    bit2_pack,
    bit2_unpack,
    bitcos_gemv,
    bitcos_gemv_grouped,
    bitcos_gemv_host,
    bitcos_gemv_host_staging_bytes,
    bitcos_gemv_static,
    bitcos_gemv_multi,
    MultiJobs,
    bitcos_gemv_multi_host,
    bitcos_quantize_activations,
    bitcos_gemv_group_scales,
    bitcos_gemv_bf16,
    bitcos_gemv_multi_bf16,
    bitcos_gemv_blend_bf16,
    bitcos_gemv_multi_group_scales,
    bitcos_choose_format,
    bitcos_count_nnz_device,
    bitcos_pack_device,
    MultiHostJobs,
    bitcos_decode_probe,
    bitcos_decode_probe_variant,
    PROBE_VARIANTS,
    group_pairs,
    plain_to_device,
    scales_tile,
    scales_untile,
    bitcos_gemv_workspace_bytes,
    bitcos_pack,
    bitcos_unpack,
    library_path,
    load_library,
    make_workspace,
    trit5_gemv,
    trit5_pack,
    trit5_unpack,
    workspace_status,
    EXPORTED_SYMBOLS,
)
