"""B200-native NOVA pruned-scale step: thin Python binding over the C-ABI library libnova.so.

The binding only marshals arguments (torch tensors -> raw pointers and sizes); every step of
the path runs in the library's CUDA kernels. There is no CPU fallback: if libnova.so is
missing or cannot be loaded, importing this package fails.
"""
from .binding import (  # noqa: F401
    NovaError, Context, SchedParams, BlockWeights, BlockShape,
    nova_scale_entropy, nova_head_entropy, nova_keep_ratios, nova_select_topk,
    nova_pruned_block_forward, nova_restore_from_cache, nova_block_workspace_bytes,
    nova_pruned_block_forward_static, nova_static_scratch_bytes,
    nova_keep_ratios_device, nova_select_topk_device, nova_pruned_block_forward_device,
    nova_restore_from_cache_device, nova_pruned_block_forward_adaln, MODULATION_NAMES,
    nova_pruned_layer_forward, nova_pruned_block_forward_ext, EXTRA_NAMES, nova_score_mse, nova_score_attention_mass, nova_scale_entropy_layers, nova_keep_ratios_layers, nova_select_topk_grouped, nova_keep_ratios_layers_device,
    lib_path, STATUS_NAMES,
)
