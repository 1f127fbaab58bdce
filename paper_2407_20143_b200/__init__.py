"""B200-native load-time checkpoint resharding (arXiv 2407.20143): binding of libbcp.so."""
from .api import (BcpError, Plan, Stager, bcp_decompose, bcp_dedup_assign, bcp_pack, bcp_pack_cache_clear, bcp_pack_layout, bcp_pack_static, bcp_plan,
                  bcp_plan_device_status, bcp_reshard, bcp_reshard_host, bcp_safetensors_export, bcp_safetensors_layout, bcp_unpack, bcp_version)

__all__ = ["BcpError", "Plan", "Stager", "bcp_decompose", "bcp_dedup_assign", "bcp_pack", "bcp_pack_cache_clear", "bcp_pack_layout", "bcp_pack_static", "bcp_plan",
           "bcp_plan_device_status", "bcp_reshard", "bcp_reshard_host", "bcp_safetensors_export", "bcp_safetensors_layout", "bcp_unpack", "bcp_version"]
