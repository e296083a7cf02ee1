"""B200-native bytecode virtual machine for fused dynamic tensor operators.

The product is the C-ABI library ``libdvm.so`` (see ``include/dvm.h``); this
package is its thin ctypes binding.  There is no CPU fallback: importing the
binding without the built library raises.
"""
from .binding import (  # noqa: F401
    DvmError, Program, Code, encode, launch, launch_stacked, run_host, verify, disassemble,
    code_info, last_device_status, launch_count, hardware_align_div, vm_tile_range,
    set_num_cores, get_num_cores, program_from_nodes, lib, LIB_PATH,
)
