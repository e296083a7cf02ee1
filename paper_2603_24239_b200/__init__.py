"""B200-native bytecode virtual machine for fused dynamic tensor operators.

The product is the C-ABI library ``libdvm.so`` (see ``include/dvm.h``); this
package is its thin ctypes binding (``paper_2603_24239_b200.binding``, loaded on
first use so that ``paper_2603_24239_b200.build`` can run before the library
exists).  There is no CPU fallback: using the binding without the built
library raises.
"""
import importlib

_BINDING_NAMES = (
    "DvmError", "Program", "Code", "Encoder", "encode", "launch", "launch_stacked", "run_host", "verify",
    "disassemble", "code_info", "last_device_status", "launch_count", "hardware_align_div",
    "vm_tile_range", "set_num_cores", "get_num_cores", "set_elems_per_thread", "set_min_resident_ctas", "set_stacked_one_slot", "set_matmul_tail_split", "set_matmul_cta_pairs", "matmul_tail_plan", "last_launch_variant", "set_lean_kernel", "program_from_nodes",
    "BatchEncoder", "selftest_bounded_wait", "Fuser", "tensor_extents", "launch_checked",
    "lib", "LIB_PATH",
)


def __getattr__(name):
    if name == "binding" or name in _BINDING_NAMES:
        b = importlib.import_module(".binding", __name__)
        return b if name == "binding" else getattr(b, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
