"""B200 (sm_100a) tANS weight decoder: thin Python face of the C-ABI library."""
from .binding import *  # noqa: F401,F403
from .binding import lib, lib_path, ans_layer_desc, AnsError  # noqa: F401
