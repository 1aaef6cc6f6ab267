"""B200-native draft attention for Windowed-MTP: ring-buffer KV store, windowed and full-context
split-KV decode attention, behind the C ABI of include/wmtp.h (libwmtp.so)."""
from .binding import *  # noqa: F401,F403
from .binding import LIB_PATH, KV, Ring, Workspace, WmtpError, lib  # noqa: F401
