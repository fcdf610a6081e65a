"""CPU checker for the OCS hot path.  Test infrastructure only (see ocs_oracle.h)."""
